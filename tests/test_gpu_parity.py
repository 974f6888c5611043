"""GPU parity: the CUDA library (through its C ABI) against the float64 CPU oracle,
element by element on the same seeded bf16 inputs.

Tolerances (stated for the plasticity path): row-normalised Gram entries within 1e-4
absolute; loss within 1e-3 relative or 1e-7 absolute; freeze masks identical except
where the oracle's |slope| is within 1e-6 of T.
"""
from pathlib import Path

import numpy as np
import pytest
import torch

import oracle
from paper_2201_06227_b200 import binding as eg
from paper_2201_06227_b200 import workloads as wl

pytestmark = pytest.mark.gpu

GOLDEN = Path(__file__).parent / "golden"
ENTRY_ATOL = 1e-4
LOSS_RTOL, LOSS_ATOL = 1e-3, 1e-7
DEV = "cuda"


def assert_loss_close(gpu, ref, what=""):
    gpu, ref = np.asarray(gpu, dtype=np.float64), np.asarray(ref, dtype=np.float64)
    tol = np.maximum(LOSS_RTOL * np.abs(ref), LOSS_ATOL)
    bad = ~(np.abs(gpu - ref) <= tol)
    assert not bad.any(), f"{what} loss mismatch at {np.nonzero(bad)[0]}: gpu={gpu[bad]} oracle={ref[bad]}"


def run_gpu(at, ar, flags=0, keep=False, W=5, T=1e-3):
    """One evaluation through the C ABI.  at/ar: lists of CUDA bf16 [b, d_m] tensors."""
    b = at[0].shape[0]
    d = [t.shape[1] for t in at]
    ctx = eg.Context(d, b, W, T, flags | (eg.FLAG_KEEP_GRAMS if keep else 0), device=DEV)
    losses = ctx.egeria_sp_loss_batch(at, ar)
    grams = [ctx.egeria_debug_dump_gram(m, b) for m in range(len(d))] if keep else None
    ctx.check_device_status()
    out = losses.cpu().numpy()
    if keep:
        grams = [(g[0].cpu().numpy(), g[1].cpu().numpy()) for g in grams]
    ctx.close()
    return out, grams


def compare_with_oracle(at, ar, flags=0, what=""):
    losses, grams = run_gpu(at, ar, flags, keep=True)
    for m, (t, r) in enumerate(zip(at, ar)):
        ref, gt, gr = oracle.sp_loss(wl.bf16_bits(t), wl.bf16_bits(r), return_grams=True)
        np.testing.assert_allclose(grams[m][0], gt, rtol=0, atol=ENTRY_ATOL, err_msg=f"{what} G~_T module {m}")
        np.testing.assert_allclose(grams[m][1], gr, rtol=0, atol=ENTRY_ATOL, err_msg=f"{what} G~_R module {m}")
        assert_loss_close(losses[m:m + 1], [ref], f"{what} module {m}")
    return losses


# ----------------------------------------------------------------------------- small shapes

SMALL_B = [2, 3, 8, 17, 32, 64, 65, 100, 128, 129, 200, 256]
SMALL_D = [8, 64, 72, 4096, 4104]


@pytest.mark.parametrize("b", SMALL_B)
@pytest.mark.parametrize("d", SMALL_D)
def test_single_module_tensor_core_path(b, d):
    kind = "relu" if (b + d) % 2 == 0 else "normal"
    at, ar = wl.make_pair(b, d, kind, 0.3, seed=1000 * b + d, device=DEV)
    compare_with_oracle([at], [ar], what=f"b={b} d={d}")


@pytest.mark.parametrize("b,d", [(8, 64 * 148 * 9), (32, 64 * 148 * 12 + 72), (33, 64 * 148 * 9), (64, 64 * 148 * 10),
                                 (128, 64 * 148 * 5), (256, 64 * 148 * 4)])
def test_single_module_cut_over_every_cta(b, d):
    """One module alone over all 148 CTAs: a row of G has 148 partial rows per side.  At b <= 64
    the finalisation then runs in two levels ((row, chunk) tasks, chunk sums in scratch); entries
    and loss against the oracle, and the same bits on a second evaluation."""
    at, ar = wl.make_pair(b, d, "relu" if b % 2 else "normal", 0.25, seed=31 * b + 7, device=DEV)
    losses = compare_with_oracle([at], [ar], flags=eg.FLAG_EQUAL_SPLIT, what=f"alone b={b} d={d}")
    again, _ = run_gpu([at], [ar], flags=eg.FLAG_EQUAL_SPLIT)
    assert again.tobytes() == losses.tobytes()


@pytest.mark.parametrize("b,d", [(2, 1), (5, 7), (8, 100), (64, 1001), (100, 333), (130, 250), (256, 65)])
def test_single_module_cuda_core_path_for_unaligned_d(b, d):
    at, ar = wl.make_pair(b, d, "normal", 0.3, seed=77 + b + d, device=DEV)
    compare_with_oracle([at], [ar], what=f"b={b} d={d}")


@pytest.mark.parametrize("b", [8, 64, 128, 256])
def test_forced_cuda_core_path_matches_oracle(b):
    at, ar = wl.make_pair(b, 2048, "relu", 0.2, seed=5 + b, device=DEV)
    compare_with_oracle([at], [ar], flags=eg.FLAG_FORCE_SIMT, what=f"simt b={b}")


def test_misaligned_pointer_takes_cuda_core_path():
    b, d = 16, 264
    base_t = torch.zeros(b * d + 8, dtype=torch.bfloat16, device=DEV)
    base_r = torch.zeros(b * d + 8, dtype=torch.bfloat16, device=DEV)
    t, r = wl.make_pair(b, d, "normal", 0.3, seed=9, device=DEV)
    at = base_t[1:1 + b * d].view(b, d)   # 2-byte offset: not 16-byte aligned
    ar = base_r[1:1 + b * d].view(b, d)
    at.copy_(t)
    ar.copy_(r)
    assert at.data_ptr() % 16 != 0
    compare_with_oracle([at], [ar], what="misaligned")


@pytest.mark.parametrize("b", [24, 96, 160])
def test_many_modules_mixed_sizes(b):
    """Several tiles per CTA, K-ranges cut inside modules, ragged tails, one unaligned module."""
    ds = [64, 8, 4104, 12345 * 8, 520, 1001, 30000, 72, 96 * 64]
    at, ar = [], []
    for m, d in enumerate(ds):
        t, r = wl.make_pair(b, d, "relu" if m % 2 else "normal", 0.05 + 0.05 * m, seed=300 + m, device=DEV)
        at.append(t)
        ar.append(r)
    compare_with_oracle(at, ar, what=f"mixed b={b}")


@pytest.mark.parametrize("b", [5, 33, 70, 130])
def test_hundreds_of_small_modules(b):
    """More modules than CTAs: whole modules inside one CTA's range, many units per CTA, the scan
    over other modules longer than one warp, a few CUDA-core modules in between; evaluated
    repeatedly (the progress counters alternate between two sets)."""
    rng = np.random.default_rng(b)
    M = 200
    ds = [int(rng.integers(1, 200)) * 8 for _ in range(M)]
    for m in (3, 77, 150):
        ds[m] += 3                                           # not a multiple of 8: CUDA-core path
    at, ar = [], []
    for m, d in enumerate(ds):
        t, r = wl.make_pair(b, d, "relu" if m % 3 else "normal", 0.02 + 0.002 * m, seed=5000 + m, device=DEV)
        at.append(t)
        ar.append(r)
    ref = oracle.sp_loss_batch([wl.bf16_bits(t) for t in at], [wl.bf16_bits(r) for r in ar])
    ctx = eg.Context(ds, b, 4, 1e-3, device=DEV)
    for rep in range(3):
        losses, slopes, mask = ctx.egeria_plasticity_evaluate(at, ar)
        assert_loss_close(losses.cpu().numpy(), ref, f"many modules b={b} rep={rep}")
    ctx.check_device_status()
    # three identical readings per module: slope 0 from the second on, not yet frozen (W = 4)
    assert np.all(slopes.cpu().numpy() == 0.0) and not mask.cpu().numpy().any()
    ctx.close()


@pytest.mark.parametrize("seed", range(4))
def test_random_shapes_repeat_bit_for_bit(seed):
    """Random b, module counts and sizes; six evaluations each: every one within tolerance of the
    oracle, and with the equal split all six bit-identical (the in-kernel finalisation must not
    depend on which CTA or warp did what)."""
    rng = np.random.default_rng(900 + seed)
    for _ in range(10):
        b = int(rng.choice([2, 7, 16, 31, 32, 33, 48, 64, 65, 100, 128, 129, 192, 256]))
        M = int(rng.choice([1, 2, 5, 13, 40]))
        top = 4000 if rng.random() < 0.3 else 300
        ds = [int(rng.integers(1, top)) * 8 for _ in range(M)]
        if M > 2 and rng.random() < 0.3:
            ds[int(rng.integers(M))] += 5                    # one CUDA-core module
        if b >= 128 and M >= 40:
            ds = [min(d, 2048) for d in ds]                  # keeps the oracle quick
        at, ar = [], []
        for m, d in enumerate(ds):
            t, r = wl.make_pair(b, d, "relu" if m % 2 else "normal", 0.02 + 0.3 * rng.random(),
                                seed=int(rng.integers(1 << 30)), device=DEV)
            at.append(t)
            ar.append(r)
        ref = oracle.sp_loss_batch([wl.bf16_bits(t) for t in at], [wl.bf16_bits(r) for r in ar])
        ctx = eg.Context(ds, b, 4, 1e-3, eg.FLAG_EQUAL_SPLIT, device=DEV)
        outs = [ctx.egeria_plasticity_evaluate(at, ar)[0].cpu().numpy().copy() for _ in range(6)]
        ctx.check_device_status()
        ctx.close()
        for o in outs:
            assert_loss_close(o, ref, f"random b={b} M={M}")
            assert o.tobytes() == outs[0].tobytes()


# ----------------------------------------------------------------------------- closed forms / invariants on the GPU

def _fixture_cases():
    for line in (GOLDEN / "sp_loss_closed_forms.txt").read_text().splitlines():
        if not line.strip() or line.startswith("#"):
            continue
        name, b, d, at, ar, exp = [f.strip() for f in line.split("|")]
        parse = lambda s: [[float(v) for v in row.split()] for row in s.split(";")]
        yield pytest.param(parse(at), parse(ar), float(exp), id=name)


@pytest.mark.parametrize("at,ar,expected", list(_fixture_cases()))
def test_closed_form_fixture_on_gpu(at, ar, expected):
    t = torch.tensor(at, dtype=torch.bfloat16, device=DEV)
    r = torch.tensor(ar, dtype=torch.bfloat16, device=DEV)
    losses, _ = run_gpu([t], [r])
    assert_loss_close(losses, [expected])


@pytest.mark.parametrize("b,d", [(8, 4096), (64, 8192), (128, 4096), (256, 2048)])
def test_invariants_on_gpu(b, d):
    at, ar = wl.make_pair(b, d, "relu", 0.2, seed=b + d, device=DEV)
    base, _ = run_gpu([at], [ar])
    same, _ = run_gpu([at], [at.clone()])
    assert abs(same[0]) <= 1e-7
    again, _ = run_gpu([at], [ar])
    assert again[0].tobytes() == base[0].tobytes()              # deterministic
    scaled, _ = run_gpu([at * 4.0], [ar * 0.125])               # exact in bf16, exact in fp32
    assert scaled[0].tobytes() == base[0].tobytes()
    perm = torch.randperm(b, generator=torch.Generator().manual_seed(1)).to(DEV)
    permuted, _ = run_gpu([at[perm].contiguous()], [ar[perm].contiguous()])
    assert_loss_close(permuted, base.astype(np.float64))


def test_nan_propagates_and_zero_rows_are_clamped():
    at, ar = wl.make_pair(16, 256, "normal", 0.2, seed=3, device=DEV)
    z = at.clone()
    z[5] = 0
    losses, grams = run_gpu([z], [ar], keep=True)
    assert np.all(grams[0][0][5] == 0.0) and np.isfinite(losses).all()
    ref = oracle.sp_loss(wl.bf16_bits(z), wl.bf16_bits(ar))
    assert_loss_close(losses, [ref])
    n = at.clone()
    n[2, 7] = float("nan")
    losses, _ = run_gpu([n], [ar])
    assert np.isnan(losses[0])


@pytest.mark.parametrize("b,d", [(16, 256), (64, 64 * 148 * 3), (128, 4096)])
def test_nan_of_any_bit_pattern_is_a_value_not_a_missing_row(b, d):
    """The finish tells a partial row that has arrived from one that has not by its contents: the
    bit pattern that means "not here yet" is a NaN.  Inputs that are NaNs with every payload bit set
    (and infinities, whose products and differences are NaNs too) must come out as a NaN loss like
    any other NaN -- not as a wait that runs out -- and leave the context as it was."""
    at, ar = wl.make_pair(b, d, "normal", 0.2, seed=11 + b, device=DEV)
    ctx = eg.Context([d], b, 5, 1e-3, eg.FLAG_EQUAL_SPLIT, device=DEV)
    good = ctx.egeria_sp_loss_batch([at], [ar]).cpu().numpy().copy()
    for bits, where in ((-1, (1, 5)), (0x7F80, (0, 0)), (-128, (b - 1, d - 1))):   # 0xFFFF, +Inf, 0xFF80 = -Inf
        n = at.clone()
        n.view(torch.int16)[where] = bits
        m = ar.clone()
        m.view(torch.int16)[where] = bits
        losses = ctx.egeria_sp_loss_batch([n], [m]).cpu().numpy()
        assert ctx.egeria_device_status() == eg.OK
        assert np.isnan(losses[0]), (hex(bits & 0xFFFF), losses)
        again = ctx.egeria_sp_loss_batch([at], [ar]).cpu().numpy()
        assert again.tobytes() == good.tobytes()
    ctx.close()


# ----------------------------------------------------------------------------- named workloads

def test_tiny_workload_full():
    w = wl.WORKLOADS["tiny"]
    at, ar = wl.make_activations(w, DEV)
    compare_with_oracle(at, ar, what="tiny")


def test_resnet56_workload_full():
    w = wl.WORKLOADS["resnet56"]
    at, ar = wl.make_activations(w, DEV)
    compare_with_oracle(at, ar, what="resnet56")


def test_bert_base_workload_full():
    w = wl.WORKLOADS["bert_base"]
    at, ar = wl.make_activations(w, DEV)
    compare_with_oracle(at, ar, what="bert_base")


def _sampled_check(name, full_modules, row_modules, rows):
    """Full-size workload in the benchmark's launch configuration -- the call bench.py times
    (egeria_plasticity_evaluate), first with the equal split and again once the adaptive split
    has settled.  The oracle gives the loss of EVERY module; every entry of the normalised Grams
    of a few modules and sampled rows of others are compared as well."""
    w = wl.WORKLOADS[name]
    at, ar = wl.make_activations(w, DEV)
    full_ref = {m: oracle.sp_loss(wl.bf16_bits(at[m]), wl.bf16_bits(ar[m]), return_grams=True) for m in full_modules}
    loss_ref = np.array([full_ref[m][0] if m in full_ref else oracle.sp_loss(wl.bf16_bits(at[m]), wl.bf16_bits(ar[m]))
                         for m in range(w.M)])
    row_ref = {}
    for m in row_modules:
        for side, acts in enumerate((at, ar)):
            bits = wl.bf16_bits(acts[m])
            for i in rows:
                g = oracle.gram_row(bits, i)
                row_ref[(m, side, i)] = g / max(np.linalg.norm(g), oracle.EPS)
    ctx = eg.Context(list(w.d), w.b, w.W, float(np.float32(w.T)), eg.FLAG_KEEP_GRAMS, device=DEV)

    def check(what):
        losses = ctx.egeria_plasticity_evaluate(at, ar)[0].cpu().numpy()
        grams = [tuple(g.cpu().numpy() for g in ctx.egeria_debug_dump_gram(m, w.b)) for m in range(w.M)]
        ctx.check_device_status()
        assert_loss_close(losses, loss_ref, f"{name}, all {w.M} modules ({what})")
        for m, (ref, gt, gr) in full_ref.items():
            np.testing.assert_allclose(grams[m][0], gt, rtol=0, atol=ENTRY_ATOL)
            np.testing.assert_allclose(grams[m][1], gr, rtol=0, atol=ENTRY_ATOL)
        for (m, side, i), gn in row_ref.items():
            np.testing.assert_allclose(grams[m][side][i], gn, rtol=0, atol=ENTRY_ATOL)
        # properties that hold at any size: unit rows, symmetric-positive diagonal
        for m in range(w.M):
            for side in (0, 1):
                np.testing.assert_allclose(np.linalg.norm(grams[m][side].astype(np.float64), axis=1), 1.0, atol=1e-5)
                assert np.all(np.diag(grams[m][side]) > 0)
        return losses

    first = check("equal split")
    for _ in range(15):
        ctx.egeria_plasticity_evaluate(at, ar)[0].cpu()       # .cpu() waits: the launch logs land
    assert ctx.egeria_split_weights()[0] > 0                  # the shares were measured (and kept, or found no better than equal ones)
    settled = check("adaptive split")
    assert_loss_close(settled, first.astype(np.float64), f"{name} adaptive vs equal split")
    ctx.close()


def test_resnet50_workload_sampled():
    _sampled_check("resnet50", full_modules=[0, 5, 15], row_modules=[3, 9, 12], rows=[0, 31, 63])


def test_gpt2_medium_workload_sampled():
    _sampled_check("gpt2_medium", full_modules=[0, 23], row_modules=[7, 11, 16], rows=[0, 127, 128, 255])


# ----------------------------------------------------------------------------- host entry point

def test_host_entry_matches_device_entry():
    ds, b = [4096, 520, 1001], 48
    at, ar = [], []
    for m, d in enumerate(ds):
        t, r = wl.make_pair(b, d, "relu", 0.2, seed=40 + m, device="cpu")
        at.append(t.pin_memory())
        ar.append(r.pin_memory())
    ctx = eg.Context(ds, b, 5, 1e-3, eg.FLAG_HOST_STAGING | eg.FLAG_EQUAL_SPLIT, device=DEV)
    host = ctx.egeria_sp_loss_batch_host(at, ar).numpy().copy()
    dev = ctx.egeria_sp_loss_batch([t.to(DEV) for t in at], [r.to(DEV) for r in ar]).cpu().numpy()
    assert host.tobytes() == dev.tobytes()
    ref = oracle.sp_loss_batch([wl.bf16_bits(t) for t in at], [wl.bf16_bits(r) for r in ar])
    assert_loss_close(host, ref)
    ctx.close()


def test_call_error_paths():
    at, ar = wl.make_pair(8, 64, "normal", 0.1, seed=1, device=DEV)
    ctx = eg.Context([64], 8, 5, 1e-3, device=DEV)
    big_t, big_r = wl.make_pair(16, 64, "normal", 0.1, seed=1, device=DEV)
    with pytest.raises(eg.EgeriaError) as e:
        ctx.egeria_sp_loss_batch([big_t], [big_r])       # b > b_max
    assert e.value.status == eg.ERR_INVALID_ARG
    with pytest.raises(eg.EgeriaError) as e:
        ctx.egeria_sp_loss_batch_host([at.cpu()], [ar.cpu()])   # no staging reserved
    assert e.value.status == eg.ERR_WORKSPACE
    with pytest.raises(eg.EgeriaError) as e:
        ctx.egeria_debug_dump_gram(0, 8)                 # grams not kept
    assert e.value.status == eg.ERR_WORKSPACE
    out = ctx.egeria_sp_loss_batch([at], [ar])           # still usable afterwards
    assert np.isfinite(out.cpu().numpy()).all()
    ctx.close()


def test_raw_abi_argument_errors_leave_the_context_usable():
    """Requirements checked on the host and reported as status codes, through the raw C ABI (the
    binding would not let these through): a d[] that differs from creation, a NULL module
    pointer, an odd pointer, a NULL output, NULL arrays -- each EGERIA_ERR_INVALID_ARG, nothing
    launched, and the same context evaluates correctly afterwards."""
    import ctypes
    L = eg.lib()
    ds, b = [4096, 520], 24
    at, ar = [], []
    for m, d in enumerate(ds):
        t, r = wl.make_pair(b, d, "normal", 0.2, seed=70 + m, device=DEV)
        at.append(t)
        ar.append(r)
    ctx = eg.Context(ds, b, 5, 1e-3, device=DEV)
    out = torch.full((2,), -3.0, dtype=torch.float32, device=DEV)
    sp = int(torch.cuda.current_stream().cuda_stream)
    good_t, good_r = ctx._ptr_array(at, b, True), ctx._ptr_array(ar, b, True)
    d_ok = (ctypes.c_int64 * 2)(*ds)
    launched = ctx.egeria_launch_count()

    def call(pt, pr, d_arr, out_ptr, bb=b):
        return L.egeria_sp_loss_batch(ctx._h, sp, pt, pr, bb, d_arr, out_ptr)

    def ptrs(a, c):
        arr = (ctypes.c_void_p * 2)()
        arr[0], arr[1] = a, c
        return arr

    assert call(good_t, good_r, (ctypes.c_int64 * 2)(4096, 528), out.data_ptr()) == eg.ERR_INVALID_ARG   # d[] mismatch
    assert call(ptrs(at[0].data_ptr(), None), good_r, d_ok, out.data_ptr()) == eg.ERR_INVALID_ARG        # NULL module
    assert call(good_t, ptrs(ar[0].data_ptr(), ar[1].data_ptr() + 1), d_ok, out.data_ptr()) == eg.ERR_INVALID_ARG  # odd
    assert call(good_t, good_r, d_ok, None) == eg.ERR_INVALID_ARG                                        # no output
    assert call(None, good_r, d_ok, out.data_ptr()) == eg.ERR_INVALID_ARG
    assert call(good_t, good_r, None, out.data_ptr()) == eg.ERR_INVALID_ARG
    assert call(good_t, good_r, d_ok, out.data_ptr(), bb=1) == eg.ERR_INVALID_ARG                        # b < 2
    assert L.egeria_sp_loss_batch(None, sp, good_t, good_r, b, d_ok, out.data_ptr()) == eg.ERR_INVALID_ARG
    assert L.egeria_plasticity_step(ctx._h, sp, None, None, None) == eg.ERR_INVALID_ARG
    assert L.egeria_plasticity_set_lr(None, ctypes.c_double(0.1)) == eg.ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert ctx.egeria_launch_count() == launched and np.all(out.cpu().numpy() == -3.0)   # nothing ran
    assert call(good_t, good_r, d_ok, out.data_ptr()) == eg.OK
    ref = oracle.sp_loss_batch([wl.bf16_bits(t) for t in at], [wl.bf16_bits(r) for r in ar])
    assert_loss_close(out.cpu().numpy(), ref)
    ctx.check_device_status()
    ctx.close()


def test_many_pointer_sets_enqueued_ahead_of_the_gpu():
    """A caller whose activation buffers are new on every call misses the plan cache every time.
    With the GPU held busy, far more than the 16 cached plans are enqueued before any of them has
    run: every evaluation must still see its own tensor maps and work split."""
    ds, b, n = [2048, 520, 4096], 40, 48
    sets, refs = [], []
    for k in range(n):
        at, ar = [], []
        for m, d in enumerate(ds):
            t, r = wl.make_pair(b, d, "relu", 0.05 + 0.01 * k, seed=3000 + 10 * k + m, device=DEV)
            at.append(t)
            ar.append(r)
        sets.append((at, ar))
    for k in (0, 17, 33, n - 1):
        refs.append((k, oracle.sp_loss_batch([wl.bf16_bits(t) for t in sets[k][0]],
                                             [wl.bf16_bits(r) for r in sets[k][1]])))
    ctx = eg.Context(ds, b, 5, 1e-3, eg.FLAG_EQUAL_SPLIT, device=DEV)
    one = eg.Context(ds, b, 5, 1e-3, eg.FLAG_EQUAL_SPLIT, device=DEV)
    want = [one.egeria_sp_loss_batch(at, ar).cpu().numpy().copy() for at, ar in sets]   # one at a time
    outs = [torch.empty(len(ds), dtype=torch.float32, device=DEV) for _ in range(n)]
    big = torch.randn(8192, 8192, device=DEV)
    torch.cuda.synchronize()
    for _ in range(40):                       # some tens of milliseconds of work ahead of the evaluations
        big = torch.mm(big, big).clamp_(-1, 1)
    for k, (at, ar) in enumerate(sets):
        ctx.egeria_sp_loss_batch(at, ar, outs[k])
    torch.cuda.synchronize()
    ctx.check_device_status()
    for k in range(n):
        assert outs[k].cpu().numpy().tobytes() == want[k].tobytes(), f"evaluation {k}"
    for k, ref in refs:
        assert_loss_close(outs[k].cpu().numpy(), ref, f"evaluation {k}")
    ctx.close()
    one.close()


@pytest.mark.parametrize("kind", [1, 2])
@pytest.mark.parametrize("b,ds", [(64, [64 * 148 * 40]), (128, [64 * 148 * 3] * 6), (128, [64 * 148 * 2] * 15),
                                  (256, [64 * 148 * 8] * 3)])
def test_a_bounded_wait_that_runs_out_is_reported_and_the_context_recovers(kind, b, ds):
    """The give-up path of the evaluation kernel, in the form that returns: one hand-shake of the
    first thread block is left out for ONE launch whose waits are limited to a millisecond.  The
    kernel returns, the status word says EGERIA_ERR_TIMEOUT (once), and the next evaluation on
    the same context matches the oracle.  Where the finish tells an arrived partial row by its
    contents (the warps that wait for the first block's partial give up), and where it goes by the
    unit counters (more rows than warps, or b = 256); the modules the first block did not work on
    are finished all the same."""
    # every thread block gets 36 to 60 blocks of 64 features: more than the 12 (6 at b = 256) pipeline stages
    _, _, validate = eg.egeria_debug_plan_tasks(ds, b, 148)
    assert validate == (b <= 128 and len(ds) < 15)
    at, ar = [], []
    for m, d in enumerate(ds):
        t, r = wl.make_pair(b, d, "relu", 0.2, seed=4242 + m, device=DEV)
        at.append(t)
        ar.append(r)
    ref = oracle.sp_loss_batch([wl.bf16_bits(t) for t in at], [wl.bf16_bits(r) for r in ar])
    ctx = eg.Context(ds, b, 5, 1e-3, eg.FLAG_EQUAL_SPLIT, device=DEV)
    good = ctx.egeria_sp_loss_batch(at, ar).cpu().numpy().copy()
    assert_loss_close(good, ref)
    out = torch.full((len(ds),), -5.0, dtype=torch.float32, device=DEV)
    ctx.egeria_debug_stall_next(kind)
    ctx.egeria_sp_loss_batch(at, ar, out)
    assert ctx.egeria_device_status() == eg.ERR_TIMEOUT
    got = out.cpu().numpy()
    assert got[0] == -5.0                          # no loss for the module the stalled block worked on
    done = got != -5.0
    assert got[done].tobytes() == good[done].tobytes()
    assert ctx.egeria_device_status() == eg.OK     # reported once; counters and slots start afresh
    for _ in range(3):                             # both sets of progress counters come round
        again = ctx.egeria_sp_loss_batch(at, ar).cpu().numpy()
        assert again.tobytes() == good.tobytes()
    ctx.check_device_status()
    ctx.close()


def test_the_two_ways_of_finishing_alternate_on_one_context():
    """One context, evaluations that alternate between batch sizes at which the finish validates
    partial rows by their contents (two sets of slots in turn, each launch emptying what the one
    before wrote) and some at which it goes by the unit counters (b > 128: the slots stay as
    written and are cleared before the next evaluation of the first kind), a CUDA-core module
    among them: every evaluation against the oracle."""
    ds = [4096] * 6 + [1001, 8192]
    M = len(ds)
    big = [wl.make_pair(160, d, "relu" if m % 2 else "normal", 0.1 + 0.02 * m, seed=600 + m, device=DEV) for m, d in enumerate(ds)]
    assert not eg.egeria_debug_plan_tasks(ds, 160, 148)[2] and eg.egeria_debug_plan_tasks(ds, 24, 148)[2]
    ctx = eg.Context(ds, 160, 5, 1e-3, device=DEV)
    refs = {}
    for rep, b in enumerate([160, 24, 24, 128, 160, 160, 24, 100, 64, 24, 130, 128]):
        at = [t[:b].contiguous() for t, _ in big]
        ar = [r[:b].contiguous() for _, r in big]
        if b not in refs:
            refs[b] = oracle.sp_loss_batch([wl.bf16_bits(t) for t in at], [wl.bf16_bits(r) for r in ar])
        losses = ctx.egeria_sp_loss_batch(at, ar).cpu().numpy()
        assert_loss_close(losses, refs[b], f"evaluation {rep} b={b}")
    ctx.check_device_status()
    ctx.close()


@pytest.mark.parametrize("b,ds,extra", [(32, [98304] * 6, 0), (128, [16384, 8192, 4096, 4096, 520 * 8], 0),
                                        (64, [200704, 100352, 8200], 0), (256, [65536, 32768], 0),
                                        (40, [4096, 2048, 8192, 1024], "front_only")])
def test_overlapped_evaluations_give_the_same_results(b, ds, extra):
    """EGERIA_FLAG_OVERLAP: consecutive evaluations overlap on the GPU (the next one streams while
    the previous one finishes its modules).  Enqueued back to back without any synchronisation,
    on inputs that alternate between two sets, every evaluation must give bit for bit what the
    same sequence gives without the flag -- losses, slopes and masks (the rule's state is carried
    from evaluation to evaluation) -- and the first one must match the oracle."""
    n_eval, M = 24, len(ds)
    sets = []
    for k in range(2):
        at, ar = [], []
        for m, d in enumerate(ds):
            t, r = wl.make_pair(b, d, "relu" if m % 2 else "normal", 0.05 + 0.1 * k + 0.02 * m, seed=8000 + 10 * k + m, device=DEV)
            at.append(t)
            ar.append(r)
        sets.append((at, ar))
    base = eg.FLAG_EQUAL_SPLIT | ((eg.FLAG_FRONTMOST | eg.FLAG_FRONT_ONLY) if extra == "front_only" else 0)
    T = 0.5 if extra == "front_only" else 1e-3
    results = {}
    for name, flags in (("plain", base), ("overlapped", base | eg.FLAG_OVERLAP)):
        ctx = eg.Context(ds, b, 3, T, flags, device=DEV)
        outs = [(torch.full((M,), -1.0, dtype=torch.float32, device=DEV), torch.zeros(M, dtype=torch.float64, device=DEV),
                 torch.zeros(M, dtype=torch.uint8, device=DEV)) for _ in range(n_eval)]
        sp = int(torch.cuda.current_stream().cuda_stream)
        ptrs = [(ctx._ptr_array(at, b, True), ctx._ptr_array(ar, b, True)) for at, ar in sets]
        for k in range(n_eval):                                  # no synchronisation in between
            pa, pr = ptrs[k % 2]
            ctx.plasticity_evaluate_raw(pa, pr, b, outs[k][0].data_ptr(), outs[k][1].data_ptr(), outs[k][2].data_ptr(), sp)
        torch.cuda.synchronize()
        ctx.check_device_status()
        results[name] = [tuple(t.cpu().numpy().copy() for t in o) for o in outs]
        ctx.close()
    for k in range(n_eval):
        for j in range(3):
            assert results["plain"][k][j].tobytes() == results["overlapped"][k][j].tobytes(), (k, j)
    if extra != "front_only":
        ref = oracle.sp_loss_batch([wl.bf16_bits(t) for t in sets[0][0]], [wl.bf16_bits(r) for r in sets[0][1]])
        assert_loss_close(results["overlapped"][0][0], ref)
        assert results["overlapped"][-1][2].all()                # constant alternating readings: everything froze
    else:
        assert results["overlapped"][-1][2].all()


def test_changing_b_and_pointers_between_calls():
    ctx = eg.Context([4096, 264], 128, 5, 1e-3, device=DEV)
    for b in (128, 8, 70, 8):
        at, ar = [], []
        for m, d in enumerate((4096, 264)):
            t, r = wl.make_pair(b, d, "relu", 0.2, seed=b + m, device=DEV)
            at.append(t)
            ar.append(r)
        got = ctx.egeria_sp_loss_batch(at, ar).cpu().numpy()
        ref = oracle.sp_loss_batch([wl.bf16_bits(t) for t in at], [wl.bf16_bits(r) for r in ar])
        assert_loss_close(got, ref, f"b={b}")
    ctx.check_device_status()
    ctx.close()


# ----------------------------------------------------------------------------- freezing rule

def first_freeze(stale, W):
    """Evaluation at which W consecutive stale evaluations are first complete, -1 if never."""
    run = 0
    for i, st in enumerate(stale):
        run = run + 1 if st else 0
        if run >= W:
            return i
    return -1


def masks_agree(gpu_mask, gpu_fe, hist, W, T, signed=False):
    """Freeze decisions of a whole-history replay against the oracle's.  The stated criterion
    exempts a decision where the oracle's |slope| is within 1e-6 of T; it is applied per
    evaluation: an evaluation that close to T may be counted either way.  Where every such
    choice gives the same freeze evaluation, the GPU must give exactly the oracle's; elsewhere it
    must lie between the earliest and the latest possible one.  Returns (modules compared
    exactly, of which converged, modules the oracle converged)."""
    exact = exact_conv = n_conv = 0
    for m in range(hist.shape[0]):
        ref = oracle.plasticity_replay(hist[m], W, T, signed_test=signed)
        n_conv += ref["converged"]
        # the slopes of all evaluations, also past the oracle's freeze (T = 0: nothing is ever stale)
        s = oracle.plasticity_replay(hist[m], W, 0.0, signed_test=False)["slopes"]
        v = s if signed else np.abs(s)
        usable = np.isfinite(v)
        near = usable & (np.abs(v - T) <= 1e-6)
        sure = usable & (v < T) & ~near
        lo, hi = first_freeze(sure | near, W), first_freeze(sure, W)
        fe, conv = int(gpu_fe[m]), bool(gpu_mask[m])
        assert conv == (fe >= 0)
        if lo == hi:
            assert ref["freeze_eval"] == lo                      # the oracle's own decision
            assert fe == lo and conv == ref["converged"], f"module {m}: gpu {fe}, oracle {lo}"
            exact += 1
            exact_conv += ref["converged"]
        else:
            assert lo >= 0 and (fe >= lo if hi < 0 else lo <= fe <= hi), f"module {m}: gpu {fe} outside [{lo}, {hi}]"
    return exact, exact_conv, n_conv


@pytest.mark.parametrize("name,level,tau_scale", [("resnet56", None, 1.0), ("resnet56", 1e-2, 1.0),
                                                  ("resnet50", 2e-2, 1.0), ("bert_base", 5e-3, 1.0),
                                                  ("gpt2_medium", 3e-2, 1.0), ("gpt2_medium", 3e-2, 0.04),
                                                  ("resnet50", 2e-2, 0.2)])
def test_replay_matches_oracle(name, level, tau_scale):
    """The workload's window and tolerance on synthetic histories.  tau_scale < 1 makes the slope
    cross T quickly (by more than 1e-6 per evaluation), so that the freeze evaluation of most
    modules does not hinge on an evaluation within 1e-6 of T and is compared exactly."""
    w = wl.WORKLOADS[name]
    levels = [1e-6 * (1 + l) for l in range(w.M)] if level is None else [level * (1 + 0.1 * l) for l in range(w.M)]
    hist = wl.make_history(w, levels, tau_scale=tau_scale)
    T32 = np.float32(w.T)
    ctx = eg.Context([64] * w.M, 8, w.W, float(T32), device=DEV)
    slopes, mask, fe = ctx.egeria_plasticity_replay(torch.from_numpy(hist).to(DEV))
    slopes, mask, fe = slopes.cpu().numpy(), mask.cpu().numpy(), fe.cpu().numpy()
    for m in range(w.M):
        ref = oracle.plasticity_replay(hist[m], w.W, float(T32))
        live = ~np.isnan(ref["slopes"])
        assert np.array_equal(np.isnan(slopes[m]), ~live) or not ref["converged"]
        np.testing.assert_allclose(slopes[m][live], ref["slopes"][live], rtol=1e-9, atol=1e-15)
    exact, exact_conv, n_conv = masks_agree(mask, fe, hist, w.W, float(T32))
    print(f"{name} tau_scale={tau_scale}: freeze decisions compared exactly for {exact}/{w.M} modules, "
          f"{exact_conv}/{n_conv} of the converged ones")
    if level is not None and name != "bert_base":
        assert 0 < n_conv, "the synthetic history should freeze some modules"
    if tau_scale < 1.0:
        assert n_conv >= w.M // 2 and 3 * exact_conv >= n_conv, "the mask comparison must not be empty"
    ctx.close()


@pytest.mark.parametrize("signed", [False, True])
def test_step_matches_replay_and_oracle(signed):
    M, W, T, H = 6, 4, np.float32(2e-3), 40
    rng = np.random.default_rng(5)
    k = np.arange(H)
    hist = np.stack([0.05 * np.exp(-k / (2.0 + 3 * m)) * (1 + 0.5 * (m % 2) * np.sin(k)) + 0.01
                     + 1e-4 * rng.normal(size=H) for m in range(M)]).astype(np.float32)
    flags = eg.FLAG_SIGNED_SLOPE if signed else 0
    ctx = eg.Context([64] * M, 8, W, float(T), flags, device=DEV)
    hist_dev = torch.from_numpy(hist).to(DEV)
    step_slopes = np.empty((M, H))
    step_mask = np.empty((M, H), dtype=np.uint8)
    for i in range(H):
        s, mk = ctx.egeria_plasticity_step(hist_dev[:, i].contiguous())
        step_slopes[:, i], step_mask[:, i] = s.cpu().numpy(), mk.cpu().numpy()
    for m in range(M):
        for i in (3, 10, H - 1):
            ref = oracle.plasticity_replay(hist[m, : i + 1], W, float(T), signed_test=signed)
            sl = ref["slopes"][np.isfinite(ref["slopes"]) | np.isinf(ref["slopes"])]
            near = np.any(np.abs(np.abs(sl[np.isfinite(sl)]) - T) <= 1e-6)
            if not near:
                assert bool(step_mask[m, i]) == ref["converged"]
            if not ref["converged"]:
                assert step_slopes[m, i] == pytest.approx(ref["slopes"][i], rel=1e-9, abs=1e-15)
    # a reset by hand with the window halved: what follows is the plain rule with W / 2, started
    # afresh on the readings that follow
    ctx.egeria_plasticity_reset(halve_W=True)
    assert ctx.egeria_plasticity_window() == 2
    tail = hist[:, ::-1].copy()                                 # rising readings this time
    tail_dev = torch.from_numpy(tail).to(DEV)
    for i in range(H):
        s, mk = ctx.egeria_plasticity_step(tail_dev[:, i].contiguous())
        step_slopes[:, i], step_mask[:, i] = s.cpu().numpy(), mk.cpu().numpy()
    compared = 0
    for m in range(M):
        ref = oracle.plasticity_replay(tail[m], 2, float(T), signed_test=signed)
        live = ~np.isnan(ref["slopes"])
        fin = live & np.isfinite(ref["slopes"])
        np.testing.assert_allclose(step_slopes[m][fin], ref["slopes"][fin], rtol=1e-9, atol=1e-15)
        assert np.all(np.isinf(step_slopes[m][live & ~fin]))
        sl = ref["slopes"][fin]
        if np.any(np.abs((sl if signed else np.abs(sl)) - T) <= 1e-6):
            continue
        want = np.zeros(H, dtype=np.uint8)
        if ref["converged"]:
            want[ref["freeze_eval"]:] = 1
        assert np.array_equal(step_mask[m], want)
        compared += 1
    assert compared >= M // 2
    ctx.close()


def test_evaluate_equals_separate_calls():
    """egeria_plasticity_evaluate = egeria_sp_loss_batch + egeria_plasticity_step, bit for bit."""
    ds, b, W, T = [4096, 520, 1001, 8192], 72, 3, float(np.float32(5e-4))
    fused = eg.Context(ds, b, W, T, eg.FLAG_EQUAL_SPLIT, device=DEV)
    split = eg.Context(ds, b, W, T, eg.FLAG_EQUAL_SPLIT, device=DEV)
    for k in range(8):
        at, ar = [], []
        for m, d in enumerate(ds):
            t, r = wl.make_pair(b, d, "relu", 0.3 / (1 + k), seed=500 + 10 * k + m, device=DEV)
            at.append(t)
            ar.append(r)
        l1, s1, m1 = fused.egeria_plasticity_evaluate(at, ar)
        l2 = split.egeria_sp_loss_batch(at, ar)
        s2, m2 = split.egeria_plasticity_step(l2)
        assert l1.cpu().numpy().tobytes() == l2.cpu().numpy().tobytes()
        assert s1.cpu().numpy().tobytes() == s2.cpu().numpy().tobytes()
        assert m1.cpu().numpy().tobytes() == m2.cpu().numpy().tobytes()
    ref = oracle.sp_loss_batch([wl.bf16_bits(t) for t in at], [wl.bf16_bits(r) for r in ar])
    assert_loss_close(l1.cpu().numpy(), ref)
    fused.check_device_status()
    fused.close()
    split.close()


@pytest.mark.parametrize("b,ds", [(64, [401408, 200704, 100352, 802816]), (256, [131072] * 5), (128, [65536] * 7)])
def test_adaptive_split_keeps_the_result(b, ds):
    """After three evaluations that fill every SM the shares follow the measured streaming
    rates; the losses stay within the tolerance of the equal split's, and with
    EGERIA_FLAG_EQUAL_SPLIT every evaluation gives the same bits."""
    at, ar = [], []
    for m, d in enumerate(ds):
        t, r = wl.make_pair(b, d, "relu", 0.05 + 0.05 * m, seed=7000 + m, device=DEV)
        at.append(t)
        ar.append(r)
    fixed = eg.Context(ds, b, 5, 1e-3, eg.FLAG_EQUAL_SPLIT, device=DEV)
    ref = [fixed.egeria_sp_loss_batch(at, ar).cpu().numpy().copy() for _ in range(3)]
    assert ref[0].tobytes() == ref[1].tobytes() == ref[2].tobytes()
    assert fixed.egeria_split_weights()[0] == 0
    fixed.close()
    ctx = eg.Context(ds, b, 5, 1e-3, device=DEV)
    outs = []
    for k in range(17):
        outs.append(ctx.egeria_sp_loss_batch(at, ar).cpu().numpy().copy())   # .cpu() waits: the logs have landed
    n, w = ctx.egeria_split_weights()
    assert n > 0 and len(w) == n
    assert np.all(w >= 0.5) and np.all(w <= 2.0) and abs(float(w.mean()) - 1.0) < 0.05
    assert outs[0].tobytes() == ref[0].tobytes()          # the first evaluations use the equal split
    for o in outs:
        assert_loss_close(o, ref[0].astype(np.float64), "adaptive split")
    assert outs[-1].tobytes() == outs[-2].tobytes() == outs[-3].tobytes()   # and the shares settle
    ctx.check_device_status()
    ctx.close()


def test_step_with_a_window_too_long_for_registers():
    """W > 128 takes the freezing rule's loop path; it must agree with the oracle too."""
    M, W, T, H = 3, 150, np.float32(1e-4), 400
    k = np.arange(H)
    hist = np.stack([0.02 * np.exp(-k / (20.0 + 30 * m)) + 0.003 + 1e-5 * np.cos(0.7 * k + m)
                     for m in range(M)]).astype(np.float32)
    ctx = eg.Context([64] * M, 8, W, float(T), device=DEV)
    hist_dev = torch.from_numpy(hist).to(DEV)
    slopes = np.empty((M, H))
    masks = np.empty((M, H), dtype=np.uint8)
    for i in range(H):
        s, mk = ctx.egeria_plasticity_step(hist_dev[:, i].contiguous())
        slopes[:, i], masks[:, i] = s.cpu().numpy(), mk.cpu().numpy()
    for m in range(M):
        ref = oracle.plasticity_replay(hist[m], W, float(T))
        live = np.isfinite(ref["slopes"])
        np.testing.assert_allclose(slopes[m][live], ref["slopes"][live], rtol=1e-9, atol=1e-15)
        sl = ref["slopes"][live]
        if not np.any(np.abs(np.abs(sl) - T) <= 1e-6):
            assert bool(masks[m, -1]) == ref["converged"]
    ctx.close()


# ----------------------------------------------------------------------------- policies around Algorithm 1

def _policy_histories(M, H, seed):
    rng = np.random.default_rng(seed)
    k = np.arange(H)
    return np.stack([0.3 * np.exp(-k / rng.uniform(2, 12)) * (1 + 0.2 * np.sin(0.9 * k + m)) + 0.01 * (m + 1)
                     + 1e-4 * rng.standard_normal(H) for m in range(M)]).astype(np.float32)


def _near_T(slopes, T):
    s = slopes[np.isfinite(slopes)]
    return bool(np.any(np.abs(np.abs(s) - T) <= 1e-6))


@pytest.mark.parametrize("W", [3, 10, 150])
def test_auto_tolerance_matches_oracle(W):
    M, H = 5, 420 if W > 100 else 90
    hist = _policy_histories(M, H, seed=W)
    ctx = eg.Context([64] * M, 8, W, 1.0, eg.FLAG_AUTO_T, device=DEV)      # the T given is ignored
    hist_dev = torch.from_numpy(hist).to(DEV)
    r_slopes, r_mask, r_fe = [t.cpu().numpy() for t in ctx.egeria_plasticity_replay(hist_dev)]
    step_masks = np.empty((M, H), dtype=np.uint8)
    step_slopes = np.empty((M, H))
    for i in range(H):
        s, mk = ctx.egeria_plasticity_step(hist_dev[:, i].contiguous())
        step_slopes[:, i], step_masks[:, i] = s.cpu().numpy(), mk.cpu().numpy()
    for m in range(M):
        ref = oracle.plasticity_replay_auto(hist[m], W)
        live = ~np.isnan(ref["slopes"])
        assert np.array_equal(np.isnan(r_slopes[m]), ~live)
        fin = live & np.isfinite(ref["slopes"])
        np.testing.assert_allclose(r_slopes[m][fin], ref["slopes"][fin], rtol=1e-9, atol=1e-15)
        np.testing.assert_allclose(step_slopes[m][fin], ref["slopes"][fin], rtol=1e-9, atol=1e-15)
        if not (np.isfinite(ref["T"]) and _near_T(ref["slopes"], ref["T"])):
            assert int(r_fe[m]) == ref["freeze_eval"]
            assert bool(r_mask[m]) == ref["converged"]
            want = np.zeros(H, dtype=np.uint8)
            if ref["converged"]:
                want[ref["freeze_eval"]:] = 1
            assert np.array_equal(step_masks[m], want)
    ctx.close()


@pytest.mark.parametrize("auto,H", [(False, 45), (True, 100)])
def test_frontmost_policy_matches_oracle(auto, H):
    M, W = 6, 4
    hist = _policy_histories(M, H, seed=77 + auto)
    T = np.linspace(4e-3, 1.2e-2, M).astype(np.float32)
    flags = eg.FLAG_FRONTMOST | (eg.FLAG_AUTO_T if auto else 0)
    ctx = eg.Context([64] * M, 8, W, T, flags, device=DEV)
    ref = oracle.frontmost_replay(hist, W, None if auto else T.astype(np.float64))
    assert 1 <= ref["frozen"] < M                              # the case is not a trivial one
    hist_dev = torch.from_numpy(hist).to(DEV)
    slopes, mask, fe = [t.cpu().numpy() for t in ctx.egeria_plasticity_replay(hist_dev)]
    assert fe.tolist() == ref["freeze_eval"].tolist()
    assert mask.tolist() == [1] * ref["frozen"] + [0] * (M - ref["frozen"])
    for i in range(H):
        l = ref["monitored"][i]
        for m in range(M):
            if m == l:
                if np.isfinite(ref["slopes"][i]):
                    assert slopes[m, i] == pytest.approx(ref["slopes"][i], rel=1e-9, abs=1e-15)
                else:
                    assert np.isinf(slopes[m, i])
            else:
                assert np.isnan(slopes[m, i])
    # the same through one evaluation at a time: prefix mask, slope of the monitored module
    for i in range(H):
        s, mk = ctx.egeria_plasticity_step(hist_dev[:, i].contiguous())
        s, mk = s.cpu().numpy(), mk.cpu().numpy()
        frozen_after = int(np.sum((ref["freeze_eval"] >= 0) & (ref["freeze_eval"] <= i)))
        assert mk.tolist() == [1] * frozen_after + [0] * (M - frozen_after)
        l = ref["monitored"][i]
        if np.isfinite(ref["slopes"][i]):
            assert s[l] == pytest.approx(ref["slopes"][i], rel=1e-9, abs=1e-15)
        assert np.all(np.isinf(s[l + 1:]))
    ctx.close()


def test_frontmost_policy_inside_the_fused_evaluation():
    """egeria_plasticity_evaluate with the frontmost policy: same decisions as the losses fed to
    egeria_plasticity_step of a second context."""
    ds, b, W = [4096, 2048, 1001, 8192], 40, 2
    flags = eg.FLAG_FRONTMOST | eg.FLAG_EQUAL_SPLIT
    fused = eg.Context(ds, b, W, 0.5, flags, device=DEV)       # a generous T: modules freeze quickly
    split = eg.Context(ds, b, W, 0.5, flags, device=DEV)
    seen = []
    for k in range(12):
        at, ar = [], []
        for m, d in enumerate(ds):
            t, r = wl.make_pair(b, d, "relu", 0.3, seed=800 + 10 * k + m, device=DEV)
            at.append(t)
            ar.append(r)
        l1, s1, m1 = fused.egeria_plasticity_evaluate(at, ar)
        l2 = split.egeria_sp_loss_batch(at, ar)
        s2, m2 = split.egeria_plasticity_step(l2)
        assert l1.cpu().numpy().tobytes() == l2.cpu().numpy().tobytes()
        assert s1.cpu().numpy().tobytes() == s2.cpu().numpy().tobytes()
        assert m1.cpu().numpy().tobytes() == m2.cpu().numpy().tobytes()
        seen.append(int(m1.sum()))
    assert seen == sorted(seen) and seen[-1] == len(ds) and seen[0] == 0   # froze front to back, all of them
    fused.close()
    split.close()


def test_subset_evaluation_touches_only_the_active_modules():
    ds, b = [4096, 1001, 30000, 520, 8192, 64], 72
    at, ar = [], []
    for m, d in enumerate(ds):
        t, r = wl.make_pair(b, d, "relu", 0.05 + 0.05 * m, seed=600 + m, device=DEV)
        at.append(t)
        ar.append(r)
    ref = oracle.sp_loss_batch([wl.bf16_bits(t) for t in at], [wl.bf16_bits(r) for r in ar])
    ctx = eg.Context(ds, b, 3, 1e-3, device=DEV)
    for active in ([1, 0, 0, 0, 0, 0], [0, 1, 0, 0, 0, 0], [0, 0, 1, 0, 1, 0], [1, 1, 1, 1, 1, 1], [0, 0, 0, 1, 0, 1]):
        out = torch.full((len(ds),), -7.0, dtype=torch.float32, device=DEV)
        left_out = [None if not a else t for t, a in zip(at, active)]       # pointers of the others are not read
        ctx.egeria_sp_loss_subset(left_out, [None if not a else r for r, a in zip(ar, active)], active, out)
        got = out.cpu().numpy()
        act = np.array(active, dtype=bool)
        assert_loss_close(got[act], ref[act], f"subset {active}")
        assert np.all(got[~act] == -7.0)
    ctx.check_device_status()
    with pytest.raises(eg.EgeriaError) as e:
        ctx.egeria_sp_loss_subset(at, ar, [0] * len(ds), out)
    assert e.value.status == eg.ERR_INVALID_ARG
    # the rule advances for the active modules only
    losses = torch.zeros(len(ds), dtype=torch.float32, device=DEV)
    slopes = torch.full((len(ds),), -1.0, dtype=torch.float64, device=DEV)
    mask = torch.full((len(ds),), 9, dtype=torch.uint8, device=DEV)
    for _ in range(2):
        ctx.egeria_plasticity_evaluate_subset(at, ar, [0, 0, 1, 0, 0, 0], losses, slopes, mask)
    s, mk = slopes.cpu().numpy(), mask.cpu().numpy()
    assert s[2] == 0.0 and mk[2] == 0                       # two equal readings: slope 0, not frozen yet (W = 3)
    assert np.all(s[[0, 1, 3, 4, 5]] == -1.0) and np.all(mk[[0, 1, 3, 4, 5]] == 9)
    ctx.close()


def test_frontmost_policy_evaluating_only_the_front_module():
    """The intended use of the frontmost policy: read the mask back, evaluate only the first module
    that is not frozen.  Same decisions as evaluating everything."""
    ds, b, W = [4096, 2048, 1001, 8192, 520], 40, 2
    flags = eg.FLAG_FRONTMOST
    full = eg.Context(ds, b, W, 0.5, flags, device=DEV)
    front_only = eg.Context(ds, b, W, 0.5, flags, device=DEV)
    M = len(ds)
    losses = torch.zeros(M, dtype=torch.float32, device=DEV)
    slopes = torch.zeros(M, dtype=torch.float64, device=DEV)
    mask = torch.zeros(M, dtype=torch.uint8, device=DEV)
    front, seen = 0, []
    for k in range(16):
        at, ar = [], []
        for m, d in enumerate(ds):
            t, r = wl.make_pair(b, d, "relu", 0.3, seed=800 + 10 * k + m, device=DEV)
            at.append(t)
            ar.append(r)
        l1, s1, m1 = full.egeria_plasticity_evaluate(at, ar)
        if front < M:
            active = [1 if m == front else 0 for m in range(M)]
            front_only.egeria_plasticity_evaluate_subset(at, ar, active, losses, slopes, mask)
            assert_loss_close(losses.cpu().numpy()[front:front + 1], l1.cpu().numpy().astype(np.float64)[front:front + 1])
        assert mask.cpu().numpy().tolist() == m1.cpu().numpy().tolist()
        front = int(mask.cpu().numpy().sum())
        seen.append(front)
    assert seen[-1] == M and seen[0] == 0
    full.close()
    front_only.close()


# ----------------------------------------------------------------------------- unfreezing on learning-rate annealing

def _unfreeze_case(seed, M, H, period):
    """Histories that decay within each learning-rate period, and a step decay by 10x per period."""
    rng = np.random.default_rng(seed)
    k = np.arange(H)
    hist = np.stack([0.3 * np.exp(-(k % period) / rng.uniform(2, 8)) + 0.01 * (m + 1) + 1e-4 * rng.standard_normal(H)
                     for m in range(M)]).astype(np.float32)
    T = rng.uniform(3e-3, 2e-2, size=M).astype(np.float32)
    lr = 0.1 * np.power(0.1, k // period).astype(np.float64)
    return hist, T, lr


def _clear_of_T(ref, T, auto=False):
    """No finite oracle slope within 1e-6 of its tolerance: every decision may be compared."""
    if auto:
        return True        # checked by the caller through the masks' agreement with the slopes
    for m in range(ref["slopes"].shape[0]):
        s = ref["slopes"][m]
        s = s[np.isfinite(s)]
        if np.any(np.abs(np.abs(s) - float(T[m])) <= 1e-6):
            return False
    return True


@pytest.mark.parametrize("frontmost", [False, True])
@pytest.mark.parametrize("auto", [False, True])
def test_unfreeze_one_evaluation_at_a_time_matches_oracle(frontmost, auto):
    """egeria_plasticity_set_lr + egeria_plasticity_step across two tenfold drops of the learning
    rate: slopes, masks, the window in force and the restarts against oracle.unfreeze_replay."""
    M, H, W, period = 4, 165, 6, 55
    hist, T, lr = _unfreeze_case(21 + auto, M, H, period)
    ref = oracle.unfreeze_replay(hist, lr, W, None if auto else T.astype(np.float64), frontmost=frontmost)
    assert ref["restarts"] == 2 and _clear_of_T(ref, T, auto)
    flags = (eg.FLAG_FRONTMOST if frontmost else 0) | (eg.FLAG_AUTO_T if auto else 0)
    ctx = eg.Context([64] * M, 8, W, T, flags, device=DEV)
    dev = torch.from_numpy(hist).to(DEV)
    for i in range(H):
        ctx.egeria_plasticity_set_lr(float(lr[i]))
        s, mk = ctx.egeria_plasticity_step(dev[:, i].contiguous())
        s, mk = s.cpu().numpy(), mk.cpu().numpy()
        assert mk.tolist() == ref["frozen"][i].tolist(), f"evaluation {i}"
        adv = ~np.isnan(ref["slopes"][:, i])
        fin = adv & np.isfinite(ref["slopes"][:, i])
        np.testing.assert_allclose(s[fin], ref["slopes"][fin, i], rtol=1e-9, atol=1e-15)
        assert np.all(np.isinf(s[adv & ~fin]))
        if i in (0, period - 1, period, period + 1, 2 * period + 3):
            assert ctx.egeria_plasticity_window() == ref["window"][i + 1]   # what the NEXT evaluation will use
    assert ctx.egeria_plasticity_restarts() == ref["restarts"]
    ctx.close()


@pytest.mark.parametrize("M,H,W,period,frontmost", [(4, 165, 6, 55, False), (4, 165, 6, 55, True),
                                                    (24, 1000, 50, 334, False), (24, 1000, 50, 334, True),
                                                    (70, 300, 9, 100, False)])
def test_unfreeze_whole_histories_match_oracle(M, H, W, period, frontmost):
    """egeria_plasticity_replay_lr: one launch over the whole history, against oracle.unfreeze_replay."""
    hist, T, lr = _unfreeze_case(100 + M + W, M, H, period)
    if W >= 50:                                                   # long windows: slower decays, so that modules still freeze
        k = np.arange(H)
        rng = np.random.default_rng(7)
        hist = np.stack([0.3 * np.exp(-(k % period) / rng.uniform(5, 30)) + 0.01 * (m + 1)
                         + 1e-5 * rng.standard_normal(H) for m in range(M)]).astype(np.float32)
    ref = oracle.unfreeze_replay(hist, lr, W, T.astype(np.float64), frontmost=frontmost)
    assert ref["restarts"] >= 1 and ref["frozen"].any()
    ctx = eg.Context([64] * M, 8, W, T, eg.FLAG_FRONTMOST if frontmost else 0, device=DEV)
    out = ctx.egeria_plasticity_replay_lr(torch.from_numpy(hist).to(DEV), torch.from_numpy(lr).to(DEV))
    slopes, frozen, window, restarted, mask, fe = [t.cpu().numpy() for t in out]
    assert window.tolist() == ref["window"].tolist()
    assert restarted.tolist() == ref["restarted"].tolist()
    assert np.array_equal(np.isnan(slopes), np.isnan(ref["slopes"]))
    fin = np.isfinite(ref["slopes"])
    np.testing.assert_allclose(slopes[fin], ref["slopes"][fin], rtol=1e-9, atol=1e-15)
    # decisions: compared wherever no slope of the module's current run came within 1e-6 of T
    near = np.zeros((H, M), dtype=bool)
    for m in range(M):
        close = np.isfinite(ref["slopes"][m]) & (np.abs(np.abs(ref["slopes"][m]) - float(T[m])) <= 1e-6)
        run_start = 0
        for i in range(H):
            near[i, m] = close[run_start:i + 1].any()
            if ref["restarted"][i]:
                run_start = i + 1
    if frontmost:
        near = np.repeat(near.any(axis=1)[:, None], M, axis=1)
    assert (~near).mean() > 0.8
    assert np.array_equal(frozen[~near], ref["frozen"][~near])
    assert mask.tolist() == frozen[-1].tolist()
    # without a learning rate the call is the plain replay
    s2, fz2, w2, r2, mk2, fe2 = [t.cpu().numpy() for t in
                                 ctx.egeria_plasticity_replay_lr(torch.from_numpy(hist).to(DEV), None)]
    s1, mk1, fe1 = [t.cpu().numpy() for t in ctx.egeria_plasticity_replay(torch.from_numpy(hist).to(DEV))]
    assert not r2.any() and np.all(w2 == W)
    assert np.array_equal(np.isnan(s1), np.isnan(s2)) and np.array_equal(s1[~np.isnan(s1)], s2[~np.isnan(s2)])
    assert mk1.tolist() == mk2.tolist() and fe1.tolist() == fe2.tolist()
    ctx.close()


def test_unfreeze_hand_traces_on_gpu():
    for line in (GOLDEN / "unfreeze_traces.txt").read_text().splitlines():
        if not line.strip() or line.startswith("#"):
            continue
        f = [x.strip() for x in line.split("|")]
        frontmost, W = bool(int(f[1])), int(f[2])
        T = np.array([float(v) for v in f[3].split()], dtype=np.float32)
        hist = np.array([[float(v) for v in row.split()] for row in f[4].split(";")], dtype=np.float32)
        lr = np.array([float(v) for v in f[5].split()])
        M, H = hist.shape
        ctx = eg.Context([64] * M, 8, W, T, eg.FLAG_FRONTMOST if frontmost else 0, device=DEV)
        out = ctx.egeria_plasticity_replay_lr(torch.from_numpy(hist).to(DEV), torch.from_numpy(lr).to(DEV))
        slopes, frozen, window, restarted = [t.cpu().numpy() for t in out[:4]]
        assert window.tolist() == [int(v) for v in f[6].split()]
        assert ["".join(str(int(v)) for v in row) for row in frozen] == f[7].split()
        assert np.nonzero(restarted)[0].tolist() == [int(v) for v in f[8].split()]
        # and one evaluation at a time
        dev = torch.from_numpy(hist).to(DEV)
        for i in range(H):
            ctx.egeria_plasticity_set_lr(float(lr[i]))
            _, mk = ctx.egeria_plasticity_step(dev[:, i].contiguous())
            assert "".join(str(int(v)) for v in mk.cpu().numpy()) == f[7].split()[i], (f[0], i)
        assert ctx.egeria_plasticity_restarts() == len(f[8].split())
        ctx.close()


def test_unfreeze_inside_the_fused_evaluation():
    """egeria_plasticity_evaluate under a learning rate that drops tenfold: same losses, slopes and
    masks as egeria_sp_loss_batch + egeria_plasticity_step on a second context, one restart, the
    window halved, and the state survives export / import."""
    ds, b, W = [4096, 2048, 1001], 40, 4
    flags = eg.FLAG_EQUAL_SPLIT
    fused = eg.Context(ds, b, W, 0.5, flags, device=DEV)       # a generous T: modules freeze at evaluation W
    split = eg.Context(ds, b, W, 0.5, flags, device=DEV)
    masks = []
    for k in range(14):
        rate = 0.1 if k < 7 else 0.01
        at, ar = [], []
        for m, d in enumerate(ds):
            t, r = wl.make_pair(b, d, "relu", 0.3, seed=900 + 10 * k + m, device=DEV)
            at.append(t)
            ar.append(r)
        for c in (fused, split):
            c.egeria_plasticity_set_lr(rate)
        l1, s1, m1 = fused.egeria_plasticity_evaluate(at, ar)
        l2 = split.egeria_sp_loss_batch(at, ar)
        s2, m2 = split.egeria_plasticity_step(l2)
        assert l1.cpu().numpy().tobytes() == l2.cpu().numpy().tobytes()
        assert s1.cpu().numpy().tobytes() == s2.cpu().numpy().tobytes()
        assert m1.cpu().numpy().tobytes() == m2.cpu().numpy().tobytes()
        masks.append(m1.cpu().numpy().tolist())
        if k == 9:                                              # carry on from a checkpoint
            saved = fused.egeria_plasticity_export()
            fused.close()
            fused = eg.Context(ds, b, W, 0.5, flags, device=DEV)
            fused.egeria_plasticity_import(saved)
    # frozen at evaluation W = 4; restart at 7 (the first evaluation under 0.01); W = 2: frozen again at 10
    assert masks[3] == [0, 0, 0] and masks[4] == [1, 1, 1] and masks[6] == [1, 1, 1]
    assert masks[7] == [0, 0, 0] and masks[9] == [0, 0, 0] and masks[10] == [1, 1, 1]
    assert fused.egeria_plasticity_restarts() == 1 and fused.egeria_plasticity_window() == 2
    fused.close()
    split.close()


def test_front_only_evaluation_follows_the_front_on_the_device():
    """EGERIA_FLAG_FRONT_ONLY: every evaluation computes the monitored module only, chosen on the
    device.  Decisions against oracle.frontmost_replay on the oracle's own losses of the same
    activations; the loss written is the front module's and nothing else is touched; after a
    restart by the unfreezing rule the front is module 0 again."""
    ds, b, W, K = [4096, 2048, 8192, 1024, 4160], 40, 2, 18
    M = len(ds)
    T = 0.5                                                    # generous: a module freezes W evaluations after its start
    fo = eg.Context(ds, b, W, T, eg.FLAG_FRONTMOST | eg.FLAG_FRONT_ONLY, device=DEV)
    full = eg.Context(ds, b, W, T, eg.FLAG_FRONTMOST, device=DEV)
    losses = torch.full((M,), -9.0, dtype=torch.float32, device=DEV)
    slopes = torch.zeros(M, dtype=torch.float64, device=DEV)
    mask = torch.zeros(M, dtype=torch.uint8, device=DEV)
    sp = int(torch.cuda.current_stream().cuda_stream)
    hist = np.zeros((M, K), dtype=np.float32)
    got_masks, fronts = [], []
    front = 0
    for c in (fo, full):
        c.egeria_plasticity_set_lr(0.1)
    for k in range(K):
        at, ar = [], []
        for m, d in enumerate(ds):
            t, r = wl.make_pair(b, d, "relu", 0.3, seed=1200 + 10 * k + m, device=DEV)
            at.append(t)
            ar.append(r)
            hist[m, k] = oracle.sp_loss(wl.bf16_bits(t), wl.bf16_bits(r))
        losses.fill_(-9.0)
        launches = fo.egeria_launch_count()
        fo.plasticity_evaluate_raw(fo._ptr_array(at, b, True), fo._ptr_array(ar, b, True), b, losses.data_ptr(),
                                   slopes.data_ptr(), mask.data_ptr(), sp)
        l1, s1, m1 = full.egeria_plasticity_evaluate(at, ar)
        got = losses.cpu().numpy()
        assert fo.egeria_launch_count() == launches + 1            # one kernel, whatever the front
        if front < M:
            assert_loss_close(got[front:front + 1], hist[front:front + 1, k].astype(np.float64), f"evaluation {k}")
            assert np.all(np.delete(got, front) == -9.0)           # only the monitored module was computed
        else:
            assert np.all(got == -9.0)
        assert mask.cpu().numpy().tolist() == m1.cpu().numpy().tolist()
        got_masks.append(mask.cpu().numpy().tolist())
        fronts.append(front)
        front = int(mask.cpu().numpy().sum())
    ref = oracle.frontmost_replay(hist, W, np.full(M, T))
    assert ref["frozen"] == M                                      # all frozen within the history ...
    assert fronts == ref["monitored"].tolist()
    for k in range(K):
        want = [int(0 <= ref["freeze_eval"][m] <= k) for m in range(M)]
        assert got_masks[k] == want, f"evaluation {k}"
    assert got_masks[-1] == [1] * M                                # ... and an evaluation then only reports
    fo.check_device_status()
    # the learning rate falls tenfold: everything restarts, the device goes back to module 0
    fo.egeria_plasticity_set_lr(0.01)
    for k in range(3):
        losses.fill_(-9.0)
        fo.plasticity_evaluate_raw(fo._ptr_array(at, b, True), fo._ptr_array(ar, b, True), b, losses.data_ptr(),
                                   slopes.data_ptr(), mask.data_ptr(), sp)
        got = losses.cpu().numpy()
        if k == 0:
            assert np.all(got == -9.0) and mask.cpu().numpy().tolist() == [0] * M    # the restart itself
        else:
            assert got[0] > 0 and np.all(got[1:] == -9.0)
    assert fo.egeria_plasticity_restarts() == 1
    fo.check_device_status()
    fo.close()
    full.close()
    # a module that cannot take the tensor-core kernel is refused, as is the subset form
    bad = eg.Context([4096, 1001], b, W, T, eg.FLAG_FRONTMOST | eg.FLAG_FRONT_ONLY, device=DEV)
    pair = [wl.make_pair(b, d, "relu", 0.3, seed=5, device=DEV) for d in (4096, 1001)]
    with pytest.raises(eg.EgeriaError) as e:
        bad.egeria_plasticity_evaluate([p[0] for p in pair], [p[1] for p in pair])
    assert e.value.status == eg.ERR_UNSUPPORTED_SHAPE
    bad.close()
    with pytest.raises(eg.EgeriaError) as e:
        eg.Context([4096], b, W, T, eg.FLAG_FRONT_ONLY, device=DEV)       # needs the frontmost policy
    assert e.value.status == eg.ERR_INVALID_ARG


def test_bootstrap_detector_matches_oracle():
    rng = np.random.default_rng(11)
    H, W = 120, 8
    loss = (2.5 * np.exp(-np.arange(H) / 15.0) + 0.4 + 0.01 * rng.standard_normal(H)).astype(np.float32)
    ctx = eg.Context([64], 8, W, 1e-3, device=DEV)
    for tol in (0.1, 0.02):
        ref = oracle.bootstrap_replay(loss, W, tol)
        assert 2 * W < ref["end"] < H - 5
        rates, end = ctx.egeria_bootstrap_replay(torch.from_numpy(loss).to(DEV), tol)
        rates = rates.cpu().numpy()
        near = np.nanmin(np.abs(ref["rates"] - tol)) < 1e-9
        if not near:
            assert int(end.cpu()[0]) == ref["end"]
        live = ~np.isnan(ref["rates"])
        assert np.array_equal(np.isnan(rates), ~live)
        np.testing.assert_allclose(rates[live], ref["rates"][live], rtol=1e-9)
        # one reading at a time
        ctx.egeria_bootstrap_reset()
        dev = torch.from_numpy(loss).to(DEV)
        ended = -1
        for i in range(H):
            rate, done = ctx.egeria_bootstrap_step(dev[i:i + 1], tol)
            if live[i]:
                assert float(rate.cpu()[0]) == pytest.approx(ref["rates"][i], rel=1e-9)
            if ended < 0 and int(done.cpu()[0]):
                ended = i
        if not near:
            assert ended == ref["end"]
    ctx.close()


def test_state_export_import_resumes_the_same_decisions():
    M, H, W = 4, 60, 5
    hist = _policy_histories(M, H, seed=5)
    dev = torch.from_numpy(hist).to(DEV)
    flags = eg.FLAG_AUTO_T
    a = eg.Context([64] * M, 8, W, 1e-3, flags, device=DEV)
    full = []
    for i in range(H):
        s, mk = a.egeria_plasticity_step(dev[:, i].contiguous())
        full.append((s.cpu().numpy().copy(), mk.cpu().numpy().copy()))
        if i == 22:
            a.egeria_bootstrap_step(dev[0, i:i + 1])
            saved = a.egeria_plasticity_export()
    assert saved.nbytes == a.egeria_plasticity_state_bytes()
    b2 = eg.Context([64] * M, 8, W, 1e-3, flags, device=DEV)
    b2.egeria_plasticity_import(saved)
    for i in range(23, H):
        s, mk = b2.egeria_plasticity_step(dev[:, i].contiguous())
        assert s.cpu().numpy().tobytes() == full[i][0].tobytes()
        assert mk.cpu().numpy().tobytes() == full[i][1].tobytes()
    # a context with another window, module count or rule refuses the buffer
    for other in (eg.Context([64] * M, 8, W + 1, 1e-3, flags, device=DEV),
                  eg.Context([64] * (M + 1), 8, W, 1e-3, flags, device=DEV),
                  eg.Context([64] * M, 8, W, 1e-3, 0, device=DEV)):
        with pytest.raises(eg.EgeriaError) as e:
            other.egeria_plasticity_import(saved)
        assert e.value.status == eg.ERR_INVALID_ARG
        other.close()
    with pytest.raises(eg.EgeriaError) as e:
        b2.egeria_plasticity_import(saved[:-8])
    assert e.value.status == eg.ERR_WORKSPACE
    a.close()
    b2.close()


def test_alg1_hand_traces_on_gpu():
    from fractions import Fraction
    for line in (GOLDEN / "alg1_traces.txt").read_text().splitlines():
        if not line.strip() or line.startswith("#"):
            continue
        f = [s.strip() for s in line.split("|")]
        W, T, signed = int(f[1]), float(f[2]), bool(int(f[3]))
        hist = np.array([[float(v) for v in f[4].split()]], dtype=np.float32)
        ctx = eg.Context([64], 8, W, T, eg.FLAG_SIGNED_SLOPE if signed else 0, device=DEV)
        slopes, mask, fe = ctx.egeria_plasticity_replay(torch.from_numpy(hist).to(DEV))
        assert int(fe[0]) == int(f[8]), f[0]
        assert bool(mask[0]) == (int(f[8]) >= 0)
        for i, tok in enumerate(f[6].split()):
            got = float(slopes[0, i])
            if tok == "x":
                assert np.isnan(got)
            elif tok == "inf":
                assert np.isinf(got)
            else:
                assert got == pytest.approx(float(Fraction(tok)), rel=1e-6, abs=1e-7)
        ctx.close()


def test_tiny_end_to_end_chain():
    """20 real evaluations of the tiny workload: GPU losses -> GPU slopes/mask against
    oracle losses -> oracle slopes/mask."""
    w = wl.WORKLOADS["tiny"]
    T32 = float(np.float32(w.T))
    ctx = eg.Context(list(w.d), w.b, w.W, T32, device=DEV)
    gpu_losses, ref_losses, masks = [], [], []
    for k, sigma in enumerate(wl.tiny_history_sigmas(w)):
        at, ar = wl.make_module(w, 0, DEV, sigma=sigma, seed_offset=k)
        out = ctx.egeria_sp_loss_batch([at], [ar])
        s, mk = ctx.egeria_plasticity_step(out)
        gpu_losses.append(float(out.cpu()[0]))
        masks.append(int(mk.cpu()[0]))
        ref_losses.append(oracle.sp_loss(wl.bf16_bits(at), wl.bf16_bits(ar)))
    assert_loss_close(gpu_losses, ref_losses, "tiny history")
    ref = oracle.plasticity_replay(np.array(ref_losses, dtype=np.float32), w.W, T32)
    sl = ref["slopes"][np.isfinite(ref["slopes"])]
    if not np.any(np.abs(np.abs(sl) - T32) <= 1e-6):
        assert bool(masks[-1]) == ref["converged"]
    ctx.check_device_status()
    ctx.close()


def test_an_evaluation_is_turned_away_from_a_capturing_stream():
    """An evaluation carries per-call state (which set of counters and partial slots, the rule's
    serial number); replayed from a graph it would be wrong without a sign.  On a capturing
    stream the call returns EGERIA_ERR_INVALID_ARG, records nothing, and the context goes on."""
    at, ar = wl.make_pair(48, 4096, "relu", 0.2, seed=77, device=DEV)
    ctx = eg.Context([4096], 48, 5, 1e-3, eg.FLAG_EQUAL_SPLIT, device=DEV)
    good = ctx.egeria_sp_loss_batch([at], [ar]).cpu().numpy().copy()
    out = torch.full((1,), -3.0, dtype=torch.float32, device=DEV)
    x = torch.zeros(4, device=DEV)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        g.capture_begin()
        try:
            x.add_(1.0)
            with pytest.raises(eg.EgeriaError) as e:
                ctx.egeria_sp_loss_batch([at], [ar], out, stream=side)
        finally:
            g.capture_end()
    assert e.value.status == eg.ERR_INVALID_ARG
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    g.replay()
    torch.cuda.synchronize()
    assert float(out.cpu()[0]) == -3.0 and float(x.cpu()[0]) == 1.0    # the graph holds the add and nothing of ours
    again = ctx.egeria_sp_loss_batch([at], [ar]).cpu().numpy()
    assert again.tobytes() == good.tobytes()
    ctx.check_device_status()
    ctx.close()


def test_checked_build_finds_nothing_on_the_parity_cases():
    """The second library the build makes (index checks inside the kernels: unit table, slot
    ranges, first tasks, cursors, offsets into slots, stages, chunk scratch and tensor memory) runs
    a cross-section of this file -- every kernel mode, both ways of finishing, two levels, front-only,
    CUDA-core modules, the bounded waits -- in a process of its own: same results, and no check fires
    (every test there ends with a status query, which would say EGERIA_ERR_CHECK)."""
    import subprocess
    import sys
    assert eg.lib().egeria_build_is_checked() in (0, 1)
    sel = ("single_module_tensor_core_path or cut_over_every_cta or many_modules or hundreds or two_ways or "
           "bounded_wait or front_only or overlapped or resnet56_workload_full or bert_base_workload_full or "
           "tiny_workload_full or nan_of_any or unfreez")
    r = subprocess.run([sys.executable, "-m", "pytest", str(Path(__file__)), "-m", "gpu", "-x", "-q", "--checked-library",
                        "-k", sel, "-p", "no:cacheprovider"], capture_output=True, text=True, cwd=str(Path(__file__).parent.parent))
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-2000:]
    assert " passed" in r.stdout and "failed" not in r.stdout
