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
    has settled; the oracle checks the whole loss of a few modules and sampled rows of the
    normalised Grams of others."""
    w = wl.WORKLOADS[name]
    at, ar = wl.make_activations(w, DEV)
    full_ref = {m: oracle.sp_loss(wl.bf16_bits(at[m]), wl.bf16_bits(ar[m]), return_grams=True) for m in full_modules}
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
        assert np.isfinite(losses).all() and np.all(losses >= 0) and np.all(losses <= 4.0 / w.b)
        for m, (ref, gt, gr) in full_ref.items():
            np.testing.assert_allclose(grams[m][0], gt, rtol=0, atol=ENTRY_ATOL)
            np.testing.assert_allclose(grams[m][1], gr, rtol=0, atol=ENTRY_ATOL)
            assert_loss_close(losses[m:m + 1], [ref], f"{name} module {m} ({what})")
        for (m, side, i), gn in row_ref.items():
            np.testing.assert_allclose(grams[m][side][i], gn, rtol=0, atol=ENTRY_ATOL)
        # properties that hold at any size: unit rows, symmetric-positive diagonal
        for m in range(w.M):
            for side in (0, 1):
                np.testing.assert_allclose(np.linalg.norm(grams[m][side].astype(np.float64), axis=1), 1.0, atol=1e-5)
                assert np.all(np.diag(grams[m][side]) > 0)
        return losses

    first = check("equal split")
    for _ in range(12):
        ctx.egeria_plasticity_evaluate(at, ar)[0].cpu()       # .cpu() waits: the launch logs land
    assert ctx.egeria_split_weights()[0] > 0                  # the shares now follow the measured rates
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

def masks_agree(gpu_mask, gpu_fe, hist, W, T, signed=False):
    for m in range(hist.shape[0]):
        ref = oracle.plasticity_replay(hist[m], W, T, signed_test=signed)
        s = ref["slopes"][np.isfinite(ref["slopes"])]
        near = np.any(np.abs((s if signed else np.abs(s)) - T) <= 1e-6) if len(s) else False
        if near:
            continue
        assert bool(gpu_mask[m]) == ref["converged"], f"module {m}"
        assert int(gpu_fe[m]) == ref["freeze_eval"], f"module {m}"


@pytest.mark.parametrize("name,level", [("resnet56", None), ("resnet56", 1e-2), ("resnet50", 2e-2),
                                        ("bert_base", 5e-3), ("gpt2_medium", 3e-2)])
def test_replay_matches_oracle(name, level):
    w = wl.WORKLOADS[name]
    levels = [1e-6 * (1 + l) for l in range(w.M)] if level is None else [level * (1 + 0.1 * l) for l in range(w.M)]
    hist = wl.make_history(w, levels)
    T32 = np.float32(w.T)
    ctx = eg.Context([64] * w.M, 8, w.W, float(T32), device=DEV)
    slopes, mask, fe = ctx.egeria_plasticity_replay(torch.from_numpy(hist).to(DEV))
    slopes, mask, fe = slopes.cpu().numpy(), mask.cpu().numpy(), fe.cpu().numpy()
    n_conv = 0
    for m in range(w.M):
        ref = oracle.plasticity_replay(hist[m], w.W, float(T32))
        live = ~np.isnan(ref["slopes"])
        assert np.array_equal(np.isnan(slopes[m]), ~live) or not ref["converged"]
        np.testing.assert_allclose(slopes[m][live], ref["slopes"][live], rtol=1e-9, atol=1e-15)
        n_conv += ref["converged"]
    masks_agree(mask, fe, hist, w.W, float(T32))
    if level is not None and name != "bert_base":
        assert 0 < n_conv < w.M, "the synthetic history should give a non-trivial mask"
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
    # reset clears the state; halving the window follows the unfreezing rule
    ctx.egeria_plasticity_reset(halve_W=True)
    assert ctx.egeria_plasticity_window() == 2
    s, mk = ctx.egeria_plasticity_step(hist_dev[:, 0].contiguous())
    assert np.all(np.isinf(s.cpu().numpy())) and not mk.cpu().numpy().any()
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
    for k in range(14):
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
