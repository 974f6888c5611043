"""ctypes binding of ``libegeria.so`` -- argument marshalling only.

Every function here has the name of the C entry point it calls (``include/egeria.h``).
PyTorch appears only as the owner of device memory and streams; every step of the
plasticity evaluation runs inside the library's CUDA kernels.  There is no fallback:
if the library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
from pathlib import Path
from typing import Optional, Sequence

import numpy as np
import torch

_LIB_PATH = Path(__file__).resolve().parent / "libegeria.so"

_LIB_PATH_CHECKED = Path(__file__).resolve().parent / "libegeria_checked.so"

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED_SHAPE, ERR_UNSUPPORTED_DEVICE, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT, ERR_CHECK = range(8)
FLAG_SIGNED_SLOPE, FLAG_FORCE_SIMT, FLAG_KEEP_GRAMS, FLAG_HOST_STAGING, FLAG_TIME_GRAM = 1, 2, 4, 8, 16
FLAG_EQUAL_SPLIT, FLAG_AUTO_T, FLAG_FRONTMOST, FLAG_FRONT_ONLY, FLAG_OVERLAP = 32, 64, 128, 256, 512
MAX_B = 256
WORKSPACE_ALIGN = 1024

EXPORTS = [
    "egeria_workspace_bytes", "egeria_plasticity_create", "egeria_plasticity_destroy",
    "egeria_sp_loss_batch", "egeria_sp_loss_batch_host", "egeria_plasticity_step",
    "egeria_plasticity_replay", "egeria_plasticity_reset", "egeria_plasticity_window",
    "egeria_debug_dump_gram", "egeria_debug_plan", "egeria_debug_plan_weighted", "egeria_device_status",
    "egeria_launch_count",
    "egeria_gram_kernel_time", "egeria_sp_loss_static", "egeria_plasticity_evaluate",
    "egeria_split_weights", "egeria_status_string", "egeria_bootstrap_step", "egeria_bootstrap_replay",
    "egeria_bootstrap_reset", "egeria_plasticity_state_bytes", "egeria_plasticity_export", "egeria_plasticity_import",
    "egeria_sp_loss_subset", "egeria_plasticity_evaluate_subset",
    "egeria_sp_loss_static_status", "egeria_debug_stall_next", "egeria_debug_plan_help", "egeria_debug_plan_tasks", "egeria_build_is_checked", "egeria_debug_check_record", "egeria_plasticity_set_lr", "egeria_plasticity_restarts", "egeria_plasticity_replay_lr",
]


class EgeriaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = int(status)
        super().__init__(f"{where}: {status_string(status)} (status {int(status)})")


_lib = None


def use_checked_library(checked: bool = True) -> None:
    """Switch this process to the checked build of the library (index checks inside the kernels,
    see egeria_build_is_checked) or back.  Only with no Context open: a handle belongs to the
    library that made it."""
    global _lib, _LIB_PATH
    _LIB_PATH = _LIB_PATH_CHECKED if checked else Path(__file__).resolve().parent / "libegeria.so"
    _lib = None


def lib() -> ctypes.CDLL:
    """Load the CUDA library.  Raises if it has not been built -- there is no other path."""
    global _lib
    if _lib is not None:
        return _lib
    if not _LIB_PATH.exists():
        raise ImportError(f"{_LIB_PATH} is missing: build it with `python -m paper_2201_06227_b200.build`")
    L = ctypes.CDLL(str(_LIB_PATH))
    vp, i64p = ctypes.c_void_p, ctypes.POINTER(ctypes.c_int64)
    L.egeria_workspace_bytes.argtypes = [ctypes.c_int, i64p, ctypes.c_int, ctypes.c_int, ctypes.c_uint32]
    L.egeria_workspace_bytes.restype = ctypes.c_size_t
    L.egeria_plasticity_create.argtypes = [ctypes.POINTER(vp), ctypes.c_int, i64p, ctypes.c_int, ctypes.c_int,
                                           ctypes.POINTER(ctypes.c_float), ctypes.c_float, vp, ctypes.c_size_t,
                                           ctypes.c_uint32]
    L.egeria_plasticity_destroy.argtypes = [vp]
    L.egeria_sp_loss_batch.argtypes = [vp, vp, ctypes.POINTER(vp), ctypes.POINTER(vp), ctypes.c_int, i64p, vp]
    L.egeria_sp_loss_batch_host.argtypes = [vp, vp, ctypes.POINTER(vp), ctypes.POINTER(vp), ctypes.c_int, i64p, vp]
    L.egeria_plasticity_step.argtypes = [vp, vp, vp, vp, vp]
    L.egeria_plasticity_evaluate.argtypes = [vp, vp, ctypes.POINTER(vp), ctypes.POINTER(vp), ctypes.c_int, i64p,
                                             vp, vp, vp]
    L.egeria_sp_loss_subset.argtypes = [vp, vp, ctypes.POINTER(vp), ctypes.POINTER(vp), ctypes.c_int, i64p,
                                        ctypes.POINTER(ctypes.c_uint8), vp]
    L.egeria_plasticity_evaluate_subset.argtypes = [vp, vp, ctypes.POINTER(vp), ctypes.POINTER(vp), ctypes.c_int, i64p,
                                                    ctypes.POINTER(ctypes.c_uint8), vp, vp, vp]
    L.egeria_plasticity_replay.argtypes = [vp, vp, vp, ctypes.c_int, vp, vp, vp]
    L.egeria_plasticity_reset.argtypes = [vp, vp, ctypes.c_int]
    L.egeria_plasticity_window.argtypes = [vp]
    L.egeria_plasticity_restarts.argtypes = [vp]
    L.egeria_plasticity_set_lr.argtypes = [vp, ctypes.c_double]
    L.egeria_plasticity_replay_lr.argtypes = [vp, vp, vp, vp, ctypes.c_int, vp, vp, vp, vp, vp, vp]
    L.egeria_debug_dump_gram.argtypes = [vp, vp, ctypes.c_int, vp, vp]
    L.egeria_debug_plan.argtypes = [ctypes.c_int, i64p, ctypes.c_int, ctypes.c_int,
                                    ctypes.POINTER(ctypes.c_int32), ctypes.c_int, ctypes.POINTER(ctypes.c_int)]
    L.egeria_debug_plan_weighted.argtypes = [ctypes.c_int, i64p, ctypes.c_int, ctypes.c_int,
                                             ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_int32),
                                             ctypes.c_int, ctypes.POINTER(ctypes.c_int)]
    L.egeria_split_weights.argtypes = [vp, ctypes.POINTER(ctypes.c_float), ctypes.c_int]
    L.egeria_bootstrap_step.argtypes = [vp, vp, vp, ctypes.c_float, vp, vp]
    L.egeria_bootstrap_replay.argtypes = [vp, vp, vp, ctypes.c_int, ctypes.c_float, vp, vp]
    L.egeria_bootstrap_reset.argtypes = [vp, vp]
    L.egeria_plasticity_state_bytes.argtypes = [vp]
    L.egeria_plasticity_state_bytes.restype = ctypes.c_size_t
    L.egeria_plasticity_export.argtypes = [vp, vp, vp, ctypes.c_size_t]
    L.egeria_plasticity_import.argtypes = [vp, vp, vp, ctypes.c_size_t]
    L.egeria_device_status.argtypes = [vp]
    L.egeria_gram_kernel_time.argtypes = [vp, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_int64)]
    L.egeria_sp_loss_static.argtypes = [vp, vp, vp, ctypes.c_int, ctypes.c_int64, vp]
    L.egeria_sp_loss_static_status.argtypes = []
    L.egeria_debug_stall_next.argtypes = [vp, ctypes.c_int]
    L.egeria_debug_plan_help.argtypes = [ctypes.c_int, i64p, ctypes.c_int, ctypes.c_int, ctypes.POINTER(ctypes.c_int32)]
    L.egeria_debug_plan_tasks.argtypes = [ctypes.c_int, i64p, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                          ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_int32),
                                          ctypes.POINTER(ctypes.c_int)]
    L.egeria_build_is_checked.argtypes = []
    L.egeria_debug_check_record.argtypes = [vp, ctypes.POINTER(ctypes.c_int32)]
    L.egeria_launch_count.argtypes = [vp]
    L.egeria_launch_count.restype = ctypes.c_int64
    L.egeria_status_string.argtypes = [ctypes.c_int]
    L.egeria_status_string.restype = ctypes.c_char_p
    _lib = L
    return L


def status_string(status: int) -> str:
    return lib().egeria_status_string(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != OK:
        raise EgeriaError(status, where)


def _i64(seq: Sequence[int]):
    arr = (ctypes.c_int64 * len(seq))(*[int(v) for v in seq])
    return arr


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


def egeria_workspace_bytes(M: int, d: Sequence[int], b_max: int, W: int, flags: int = 0) -> int:
    return int(lib().egeria_workspace_bytes(int(M), _i64(d), int(b_max), int(W), int(flags)))


def egeria_debug_plan(d: Sequence[int], b: int, n_ctas: int) -> np.ndarray:
    """Rows {module, side, first block, blocks, cta} of the static work split."""
    M = len(d)
    cap = 2 * M + n_ctas + 8
    out = np.zeros((cap, 5), dtype=np.int32)
    n = ctypes.c_int(0)
    st = lib().egeria_debug_plan(M, _i64(d), int(b), int(n_ctas),
                                 out.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)), cap, ctypes.byref(n))
    _check(st, "egeria_debug_plan")
    return out[: n.value].copy()


def egeria_debug_plan_help(d: Sequence[int], b: int, n_ctas: int) -> np.ndarray:
    """Rows {module helped (-1: none), warps lent} per CTA: the help planned for the end of a launch."""
    out = np.zeros((n_ctas, 2), dtype=np.int32)
    st = lib().egeria_debug_plan_help(len(d), _i64(d), int(b), int(n_ctas),
                                      out.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)))
    _check(st, "egeria_debug_plan_help")
    return out


def egeria_debug_plan_tasks(d: Sequence[int], b: int, n_ctas: int, only_module: int = -1):
    """How the end of a launch is cut into tasks: (first[n_ctas, 12] = (module << 16) | task or -1,
    tasks[M, 2] = {tasks, tasks with a warp of their own}, validate)."""
    first = np.zeros((n_ctas, 12), dtype=np.int32)
    tasks = np.zeros((len(d), 2), dtype=np.int32)
    v = ctypes.c_int(0)
    st = lib().egeria_debug_plan_tasks(len(d), _i64(d), int(b), int(n_ctas), int(only_module),
                                       first.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)),
                                       tasks.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)), ctypes.byref(v))
    _check(st, "egeria_debug_plan_tasks")
    return first, tasks, bool(v.value)


def egeria_debug_plan_weighted(d: Sequence[int], b: int, n_ctas: int, weights) -> np.ndarray:
    """The same split with one weight per CTA (None = equal shares)."""
    M = len(d)
    cap = 2 * M + n_ctas + 8
    out = np.zeros((cap, 5), dtype=np.int32)
    n = ctypes.c_int(0)
    wp = None
    if weights is not None:
        w = np.ascontiguousarray(weights, dtype=np.float32)
        assert w.shape == (n_ctas,)
        wp = w.ctypes.data_as(ctypes.POINTER(ctypes.c_float))
    st = lib().egeria_debug_plan_weighted(M, _i64(d), int(b), int(n_ctas), wp,
                                          out.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)), cap, ctypes.byref(n))
    _check(st, "egeria_debug_plan_weighted")
    return out[: n.value].copy()


def egeria_sp_loss_static(At: torch.Tensor, Ar: torch.Tensor, out_loss: Optional[torch.Tensor] = None,
                          stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    """Plasticity of one module through the entry point that allocates nothing.

    The library uses only its built-in scratch array; `out_loss` (device float[1]) is the
    caller's.  Pass it in to keep this wrapper allocation-free as well."""
    if At.dtype != torch.bfloat16 or At.shape != Ar.shape or At.dim() != 2 or not (At.is_cuda and Ar.is_cuda):
        raise ValueError("expected two CUDA bfloat16 [b, d] tensors of the same shape")
    if not (At.is_contiguous() and Ar.is_contiguous()):
        raise ValueError("activations must be contiguous")
    if out_loss is None:
        out_loss = torch.empty(1, dtype=torch.float32, device=At.device)
    with torch.cuda.device(At.device):
        st = lib().egeria_sp_loss_static(_stream_ptr(stream), At.data_ptr(), Ar.data_ptr(), int(At.shape[0]),
                                         int(At.shape[1]), out_loss.data_ptr())
    _check(st, "egeria_sp_loss_static")
    return out_loss


def egeria_sp_loss_static_status(device=None) -> int:
    """Status word of the last egeria_sp_loss_static call on `device` (the current one if None);
    call it after synchronising that call's stream."""
    with torch.cuda.device(device):
        return int(lib().egeria_sp_loss_static_status())


class Context:
    """Owner of one ``egeria_ctx`` and of its workspace tensor."""

    def __init__(self, d: Sequence[int], b_max: int, W: int, T, flags: int = 0, device="cuda"):
        self.d = [int(v) for v in d]
        self.M = len(self.d)
        self.b_max = int(b_max)
        self.flags = int(flags)
        self.device = torch.device(device)
        self._d_arr = _i64(self.d)
        nbytes = egeria_workspace_bytes(self.M, self.d, b_max, W, flags)
        if nbytes == 0:
            raise EgeriaError(ERR_INVALID_ARG, "egeria_workspace_bytes")
        self.workspace_bytes = nbytes
        raw = torch.empty(nbytes + WORKSPACE_ALIGN, dtype=torch.uint8, device=self.device)
        off = (-raw.data_ptr()) % WORKSPACE_ALIGN
        self._raw = raw
        self._ws_ptr = raw.data_ptr() + off
        if np.isscalar(T):
            t_arr, t_all = None, float(T)
        else:
            t_np = np.ascontiguousarray(T, dtype=np.float32)
            assert t_np.shape == (self.M,)
            t_arr, t_all = t_np.ctypes.data_as(ctypes.POINTER(ctypes.c_float)), 0.0
        handle = ctypes.c_void_p()
        with torch.cuda.device(self.device):
            st = lib().egeria_plasticity_create(ctypes.byref(handle), self.M, self._d_arr, self.b_max, int(W),
                                                t_arr, ctypes.c_float(t_all), ctypes.c_void_p(self._ws_ptr),
                                                nbytes, self.flags)
        _check(st, "egeria_plasticity_create")
        self._h = handle

    def close(self) -> None:
        if getattr(self, "_h", None):
            lib().egeria_plasticity_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ------------------------------------------------------------------ calls
    def _ptr_array(self, tensors: Sequence[torch.Tensor], b: int, on_device: bool, active=None):
        if len(tensors) != self.M:
            raise ValueError("one activation per module is required")
        ptrs = (ctypes.c_void_p * self.M)()
        for m, t in enumerate(tensors):
            if active is not None and not active[m]:
                ptrs[m] = None
                continue
            if t.dtype != torch.bfloat16 or t.shape != (b, self.d[m]) or not t.is_contiguous():
                raise ValueError(f"module {m}: expected contiguous bfloat16 [{b}, {self.d[m]}]")
            if t.is_cuda != on_device:
                raise ValueError(f"module {m}: tensor is on the wrong side of the bus")
            ptrs[m] = t.data_ptr()
        return ptrs

    def egeria_sp_loss_batch(self, At: Sequence[torch.Tensor], Ar: Sequence[torch.Tensor],
                             out_losses: Optional[torch.Tensor] = None,
                             stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
        b = int(At[0].shape[0])
        if out_losses is None:
            out_losses = torch.empty(self.M, dtype=torch.float32, device=self.device)
        pa, pr = self._ptr_array(At, b, True), self._ptr_array(Ar, b, True)
        st = lib().egeria_sp_loss_batch(self._h, _stream_ptr(stream), pa, pr, b, self._d_arr,
                                        out_losses.data_ptr())
        _check(st, "egeria_sp_loss_batch")
        return out_losses

    def egeria_sp_loss_subset(self, At, Ar, active, out_losses: torch.Tensor,
                              stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
        """SP loss of the modules with active[m] != 0 only; the other entries of out_losses stay."""
        act = np.ascontiguousarray(active, dtype=np.uint8)
        b = int(next((t for t, a in zip(At, act) if a), next(t for t in At if t is not None)).shape[0])
        pa, pr = self._ptr_array(At, b, True, act), self._ptr_array(Ar, b, True, act)
        st = lib().egeria_sp_loss_subset(self._h, _stream_ptr(stream), pa, pr, b, self._d_arr,
                                         act.ctypes.data_as(ctypes.POINTER(ctypes.c_uint8)), out_losses.data_ptr())
        _check(st, "egeria_sp_loss_subset")
        return out_losses

    def egeria_plasticity_evaluate_subset(self, At, Ar, active, losses: torch.Tensor, slopes: torch.Tensor,
                                          mask: torch.Tensor, stream: Optional[torch.cuda.Stream] = None):
        """One evaluation (loss + freezing rule) of the active modules only, into the caller's tensors."""
        act = np.ascontiguousarray(active, dtype=np.uint8)
        b = int(next((t for t, a in zip(At, act) if a), next(t for t in At if t is not None)).shape[0])
        pa, pr = self._ptr_array(At, b, True, act), self._ptr_array(Ar, b, True, act)
        st = lib().egeria_plasticity_evaluate_subset(self._h, _stream_ptr(stream), pa, pr, b, self._d_arr,
                                                     act.ctypes.data_as(ctypes.POINTER(ctypes.c_uint8)),
                                                     losses.data_ptr(), slopes.data_ptr(), mask.data_ptr())
        _check(st, "egeria_plasticity_evaluate_subset")
        return losses, slopes, mask

    def egeria_plasticity_evaluate(self, At: Sequence[torch.Tensor], Ar: Sequence[torch.Tensor],
                                   stream: Optional[torch.cuda.Stream] = None):
        """Losses, slopes and freeze mask of one evaluation (SP loss + freezing rule)."""
        b = int(At[0].shape[0])
        losses = torch.empty(self.M, dtype=torch.float32, device=self.device)
        slopes = torch.empty(self.M, dtype=torch.float64, device=self.device)
        mask = torch.empty(self.M, dtype=torch.uint8, device=self.device)
        pa, pr = self._ptr_array(At, b, True), self._ptr_array(Ar, b, True)
        st = lib().egeria_plasticity_evaluate(self._h, _stream_ptr(stream), pa, pr, b, self._d_arr,
                                              losses.data_ptr(), slopes.data_ptr(), mask.data_ptr())
        _check(st, "egeria_plasticity_evaluate")
        return losses, slopes, mask

    def plasticity_evaluate_raw(self, pa, pr, b: int, losses_ptr: int, slopes_ptr: int, mask_ptr: int,
                                stream_ptr: int) -> None:
        """Same call with ready-made pointer arrays (benchmark loops)."""
        _check(lib().egeria_plasticity_evaluate(self._h, stream_ptr, pa, pr, b, self._d_arr, losses_ptr,
                                                slopes_ptr, mask_ptr), "egeria_plasticity_evaluate")

    def sp_loss_batch_raw(self, pa, pr, b: int, out_ptr: int, stream_ptr: int) -> None:
        """Same call with ready-made pointer arrays (benchmark loops)."""
        _check(lib().egeria_sp_loss_batch(self._h, stream_ptr, pa, pr, b, self._d_arr, out_ptr),
               "egeria_sp_loss_batch")

    def egeria_sp_loss_batch_host(self, At: Sequence[torch.Tensor], Ar: Sequence[torch.Tensor],
                                  out_losses: Optional[torch.Tensor] = None,
                                  stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
        b = int(At[0].shape[0])
        if out_losses is None:
            out_losses = torch.empty(self.M, dtype=torch.float32)
        pa, pr = self._ptr_array(At, b, False), self._ptr_array(Ar, b, False)
        st = lib().egeria_sp_loss_batch_host(self._h, _stream_ptr(stream), pa, pr, b, self._d_arr,
                                             out_losses.data_ptr())
        _check(st, "egeria_sp_loss_batch_host")
        return out_losses

    def egeria_plasticity_step(self, losses: torch.Tensor, out_slopes: Optional[torch.Tensor] = None,
                               out_mask: Optional[torch.Tensor] = None,
                               stream: Optional[torch.cuda.Stream] = None):
        assert losses.is_cuda and losses.dtype == torch.float32 and losses.numel() == self.M
        if out_slopes is None:
            out_slopes = torch.empty(self.M, dtype=torch.float64, device=self.device)
        if out_mask is None:
            out_mask = torch.empty(self.M, dtype=torch.uint8, device=self.device)
        st = lib().egeria_plasticity_step(self._h, _stream_ptr(stream), losses.data_ptr(),
                                          out_slopes.data_ptr(), out_mask.data_ptr())
        _check(st, "egeria_plasticity_step")
        return out_slopes, out_mask

    def egeria_plasticity_replay(self, hist: torch.Tensor, stream: Optional[torch.cuda.Stream] = None):
        assert hist.is_cuda and hist.dtype == torch.float32 and hist.dim() == 2 and hist.shape[0] == self.M
        hist = hist.contiguous()
        H = int(hist.shape[1])
        slopes = torch.empty((self.M, H), dtype=torch.float64, device=self.device)
        mask = torch.empty(self.M, dtype=torch.uint8, device=self.device)
        freeze_eval = torch.empty(self.M, dtype=torch.int32, device=self.device)
        st = lib().egeria_plasticity_replay(self._h, _stream_ptr(stream), hist.data_ptr(), H, slopes.data_ptr(),
                                            mask.data_ptr(), freeze_eval.data_ptr())
        _check(st, "egeria_plasticity_replay")
        return slopes, mask, freeze_eval

    def egeria_plasticity_replay_lr(self, hist: torch.Tensor, lr: Optional[torch.Tensor],
                                    stream: Optional[torch.cuda.Stream] = None):
        """Whole histories with the unfreezing rule: (slopes [M, H], frozen [H, M], window [H],
        restarted [H], mask [M], freeze_eval [M]) device tensors."""
        assert hist.is_cuda and hist.dtype == torch.float32 and hist.dim() == 2 and hist.shape[0] == self.M
        hist = hist.contiguous()
        H = int(hist.shape[1])
        if lr is not None:
            assert lr.is_cuda and lr.dtype == torch.float64 and lr.numel() == H
            lr = lr.contiguous()
        slopes = torch.empty((self.M, H), dtype=torch.float64, device=self.device)
        frozen = torch.empty((H, self.M), dtype=torch.uint8, device=self.device)
        window = torch.empty(max(H, 1), dtype=torch.int32, device=self.device)
        restarted = torch.empty(max(H, 1), dtype=torch.uint8, device=self.device)
        mask = torch.empty(self.M, dtype=torch.uint8, device=self.device)
        freeze_eval = torch.empty(self.M, dtype=torch.int32, device=self.device)
        st = lib().egeria_plasticity_replay_lr(self._h, _stream_ptr(stream), hist.data_ptr(),
                                               lr.data_ptr() if lr is not None else None, H, slopes.data_ptr(),
                                               frozen.data_ptr(), window.data_ptr(), restarted.data_ptr(),
                                               mask.data_ptr(), freeze_eval.data_ptr())
        _check(st, "egeria_plasticity_replay_lr")
        return slopes, frozen, window[:H], restarted[:H], mask, freeze_eval

    def egeria_plasticity_set_lr(self, lr: float) -> None:
        _check(lib().egeria_plasticity_set_lr(self._h, ctypes.c_double(lr)), "egeria_plasticity_set_lr")

    def egeria_plasticity_restarts(self) -> int:
        return int(lib().egeria_plasticity_restarts(self._h))

    def egeria_plasticity_reset(self, halve_W: bool = False, stream: Optional[torch.cuda.Stream] = None) -> None:
        _check(lib().egeria_plasticity_reset(self._h, _stream_ptr(stream), int(bool(halve_W))),
               "egeria_plasticity_reset")

    def egeria_bootstrap_step(self, train_loss: torch.Tensor, rate_tol: float = 0.1,
                              stream: Optional[torch.cuda.Stream] = None):
        """One more training-loss reading for the bootstrapping detector: (rate, done) device tensors."""
        assert train_loss.is_cuda and train_loss.dtype == torch.float32 and train_loss.numel() == 1
        rate = torch.empty(1, dtype=torch.float64, device=self.device)
        done = torch.empty(1, dtype=torch.uint8, device=self.device)
        _check(lib().egeria_bootstrap_step(self._h, _stream_ptr(stream), train_loss.data_ptr(), ctypes.c_float(rate_tol),
                                           rate.data_ptr(), done.data_ptr()), "egeria_bootstrap_step")
        return rate, done

    def egeria_bootstrap_replay(self, loss_hist: torch.Tensor, rate_tol: float = 0.1,
                                stream: Optional[torch.cuda.Stream] = None):
        assert loss_hist.is_cuda and loss_hist.dtype == torch.float32 and loss_hist.dim() == 1
        loss_hist = loss_hist.contiguous()
        H = int(loss_hist.shape[0])
        rates = torch.empty(max(H, 1), dtype=torch.float64, device=self.device)
        end = torch.empty(1, dtype=torch.int32, device=self.device)
        _check(lib().egeria_bootstrap_replay(self._h, _stream_ptr(stream), loss_hist.data_ptr(), H,
                                             ctypes.c_float(rate_tol), rates.data_ptr(), end.data_ptr()),
               "egeria_bootstrap_replay")
        return rates[:H], end

    def egeria_bootstrap_reset(self, stream: Optional[torch.cuda.Stream] = None) -> None:
        _check(lib().egeria_bootstrap_reset(self._h, _stream_ptr(stream)), "egeria_bootstrap_reset")

    def egeria_plasticity_state_bytes(self) -> int:
        return int(lib().egeria_plasticity_state_bytes(self._h))

    def egeria_plasticity_export(self, stream: Optional[torch.cuda.Stream] = None) -> np.ndarray:
        """The freezing-rule state as host bytes (synchronises the stream)."""
        buf = np.zeros(self.egeria_plasticity_state_bytes(), dtype=np.uint8)
        _check(lib().egeria_plasticity_export(self._h, _stream_ptr(stream), buf.ctypes.data, buf.nbytes),
               "egeria_plasticity_export")
        return buf

    def egeria_plasticity_import(self, buf: np.ndarray, stream: Optional[torch.cuda.Stream] = None) -> None:
        buf = np.ascontiguousarray(buf, dtype=np.uint8)
        _check(lib().egeria_plasticity_import(self._h, _stream_ptr(stream), buf.ctypes.data, buf.nbytes),
               "egeria_plasticity_import")

    def egeria_plasticity_window(self) -> int:
        return int(lib().egeria_plasticity_window(self._h))

    def egeria_debug_dump_gram(self, module: int, b: int, stream: Optional[torch.cuda.Stream] = None):
        gt = torch.empty((b, b), dtype=torch.float32, device=self.device)
        gr = torch.empty((b, b), dtype=torch.float32, device=self.device)
        st = lib().egeria_debug_dump_gram(self._h, _stream_ptr(stream), int(module), gt.data_ptr(), gr.data_ptr())
        _check(st, "egeria_debug_dump_gram")
        return gt, gr

    def egeria_debug_stall_next(self, kind: int) -> None:
        _check(lib().egeria_debug_stall_next(self._h, int(kind)), "egeria_debug_stall_next")

    def egeria_device_status(self) -> int:
        return int(lib().egeria_device_status(self._h))

    def check_device_status(self) -> None:
        _check(self.egeria_device_status(), "egeria_device_status")

    def egeria_debug_check_record(self) -> np.ndarray:
        """The checked build's record of the first failed index check (five int32, all zero if none)."""
        out = np.zeros(5, dtype=np.int32)
        _check(lib().egeria_debug_check_record(self._h, out.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))),
               "egeria_debug_check_record")
        return out

    def egeria_gram_kernel_time(self):
        """(total milliseconds, calls) of the Gram kernels since the last query."""
        ms, n = ctypes.c_double(), ctypes.c_int64()
        _check(lib().egeria_gram_kernel_time(self._h, ctypes.byref(ms), ctypes.byref(n)), "egeria_gram_kernel_time")
        return ms.value, n.value

    def egeria_split_weights(self):
        """(n, weights): n > 0 once the split follows measured streaming rates."""
        w = np.ones(256, dtype=np.float32)
        n = int(lib().egeria_split_weights(self._h, w.ctypes.data_as(ctypes.POINTER(ctypes.c_float)), 256))
        return n, w[: max(n, 0)].copy()

    def egeria_launch_count(self) -> int:
        return int(lib().egeria_launch_count(self._h))
