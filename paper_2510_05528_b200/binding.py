"""ctypes binding of libarmor (see include/armor.h).  Argument marshalling only: every step of the
method runs in the library's CUDA kernels.  PyTorch supplies device memory and streams.

The module-level functions carry the names of the C entry points and take torch CUDA tensors.
``ArmorContext`` bundles a configuration with its workspace.  There is no CPU path: if the shared
library is missing, or a tensor is not on a CUDA device, the call raises."""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libarmor.so")

H_FULL, H_DIAG = 0, 1
SELECT_L1_RANDOM, SELECT_L1_GREEDY, SELECT_UNIFORM_RANDOM, SELECT_L2_RANDOM = 0, 1, 2, 3
S_EXACT, S_BETA = 0, 1
AB_EXACT, AB_GD, AB_ADAM = 0, 1, 2
PREC_FP32X3, PREC_TF32, PREC_SIMT, PREC_FP16X3 = 0, 1, 2, 3
PHASE_A, PHASE_B, PHASE_S, PHASE_MASK = 1, 2, 4, 8
DTYPE_F32, DTYPE_BF16, DTYPE_BF16_SPARSE = 0, 1, 2

EXPORTS = ["armor_workspace_bytes", "armor_create", "armor_destroy", "armor_gram", "armor_init",
           "armor_bcd_step", "armor_proxy_loss", "armor_apply", "armor_packed_core_bytes", "armor_pack_core", "armor_apply_packed",
           "armor_packed_layer_bytes", "armor_pack_layer", "armor_apply_layer",
           "armor_get_device_status",
           "armor_status_string", "armor_launch_count", "armor_gemm_timing_enable", "armor_gemm_timing",
           "armor_normalize_noalloc", "armor_block_product", "armor_block_product_dual", "armor_block_product_two_sided", "armor_selftest_wait_timeout", "armor_kernel_timing_enable", "armor_use_graphs", "armor_fuse_grams",
           "armor_kernel_timing"]


class ArmorError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} (status {code})")


class armor_config(C.Structure):
    _fields_ = [("d_out", C.c_int64), ("d_in", C.c_int64), ("d_block", C.c_int32), ("n_keep", C.c_int32),
                ("m_group", C.c_int32), ("h_mode", C.c_int32), ("select_mode", C.c_int32),
                ("s_step", C.c_int32), ("precision", C.c_int32), ("normalize", C.c_int32),
                ("phases", C.c_int32), ("ab_step", C.c_int32), ("mask_sweeps", C.c_int32), ("mask_groups", C.c_int32), ("ridge", C.c_float), ("adam_lr", C.c_float),
                ("adam_beta1", C.c_float), ("adam_beta2", C.c_float), ("adam_eps", C.c_float), ("seed", C.c_uint64)]


STATS_DTYPE = np.dtype([("loss_start", "<f8"), ("loss_A", "<f8"), ("loss_B", "<f8"), ("loss_S", "<f8"),
                        ("loss_mask", "<f8"), ("delta_L_mask", "<f8"), ("tau_B", "<f4"), ("tau_S", "<f4"),
                        ("groups_changed", "<i4"), ("mask_accepted", "<i4"), ("chol_failed", "<i4"),
                        ("reserved", "<i4")])

_lib = None


def lib() -> C.CDLL:
    """Loads libarmor.so on first use; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(f"{LIB_PATH} not found: build it with `python -m paper_2510_05528_b200.build`")
        L = C.CDLL(LIB_PATH)
        vp, i32, i64 = C.c_void_p, C.c_int32, C.c_int64
        L.armor_workspace_bytes.argtypes = [C.POINTER(armor_config), C.POINTER(C.c_size_t)]
        L.armor_create.argtypes = [C.POINTER(vp), C.POINTER(armor_config), vp, C.c_size_t]
        L.armor_destroy.argtypes = [vp]
        L.armor_gram.argtypes = [vp, vp, i32, i64, i64, vp, vp]
        L.armor_init.argtypes = [vp] + [vp] * 9 + [vp]
        L.armor_bcd_step.argtypes = [vp] + [vp] * 6 + [i64, i32, vp, vp]
        L.armor_proxy_loss.argtypes = [vp] + [vp] * 6 + [vp]
        L.armor_apply.argtypes = [vp] + [vp] * 8 + [i32, i64, vp]
        L.armor_packed_core_bytes.argtypes = [C.POINTER(armor_config), C.POINTER(C.c_size_t)]
        L.armor_pack_core.argtypes = [vp, vp, vp, vp, vp]
        L.armor_apply_packed.argtypes = [vp] + [vp] * 7 + [i64, vp]
        L.armor_packed_layer_bytes.argtypes = [C.POINTER(armor_config), C.POINTER(C.c_size_t)]
        L.armor_pack_layer.argtypes = [vp] + [vp] * 7 + [vp]
        L.armor_apply_layer.argtypes = [vp, vp, vp, vp, i64, vp]
        L.armor_get_device_status.argtypes = [vp, C.POINTER(i32), i32]
        L.armor_status_string.argtypes = [C.c_int]
        L.armor_status_string.restype = C.c_char_p
        L.armor_launch_count.argtypes = [vp]
        L.armor_launch_count.restype = i64
        L.armor_normalize_noalloc.argtypes = [vp, i64, i64, vp, vp, vp, vp]
        L.armor_block_product.argtypes = [vp, i32, i32, vp, vp, vp, i64, i64, C.c_float, vp, C.c_float, i32, vp]
        L.armor_block_product_dual.argtypes = [vp, vp, vp, vp, vp, vp, i32, vp]
        L.armor_block_product_two_sided.argtypes = [vp, vp, i32, vp, vp, i32, vp, C.c_float, i32, vp]
        L.armor_gemm_timing_enable.argtypes = [vp, i32]
        L.armor_gemm_timing.argtypes = [vp, C.POINTER(i64), C.POINTER(C.c_double), C.POINTER(C.c_double)]
        L.armor_kernel_timing_enable.argtypes = [vp, i32]
        L.armor_use_graphs.argtypes = [vp, i32]
        L.armor_fuse_grams.argtypes = [vp, i32]
        L.armor_kernel_timing.argtypes = [vp, i32, C.POINTER(i64), C.POINTER(C.c_double), C.POINTER(C.c_double)]
        L.armor_selftest_wait_timeout.argtypes = [vp, i64, vp, vp]
        for name in EXPORTS:
            if name not in ("armor_status_string", "armor_launch_count"):
                getattr(L, name).restype = C.c_int
        _lib = L
    return _lib


def status_string(code: int) -> str:
    return lib().armor_status_string(int(code)).decode()


def _check(code: int, where: str) -> None:
    if code != 0:
        raise ArmorError(code, where)


def _ptr(t: torch.Tensor | None, dtype=None, name: str = "tensor") -> C.c_void_p:
    if t is None:
        return C.c_void_p(0)
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor (this library has no CPU path)")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    if dtype is not None and t.dtype != dtype:
        raise ValueError(f"{name} must have dtype {dtype}, got {t.dtype}")
    return C.c_void_p(t.data_ptr())


def _stream() -> C.c_void_p:
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def make_config(d_out, d_in, d_block, *, n_keep=2, m_group=4, h_mode=H_FULL, select_mode=SELECT_L1_RANDOM,
                s_step=S_EXACT, precision=PREC_FP16X3, normalize=0, phases=0, ab_step=AB_EXACT, mask_sweeps=1, mask_groups=1, ridge=1e-6,
                adam_lr=0.0, adam_beta1=0.0, adam_beta2=0.0, adam_eps=0.0, seed=0) -> armor_config:
    return armor_config(d_out, d_in, d_block, n_keep, m_group, h_mode, select_mode, s_step, precision,
                        int(normalize), phases, ab_step, mask_sweeps, mask_groups, ridge, adam_lr, adam_beta1, adam_beta2, adam_eps, seed)


# ---------------------------------------------------------------- C entry points, same names
def armor_workspace_bytes(cfg: armor_config) -> int:
    n = C.c_size_t(0)
    _check(lib().armor_workspace_bytes(C.byref(cfg), C.byref(n)), "armor_workspace_bytes")
    return int(n.value)


def armor_create(cfg: armor_config, workspace: torch.Tensor) -> C.c_void_p:
    ctx = C.c_void_p(0)
    _check(lib().armor_create(C.byref(ctx), C.byref(cfg), _ptr(workspace, name="workspace"),
                              workspace.numel() * workspace.element_size()), "armor_create")
    return ctx


def armor_destroy(ctx) -> None:
    _check(lib().armor_destroy(ctx), "armor_destroy")


def armor_gram(ctx, X: torch.Tensor, H: torch.Tensor) -> None:
    if X.dim() != 2 or X.stride(1) != 1:
        raise ValueError("X must be [n_rows, d_in] with unit column stride")
    if not X.is_cuda or X.dtype not in (torch.float32, torch.bfloat16):
        raise ValueError("X must be a float32 or bfloat16 CUDA tensor (this library has no CPU path)")
    ldx = X.stride(0) if X.shape[0] > 1 else X.shape[1]
    _check(lib().armor_gram(ctx, C.c_void_p(X.data_ptr()), DTYPE_BF16 if X.dtype == torch.bfloat16 else DTYPE_F32,
                            X.shape[0], ldx,
                            _ptr(H, torch.float32, "H"), _stream()), "armor_gram")


def armor_init(ctx, W, H, Wbar, r1, r2, A, B, S, M) -> None:
    f = torch.float32
    _check(lib().armor_init(ctx, _ptr(W, f, "W"), _ptr(H, f, "H"), _ptr(Wbar, f, "Wbar"), _ptr(r1, f, "r1"),
                            _ptr(r2, f, "r2"), _ptr(A, f, "A"), _ptr(B, f, "B"), _ptr(S, f, "S"),
                            _ptr(M, torch.uint8, "M"), _stream()), "armor_init")


def armor_bcd_step(ctx, Wbar, H, A, B, S, M, t_first: int, n_iters: int, stats: torch.Tensor | None) -> None:
    f = torch.float32
    _check(lib().armor_bcd_step(ctx, _ptr(Wbar, f, "Wbar"), _ptr(H, f, "H"), _ptr(A, f, "A"), _ptr(B, f, "B"),
                                _ptr(S, f, "S"), _ptr(M, torch.uint8, "M"), int(t_first), int(n_iters),
                                _ptr(stats, torch.uint8, "stats"), _stream()), "armor_bcd_step")


def armor_proxy_loss(ctx, Wbar, H, A, B, S, loss: torch.Tensor) -> None:
    f = torch.float32
    _check(lib().armor_proxy_loss(ctx, _ptr(Wbar, f, "Wbar"), _ptr(H, f, "H"), _ptr(A, f, "A"), _ptr(B, f, "B"),
                                  _ptr(S, f, "S"), _ptr(loss, torch.float64, "loss"), _stream()), "armor_proxy_loss")


def armor_apply(ctx, A, B, S, M, r1, r2, x, y, sparse: bool = False) -> None:
    f = torch.float32
    if x.dtype != y.dtype or x.dtype not in (torch.float32, torch.bfloat16):
        raise ValueError("x and y must both be float32 or both be bfloat16")
    dt = DTYPE_BF16 if x.dtype == torch.bfloat16 else DTYPE_F32
    if sparse:
        if dt != DTYPE_BF16:
            raise ValueError("the sparse tensor-core forward takes bf16 x and y")
        dt = DTYPE_BF16_SPARSE
    _check(lib().armor_apply(ctx, _ptr(A, f, "A"), _ptr(B, f, "B"), _ptr(S, f, "S"), _ptr(M, torch.uint8, "M"),
                             _ptr(r1, f, "r1"), _ptr(r2, f, "r2"), _ptr(x, x.dtype, "x"), _ptr(y, y.dtype, "y"), dt,
                             x.shape[0], _stream()), "armor_apply")


def armor_packed_core_bytes(cfg: armor_config) -> int:
    n = C.c_size_t(0)
    _check(lib().armor_packed_core_bytes(C.byref(cfg), C.byref(n)), "armor_packed_core_bytes")
    return int(n.value)


def armor_pack_core(ctx, S, M, packed) -> None:
    _check(lib().armor_pack_core(ctx, _ptr(S, torch.float32, "S"), _ptr(M, torch.uint8, "M"),
                                 _ptr(packed, torch.uint8, "packed"), _stream()), "armor_pack_core")


def armor_apply_packed(ctx, A, B, packed, r1, r2, x, y) -> None:
    f = torch.float32
    if x.dtype != torch.bfloat16 or y.dtype != torch.bfloat16:
        raise ValueError("the packed forward takes bf16 x and y")
    _check(lib().armor_apply_packed(ctx, _ptr(A, f, "A"), _ptr(B, f, "B"), _ptr(packed, torch.uint8, "packed"),
                                    _ptr(r1, f, "r1"), _ptr(r2, f, "r2"), _ptr(x, x.dtype, "x"), _ptr(y, y.dtype, "y"),
                                    x.shape[0], _stream()), "armor_apply_packed")


def armor_packed_layer_bytes(cfg: armor_config) -> int:
    n = C.c_size_t(0)
    _check(lib().armor_packed_layer_bytes(C.byref(cfg), C.byref(n)), "armor_packed_layer_bytes")
    return int(n.value)


def armor_pack_layer(ctx, A, B, S, M, r1, r2, packed) -> None:
    f = torch.float32
    _check(lib().armor_pack_layer(ctx, _ptr(A, f, "A"), _ptr(B, f, "B"), _ptr(S, f, "S"), _ptr(M, torch.uint8, "M"),
                                  _ptr(r1, f, "r1"), _ptr(r2, f, "r2"), _ptr(packed, torch.uint8, "packed"), _stream()),
           "armor_pack_layer")


def armor_apply_layer(ctx, packed, x, y) -> None:
    if x.dtype != torch.bfloat16 or y.dtype != torch.bfloat16:
        raise ValueError("the packed layer takes bf16 x and y")
    _check(lib().armor_apply_layer(ctx, _ptr(packed, torch.uint8, "packed"), _ptr(x, x.dtype, "x"), _ptr(y, y.dtype, "y"),
                                   x.shape[0], _stream()), "armor_apply_layer")


def armor_get_device_status(ctx, n: int = 16) -> list[int]:
    buf = (C.c_int32 * n)()
    _check(lib().armor_get_device_status(ctx, buf, n), "armor_get_device_status")
    return list(buf)


def armor_selftest_wait_timeout(ctx, limit_cycles: int, result: torch.Tensor) -> None:
    _check(lib().armor_selftest_wait_timeout(ctx, int(limit_cycles), _ptr(result, torch.int32, "result"), _stream()),
           "armor_selftest_wait_timeout")


def armor_launch_count(ctx) -> int:
    return int(lib().armor_launch_count(ctx))


def armor_normalize_noalloc(W: torch.Tensor, Wbar: torch.Tensor, r1: torch.Tensor, r2: torch.Tensor) -> None:
    """Normalisation without a context or a workspace, for callers that may not allocate device memory:
    the scratch is a fixed 4 MiB array inside the library (d_in <= 8192, d_out <= 65536).  All arguments are
    the caller's CUDA tensors; this wrapper allocates nothing either.  Calls that overlap on one GPU race."""
    f = torch.float32
    if W.dim() != 2:
        raise ValueError("W must be [d_out, d_in]")
    _check(lib().armor_normalize_noalloc(_ptr(W, f, "W"), W.shape[0], W.shape[1], _ptr(Wbar, f, "Wbar"),
                                         _ptr(r1, f, "r1"), _ptr(r2, f, "r2"), _stream()), "armor_normalize_noalloc")


def armor_block_product(ctx, side: int, transpose: bool, blocks, x, out, alpha=1.0, add=None, beta=0.0, path=-1) -> None:
    """out = alpha * (x . Q or Q . x) + beta * add with the block-diagonal Q (see armor.h)."""
    f = torch.float32
    _check(lib().armor_block_product(ctx, int(side), int(bool(transpose)), _ptr(blocks, f, "blocks"), _ptr(x, f, "x"),
                                     _ptr(out, f, "out"), x.shape[0], x.shape[1], float(alpha), _ptr(add, f, "add"),
                                     float(beta), int(path), _stream()), "armor_block_product")


def armor_block_product_two_sided(ctx, left, transpose_left: bool, x, right, transpose_right: bool, out, alpha=1.0,
                                  path=-1) -> None:
    """out = alpha * Lop . x . Rop with both block-diagonal wrappers (see armor.h)."""
    f = torch.float32
    _check(lib().armor_block_product_two_sided(ctx, _ptr(left, f, "left"), int(bool(transpose_left)), _ptr(x, f, "x"),
                                               _ptr(right, f, "right"), int(bool(transpose_right)), _ptr(out, f, "out"),
                                               float(alpha), int(path), _stream()), "armor_block_product_two_sided")


def armor_block_product_dual(ctx, blocks, x1, x2, out, path=-1) -> float:
    """out = Q . x2 per block row; returns <Q . x1, Q . x2> (see armor.h)."""
    f = torch.float32
    dot = torch.zeros(1, dtype=torch.float64, device=out.device)
    _check(lib().armor_block_product_dual(ctx, _ptr(blocks, f, "blocks"), _ptr(x1, f, "x1"), _ptr(x2, f, "x2"),
                                          _ptr(out, f, "out"), _ptr(dot, torch.float64, "dot"), int(path), _stream()),
           "armor_block_product_dual")
    return float(dot.item())


def armor_gemm_timing_enable(ctx, enable: bool) -> None:
    _check(lib().armor_gemm_timing_enable(ctx, int(bool(enable))), "armor_gemm_timing_enable")


KERNEL_CLASSES = ["gemm", "block_product", "block_gram", "cholesky", "axpy", "dot", "masked_copy", "mask_select",
                  "mask_guard", "operand_split", "gram_staging", "init", "small", "forward"]


def armor_fuse_grams(ctx, enable: bool) -> None:
    _check(lib().armor_fuse_grams(ctx, 1 if enable else 0), "armor_fuse_grams")


def armor_use_graphs(ctx, enable: bool) -> None:
    _check(lib().armor_use_graphs(ctx, 1 if enable else 0), "armor_use_graphs")


def armor_kernel_timing_enable(ctx, level: int) -> None:
    _check(lib().armor_kernel_timing_enable(ctx, int(level)), "armor_kernel_timing_enable")


def armor_kernel_timing(ctx) -> dict:
    """{class name: (launches, total ms, total work)} since the last read; clears the record."""
    n = len(KERNEL_CLASSES)
    cnt, ms, work = (C.c_int64 * n)(), (C.c_double * n)(), (C.c_double * n)()
    _check(lib().armor_kernel_timing(ctx, n, cnt, ms, work), "armor_kernel_timing")
    return {name: (int(cnt[k]), float(ms[k]), float(work[k])) for k, name in enumerate(KERNEL_CLASSES)}


def armor_gemm_timing(ctx) -> tuple[int, float, float]:
    """(timed launches, total milliseconds, total algorithmic flops) since the last call."""
    n, ms, fl = C.c_int64(0), C.c_double(0), C.c_double(0)
    _check(lib().armor_gemm_timing(ctx, C.byref(n), C.byref(ms), C.byref(fl)), "armor_gemm_timing")
    return int(n.value), float(ms.value), float(fl.value)


# ---------------------------------------------------------------- convenience wrapper
@dataclass
class LayerState:
    Wbar: torch.Tensor
    A: torch.Tensor
    B: torch.Tensor
    S: torch.Tensor
    M: torch.Tensor
    r1: torch.Tensor | None = None
    r2: torch.Tensor | None = None


class ArmorContext:
    """A configuration plus its device workspace.  All methods enqueue on torch's current stream."""

    def __init__(self, d_out, d_in, d_block, device="cuda:0", **kw):
        self.device = torch.device(device)
        if self.device.type != "cuda":
            raise ValueError("ArmorContext needs a CUDA device")
        self.cfg = make_config(d_out, d_in, d_block, **kw)
        self.d_out, self.d_in, self.d_block = d_out, d_in, d_block
        nbytes = armor_workspace_bytes(self.cfg)
        with torch.cuda.device(self.device):
            self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
            off = (-self.workspace.data_ptr()) % 256
            self._ws_view = self.workspace[off: off + nbytes]
            self.ctx = armor_create(self.cfg, self._ws_view)

    def close(self):
        if getattr(self, "ctx", None) is not None:
            armor_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- calls
    def new_gram(self) -> torch.Tensor:
        return torch.zeros(self.d_in, self.d_in, dtype=torch.float32, device=self.device)

    def gram(self, X: torch.Tensor, H: torch.Tensor) -> torch.Tensor:
        armor_gram(self.ctx, X, H)
        return H

    def init(self, W: torch.Tensor, H: torch.Tensor) -> LayerState:
        dev, f = self.device, torch.float32
        nbo, nbi, db = self.d_out // self.d_block, self.d_in // self.d_block, self.d_block
        st = LayerState(
            Wbar=torch.empty_like(W),
            A=torch.empty(nbo, db, db, dtype=f, device=dev), B=torch.empty(nbi, db, db, dtype=f, device=dev),
            S=torch.empty_like(W), M=torch.empty(self.d_out, self.d_in // self.cfg.m_group, dtype=torch.uint8, device=dev))
        if self.cfg.normalize:
            st.r1 = torch.empty(self.d_in, dtype=f, device=dev)
            st.r2 = torch.empty(self.d_out, dtype=f, device=dev)
        armor_init(self.ctx, W, H, st.Wbar, st.r1, st.r2, st.A, st.B, st.S, st.M)
        return st

    def bcd_step(self, st: LayerState, H: torch.Tensor, t_first: int, n_iters: int, want_stats: bool = True):
        stats = None
        if want_stats:
            stats = torch.zeros(max(n_iters, 1) * STATS_DTYPE.itemsize, dtype=torch.uint8, device=self.device)
        armor_bcd_step(self.ctx, st.Wbar, H, st.A, st.B, st.S, st.M, t_first, n_iters, stats)
        return stats

    @staticmethod
    def read_stats(stats: torch.Tensor) -> np.ndarray:
        """Device->host copy of the per-iteration records (synchronises)."""
        return stats.cpu().numpy().view(STATS_DTYPE)

    def proxy_loss(self, st: LayerState, H: torch.Tensor) -> torch.Tensor:
        out = torch.zeros(1, dtype=torch.float64, device=self.device)
        armor_proxy_loss(self.ctx, st.Wbar, H, st.A, st.B, st.S, out)
        return out

    def apply(self, st: LayerState, x: torch.Tensor, denormalize: bool = False, sparse: bool = False) -> torch.Tensor:
        y = torch.empty(x.shape[0], self.d_out, dtype=x.dtype, device=self.device)
        r1, r2 = (st.r1, st.r2) if denormalize else (None, None)
        armor_apply(self.ctx, st.A, st.B, st.S, st.M, r1, r2, x, y, sparse)
        return y

    def pack_core(self, st: LayerState) -> torch.Tensor:
        """The 2:4 core in the sparse tensor cores' format (kept values, then positions), packed once."""
        packed = torch.empty(armor_packed_core_bytes(self.cfg), dtype=torch.uint8, device=self.device)
        armor_pack_core(self.ctx, st.S, st.M, packed)
        return packed

    def apply_packed(self, st: LayerState, packed: torch.Tensor, x: torch.Tensor, denormalize: bool = False) -> torch.Tensor:
        y = torch.empty(x.shape[0], self.d_out, dtype=x.dtype, device=self.device)
        r1, r2 = (st.r1, st.r2) if denormalize else (None, None)
        armor_apply_packed(self.ctx, st.A, st.B, packed, r1, r2, x, y)
        return y

    def pack_layer(self, st: LayerState, denormalize: bool = False) -> torch.Tensor:
        """Core and wrappers packed for the all-bf16 forward (the normalisation's scales folded into the wrappers)."""
        packed = torch.empty(armor_packed_layer_bytes(self.cfg), dtype=torch.uint8, device=self.device)
        r1, r2 = (st.r1, st.r2) if denormalize else (None, None)
        armor_pack_layer(self.ctx, st.A, st.B, st.S, st.M, r1, r2, packed)
        return packed

    def apply_layer(self, packed: torch.Tensor, x: torch.Tensor) -> torch.Tensor:
        y = torch.empty(x.shape[0], self.d_out, dtype=x.dtype, device=self.device)
        armor_apply_layer(self.ctx, packed, x, y)
        return y

    def device_status(self) -> list[int]:
        torch.cuda.current_stream().synchronize()
        return armor_get_device_status(self.ctx)

    def launch_count(self) -> int:
        return armor_launch_count(self.ctx)
