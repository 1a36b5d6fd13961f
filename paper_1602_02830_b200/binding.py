"""ctypes binding of libbnn_b200.so: same names as the C ABI, argument marshalling only.

Tensors are torch tensors that own device (or, where the C call says so, host) memory; this module
passes their data pointers, leading dimensions and sizes and raises on a non-zero status.  No step of
the method is computed here.  The library is loaded on first use; if it has not been built the call
fails with an error -- there is no fallback path.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, Structure, c_double, c_int, c_int32, c_int64, c_size_t, c_void_p

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libbnn_b200.so")

BNN_F32, BNN_F16, BNN_I8 = 0, 1, 2
VARIANT_AUTO, VARIANT_PLAIN, VARIANT_CSA = 0, 1, 2
ENGINE_AUTO, ENGINE_POPC, ENGINE_TENSOR = 0, 1, 2

EXPORTS = (
    "bnn_create", "bnn_destroy", "bnn_status_string", "bnn_last_cuda_error", "bnn_set_workspace",
    "bnn_set_popc_variant", "bnn_pack_signs", "bnn_xnor_gemm", "bnn_binary_dense", "bnn_first_layer_bitplanes",
    "bnn_binary_conv2d", "bnn_mlp_workspace_bytes", "bnn_mlp_forward", "bnn_mlp_forward_host",
    "bnn_fold_batchnorm", "bnn_mlp_noalloc_max_bytes", "bnn_mlp_forward_noalloc", "bnn_set_engine",
    "bnn_gemm_workspace_bytes", "bnn_device_status", "bnn_conv_workspace_bytes", "bnn_set_tile_rows", "bnn_set_pair_mode", "bnn_expanded_ld",
    "bnn_expanded_bytes", "bnn_expand_signs", "bnn_baseline_gemm_f32", "bnn_convnet_workspace_bytes",
    "bnn_convnet_forward", "bnn_set_operand_bits", "bnn_expanded_ld_f4",
    "bnn_expanded_bytes_f4", "bnn_expand_signs_f4", "bnn_binary_dense_expanded", "bnn_set_wait_limit_ns",
    "bnn_debug_drop_loads", "bnn_debug_ring_position", "bnn_set_conv_form", "bnn_measure_pipe_rates", "bnn_last_tensor_kernel", "bnn_last_tensor_kernel_clock", "bnn_set_conv_filter_repetition",
    "bnn_filter_repetition_workspace_bytes", "bnn_filter_repetition_count",
)


class LayerDesc(Structure):
    _fields_ = [("Wp", c_void_p), ("ldw_w", c_int64), ("K", c_int64), ("N", c_int64), ("thr", c_void_p),
                ("flip", c_void_p), ("gamma", c_void_p), ("beta", c_void_p), ("mean", c_void_p), ("var", c_void_p),
                ("eps", c_double), ("W8", c_void_p), ("W4", c_void_p)]


class MlpDesc(Structure):
    _fields_ = [("n_layers", c_int32), ("layers", POINTER(LayerDesc))]


class ConvLayerDesc(Structure):
    _fields_ = [("Wp", c_void_p), ("C_in", c_int64), ("C_out", c_int64), ("pool", c_int32), ("thr", c_void_p),
                ("flip", c_void_p), ("W8", c_void_p), ("W4", c_void_p)]


class ConvNetDesc(Structure):
    _fields_ = [("n_layers", c_int32), ("layers", POINTER(ConvLayerDesc))]


class BnnError(RuntimeError):
    def __init__(self, status: int, what: str, cuda_error: int = 0):
        self.status = status
        self.cuda_error = cuda_error
        msg = f"{what} failed: {status} ({_status_string(status)})"
        if cuda_error:
            msg += f", cudaError {cuda_error}"
        super().__init__(msg)


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded C library.  Raises if it has not been built (python -m paper_1602_02830_b200.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_1602_02830_b200.build` "
                               "(there is no CPU or PyTorch fallback)")
        L = ctypes.CDLL(LIB_PATH)
        i64, vp = c_int64, c_void_p
        L.bnn_create.argtypes = [POINTER(vp), c_int, vp]
        L.bnn_destroy.argtypes = [vp]
        L.bnn_status_string.argtypes = [c_int]
        L.bnn_status_string.restype = ctypes.c_char_p
        L.bnn_last_cuda_error.argtypes = [vp]
        L.bnn_set_workspace.argtypes = [vp, vp, c_size_t]
        L.bnn_set_popc_variant.argtypes = [vp, c_int]
        L.bnn_set_engine.argtypes = [vp, c_int]
        L.bnn_set_tile_rows.argtypes = [vp, c_int]
        L.bnn_set_pair_mode.argtypes = [vp, c_int]
        L.bnn_set_operand_bits.argtypes = [vp, c_int]
        L.bnn_set_wait_limit_ns.argtypes = [vp, ctypes.c_uint64]
        L.bnn_debug_drop_loads.argtypes = [vp, c_int]
        L.bnn_debug_ring_position.argtypes = [ctypes.c_uint32] * 3 + [vp] * 8
        L.bnn_debug_ring_position.restype = c_int
        L.bnn_set_conv_form.argtypes = [vp, c_int]
        L.bnn_measure_pipe_rates.argtypes = [vp, vp, c_size_t, POINTER(c_double), POINTER(c_double), POINTER(c_double)]
        L.bnn_last_tensor_kernel.argtypes = [vp]
        L.bnn_last_tensor_kernel.restype = ctypes.c_char_p
        L.bnn_last_tensor_kernel_clock.argtypes = [vp, POINTER(c_double), POINTER(c_double)]
        L.bnn_set_conv_filter_repetition.argtypes = [vp, c_int]
        L.bnn_filter_repetition_workspace_bytes.argtypes = [i64, i64]
        L.bnn_filter_repetition_workspace_bytes.restype = c_size_t
        L.bnn_filter_repetition_count.argtypes = [vp, vp, i64, i64, POINTER(c_int64)]
        L.bnn_expanded_ld_f4.argtypes = [i64]
        L.bnn_expanded_ld_f4.restype = i64
        L.bnn_expanded_bytes_f4.argtypes = [i64, i64]
        L.bnn_expanded_bytes_f4.restype = c_size_t
        L.bnn_expand_signs_f4.argtypes = [vp, vp, i64, i64, i64, vp]
        L.bnn_binary_dense_expanded.argtypes = [vp, vp, i64, vp, i64, ctypes.c_int, vp, vp, vp, i64, vp, i64, i64, i64, i64]
        L.bnn_expanded_ld.argtypes = [i64]
        L.bnn_expanded_ld.restype = i64
        L.bnn_expanded_bytes.argtypes = [i64, i64]
        L.bnn_expanded_bytes.restype = c_size_t
        L.bnn_expand_signs.argtypes = [vp, vp, i64, i64, i64, vp]
        L.bnn_baseline_gemm_f32.argtypes = [vp, vp, vp, vp, i64, i64, i64]
        L.bnn_convnet_workspace_bytes.argtypes = [POINTER(ConvNetDesc), i64, i64, i64]
        L.bnn_convnet_workspace_bytes.restype = c_size_t
        L.bnn_convnet_forward.argtypes = [vp, POINTER(ConvNetDesc), vp, i64, i64, i64, vp, POINTER(vp)]
        L.bnn_gemm_workspace_bytes.argtypes = [i64, i64, i64]
        L.bnn_gemm_workspace_bytes.restype = c_size_t
        L.bnn_device_status.argtypes = [vp]
        L.bnn_conv_workspace_bytes.argtypes = [i64, i64, i64, i64, i64, c_int]
        L.bnn_conv_workspace_bytes.restype = c_size_t
        L.bnn_pack_signs.argtypes = [vp, vp, c_int, i64, i64, i64, c_int, c_int, vp, i64]
        L.bnn_xnor_gemm.argtypes = [vp, vp, i64, vp, i64, vp, i64, i64, i64, i64]
        L.bnn_binary_dense.argtypes = [vp, vp, i64, vp, i64, vp, vp, vp, i64, i64, i64, i64]
        L.bnn_first_layer_bitplanes.argtypes = [vp, vp, i64, vp, i64, vp, vp, vp, i64, vp, i64, i64, i64, i64]
        L.bnn_binary_conv2d.argtypes = [vp, vp, vp, i64, i64, i64, i64, vp, i64, c_int, vp, vp, vp, vp]
        L.bnn_mlp_workspace_bytes.argtypes = [POINTER(MlpDesc), i64, c_int]
        L.bnn_mlp_workspace_bytes.restype = c_size_t
        L.bnn_mlp_forward.argtypes = [vp, POINTER(MlpDesc), vp, i64, i64, vp, i64, POINTER(vp)]
        L.bnn_mlp_forward_host.argtypes = [vp, POINTER(MlpDesc), vp, i64, i64, vp, i64]
        L.bnn_fold_batchnorm.argtypes = [vp, vp, vp, vp, c_double, i64, i64, vp, vp]
        L.bnn_mlp_noalloc_max_bytes.argtypes = []
        L.bnn_mlp_noalloc_max_bytes.restype = c_size_t
        L.bnn_mlp_forward_noalloc.argtypes = [vp, POINTER(MlpDesc), vp, i64, i64, vp, i64]
        _lib = L
    return _lib


def _status_string(status: int) -> str:
    try:
        return lib().bnn_status_string(status).decode()
    except Exception:  # pragma: no cover
        return "?"


def _ptr(t):
    return None if t is None else c_void_p(t.data_ptr())


def words(k: int) -> int:
    return (k + 31) // 32


def packed_ld(k: int) -> int:
    """Smallest legal leading dimension (in 32-bit words) of a packed matrix with k bits per row."""
    return ((k + 127) // 128) * 4


class Context:
    """bnn_ctx bound to a device and to torch's current stream on it (or to an explicit stream)."""

    def __init__(self, device: int = 0, stream: "torch.cuda.Stream | None" = None):
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required; the library has no CPU path")
        self.device = device
        self.stream = stream if stream is not None else torch.cuda.current_stream(device)
        h = c_void_p()
        st = lib().bnn_create(ctypes.byref(h), device, c_void_p(self.stream.cuda_stream))
        if st:
            raise BnnError(st, "bnn_create")
        self._h = h
        self._ws = None
        self._destroy = lib().bnn_destroy      # kept here: module globals may be gone when __del__ runs at interpreter exit

    def close(self):
        h, destroy = getattr(self, "_h", None), getattr(self, "_destroy", None)
        if h and destroy is not None:
            destroy(h)
        self._h = None

    __del__ = close

    def _ck(self, st: int, what: str):
        if st:
            raise BnnError(st, what, lib().bnn_last_cuda_error(self._h))

    def empty(self, *shape, dtype=torch.int32):
        return torch.empty(*shape, dtype=dtype, device=f"cuda:{self.device}")

    # -- plumbing ------------------------------------------------------------------------------
    def set_workspace(self, ws: "torch.Tensor | None"):
        self._ws = ws
        if ws is None:
            self._ck(lib().bnn_set_workspace(self._h, None, 0), "bnn_set_workspace")
        else:
            self._ck(lib().bnn_set_workspace(self._h, _ptr(ws), ws.numel() * ws.element_size()), "bnn_set_workspace")

    def expand_signs(self, packed, rows: int, K: int):
        """bnn_expand_signs: packed rows x K -> int8 tensor [rows, bnn_expanded_ld(K)] of +1 / -1 (0 beyond K)."""
        ld = int(lib().bnn_expanded_ld(K))
        dst = self.empty(rows, ld, dtype=torch.int8)
        self._ck(lib().bnn_expand_signs(self._h, _ptr(packed), packed.stride(0), rows, K, _ptr(dst)), "bnn_expand_signs")
        return dst

    def baseline_gemm_f32(self, A, B, C=None):
        """bnn_baseline_gemm_f32: the paper's unoptimized float32 comparison kernel (context only)."""
        M, K = A.shape
        N = B.shape[1]
        if C is None:
            C = self.empty(M, N, dtype=torch.float32)
        self._ck(lib().bnn_baseline_gemm_f32(self._h, _ptr(A), _ptr(B), _ptr(C), M, N, K), "bnn_baseline_gemm_f32")
        return C

    def expand_signs_f4(self, packed, rows: int, K: int):
        """bnn_expand_signs_f4: packed rows x K -> uint8 tensor [rows, bnn_expanded_ld_f4(K)] of e2m1 nibbles."""
        ld = int(lib().bnn_expanded_ld_f4(K))
        dst = self.empty(rows, ld, dtype=torch.uint8)
        self._ck(lib().bnn_expand_signs_f4(self._h, _ptr(packed), packed.stride(0), rows, K, _ptr(dst)), "bnn_expand_signs_f4")
        return dst

    def binary_dense_expanded(self, A_exp, W_exp, bits: int, thr, flip, M, N, K, want_bits=True, want_exp=False):
        """bnn_binary_dense_expanded: operands as written by expand_signs (bits 8) or expand_signs_f4 (bits 4).
        Returns (packed signs or None, signs in the next layer's operand format or None)."""
        out = self.empty(M, packed_ld(N)) if want_bits else None
        out_exp = None
        if want_exp:
            ld = int(lib().bnn_expanded_ld_f4(N) if bits == 4 else lib().bnn_expanded_ld(N))
            out_exp = self.empty(M, ld, dtype=torch.uint8 if bits == 4 else torch.int8)
        self._ck(lib().bnn_binary_dense_expanded(self._h, _ptr(A_exp), A_exp.stride(0) * A_exp.element_size(), _ptr(W_exp),
                                                 W_exp.stride(0) * W_exp.element_size(), bits, _ptr(thr), _ptr(flip), _ptr(out),
                                                 packed_ld(N), _ptr(out_exp), out_exp.stride(0) if out_exp is not None else 0,
                                                 M, N, K), "bnn_binary_dense_expanded")
        return out, out_exp

    def set_operand_bits(self, bits: int):
        self._ck(lib().bnn_set_operand_bits(self._h, bits), "bnn_set_operand_bits")

    def set_wait_limit_ns(self, ns: int):
        self._ck(lib().bnn_set_wait_limit_ns(self._h, ns), "bnn_set_wait_limit_ns")

    def debug_drop_loads(self, on: bool):
        self._ck(lib().bnn_debug_drop_loads(self._h, int(on)), "bnn_debug_drop_loads")

    def measure_pipe_rates(self):
        """bnn_measure_pipe_rates -> dict of thread-level results per clock and SM (popc, lop3, xor+popc+add)."""
        sms = torch.cuda.get_device_properties(self.device).multi_processor_count
        scratch = self.empty(sms * 4104, dtype=torch.uint8)
        a, b, c = c_double(), c_double(), c_double()
        self._ck(lib().bnn_measure_pipe_rates(self._h, _ptr(scratch), scratch.numel(), ctypes.byref(a), ctypes.byref(b),
                                              ctypes.byref(c)), "bnn_measure_pipe_rates")
        return {"popc": a.value, "lop3": b.value, "xor_popc_add": c.value}

    def last_tensor_kernel(self) -> str:
        return lib().bnn_last_tensor_kernel(self._h).decode()

    def last_tensor_kernel_clock(self):
        """(SM MHz inside the tensor-core kernel that ran last, microseconds its first CTA lived)."""
        mhz, us = c_double(), c_double()
        self._ck(lib().bnn_last_tensor_kernel_clock(self._h, ctypes.byref(mhz), ctypes.byref(us)), "bnn_last_tensor_kernel_clock")
        return mhz.value, us.value

    def set_conv_filter_repetition(self, on: bool):
        self._ck(lib().bnn_set_conv_filter_repetition(self._h, int(on)), "bnn_set_conv_filter_repetition")

    def filter_repetition_workspace_bytes(self, C_in: int, C_out: int) -> int:
        return int(lib().bnn_filter_repetition_workspace_bytes(C_in, C_out))

    def filter_repetition_count(self, Wp, C_in: int, C_out: int) -> int:
        """bnn_filter_repetition_count: distinct 2-D filters (up to sign) summed over the input channels."""
        out = c_int64()
        self._ck(lib().bnn_filter_repetition_count(self._h, _ptr(Wp), C_in, C_out, ctypes.byref(out)), "bnn_filter_repetition_count")
        return int(out.value)

    def set_conv_form(self, form: int):
        self._ck(lib().bnn_set_conv_form(self._h, form), "bnn_set_conv_form")

    def set_pair_mode(self, mode: int):
        self._ck(lib().bnn_set_pair_mode(self._h, mode), "bnn_set_pair_mode")

    def set_tile_rows(self, rows: int):
        self._ck(lib().bnn_set_tile_rows(self._h, rows), "bnn_set_tile_rows")

    def set_engine(self, engine: int):
        self._ck(lib().bnn_set_engine(self._h, engine), "bnn_set_engine")

    def gemm_workspace_bytes(self, M: int, N: int, K: int) -> int:
        return int(lib().bnn_gemm_workspace_bytes(M, N, K))

    def conv_workspace_bytes(self, B, H, W, C_in, C_out, pool) -> int:
        return int(lib().bnn_conv_workspace_bytes(B, H, W, C_in, C_out, int(pool)))

    def device_status(self):
        """Synchronises the stream; raises if a kernel reported that one of its bounded waits gave up."""
        self._ck(lib().bnn_device_status(self._h), "bnn_device_status")

    def set_popc_variant(self, variant: int):
        self._ck(lib().bnn_set_popc_variant(self._h, variant), "bnn_set_popc_variant")

    # -- calls, one per C entry point ----------------------------------------------------------------
    def pack_signs(self, src: torch.Tensor, pack_along: int = 0, word_bits: int = 32, dst=None, dst_ld_w=None):
        """src: 2-D tensor (float32 / float16 / int8), row-major.  Returns the packed int32 tensor."""
        dtype = {torch.float32: BNN_F32, torch.float16: BNN_F16, torch.int8: BNN_I8}[src.dtype]
        rows, cols = src.shape
        assert src.stride(1) == 1 or cols <= 1
        out_rows, out_k = (rows, cols) if pack_along == 0 else (cols, rows)
        ld = dst_ld_w if dst_ld_w is not None else packed_ld(out_k)
        if dst is None:
            dst = self.empty(out_rows, ld)
        self._ck(lib().bnn_pack_signs(self._h, _ptr(src), dtype, rows, cols, src.stride(0) if rows > 1 else max(cols, 1),
                                      pack_along, word_bits, _ptr(dst), ld), "bnn_pack_signs")
        return dst

    def xnor_gemm(self, Ap, Bp, M, N, K, C=None, lda_w=None, ldb_w=None, ldc=None):
        if C is None:
            C = self.empty(M, N)
        self._ck(lib().bnn_xnor_gemm(self._h, _ptr(Ap), lda_w if lda_w is not None else Ap.stride(0), _ptr(Bp),
                                     ldb_w if ldb_w is not None else Bp.stride(0), _ptr(C),
                                     ldc if ldc is not None else (C.stride(0) if C.dim() == 2 and M > 1 else max(N, 1)),
                                     M, N, K), "bnn_xnor_gemm")
        return C

    def binary_dense(self, Ap, Wp, thr, flip, M, N, K, out=None, ldo_w=None):
        ld = ldo_w if ldo_w is not None else packed_ld(N)
        if out is None:
            out = self.empty(M, ld)
        self._ck(lib().bnn_binary_dense(self._h, _ptr(Ap), Ap.stride(0), _ptr(Wp), Wp.stride(0), _ptr(thr), _ptr(flip),
                                        _ptr(out), ld, M, N, K), "bnn_binary_dense")
        return out

    def first_layer_bitplanes(self, X, Wp, M, N, K, thr=None, flip=None, want_bits=True, want_sums=False):
        ld = packed_ld(N)
        bits = self.empty(M, ld) if want_bits else None
        sums = self.empty(M, N) if want_sums else None
        self._ck(lib().bnn_first_layer_bitplanes(self._h, _ptr(X), X.stride(0) if M > 1 else max(K, 1), _ptr(Wp),
                                                 Wp.stride(0), _ptr(thr), _ptr(flip), _ptr(bits), ld, _ptr(sums), N,
                                                 M, N, K), "bnn_first_layer_bitplanes")
        return bits, sums

    def binary_conv2d(self, act, B, H, W, C_in, Wp, C_out, pool=False, thr=None, flip=None, want_bits=True,
                      want_sums=False):
        """act: packed int32 [B,H,W,C_in/32] or uint8 [B,H,W,C_in] (first layer)."""
        Ho, Wo = (H // 2, W // 2) if pool else (H, W)
        bits = self.empty(B, Ho, Wo, words(C_out)) if want_bits else None
        sums = self.empty(B, Ho, Wo, C_out) if want_sums else None
        is_u8 = act.dtype == torch.uint8
        self._ck(lib().bnn_binary_conv2d(self._h, None if is_u8 else _ptr(act), _ptr(act) if is_u8 else None, B, H, W,
                                         C_in, _ptr(Wp), C_out, int(pool), _ptr(thr), _ptr(flip), _ptr(bits),
                                         _ptr(sums)), "bnn_binary_conv2d")
        return bits, sums

    def make_mlp_desc(self, layers):
        """layers: list of dicts with Wp, K, N and thr/flip (hidden) or gamma/beta/mean/var/eps (last).
        Returns (MlpDesc, keep-alive tuple)."""
        arr = (LayerDesc * len(layers))()
        for d, L in zip(arr, layers):
            d.Wp = L["Wp"].data_ptr()
            d.ldw_w = L["Wp"].stride(0)
            d.K, d.N = L["K"], L["N"]
            for name in ("thr", "flip", "gamma", "beta", "mean", "var", "W8", "W4"):
                t = L.get(name)
                setattr(d, name, t.data_ptr() if t is not None else None)
            d.eps = float(L.get("eps", 0.0))
        desc = MlpDesc(len(layers), arr)
        return desc, (arr, layers)

    def make_convnet_desc(self, layers):
        """layers: list of dicts with Wp, Cin, Cout, pool, thr, flip and optionally W8, W4.  Returns (ConvNetDesc, keep-alive)."""
        arr = (ConvLayerDesc * len(layers))()
        for d, L in zip(arr, layers):
            d.Wp = L["Wp"].data_ptr()
            d.C_in, d.C_out, d.pool = L["Cin"], L["Cout"], int(L["pool"])
            d.thr = L["thr"].data_ptr()
            d.flip = L["flip"].data_ptr() if L.get("flip") is not None else None
            d.W8 = L["W8"].data_ptr() if L.get("W8") is not None else None
            d.W4 = L["W4"].data_ptr() if L.get("W4") is not None else None
        return ConvNetDesc(len(layers), arr), (arr, layers)

    def convnet_workspace_bytes(self, desc, B: int, H: int, W: int) -> int:
        return int(lib().bnn_convnet_workspace_bytes(ctypes.byref(desc), B, H, W))

    def convnet_forward(self, desc, X, B: int, H: int, W: int, out_bits, layer_out=None):
        hp = None
        if layer_out is not None:
            hp = (c_void_p * desc.n_layers)(*[t.data_ptr() if t is not None else None for t in layer_out])
        self._ck(lib().bnn_convnet_forward(self._h, ctypes.byref(desc), _ptr(X), B, H, W, _ptr(out_bits), hp),
                 "bnn_convnet_forward")
        return out_bits

    def mlp_workspace_bytes(self, desc, batch: int, host_io: bool = False) -> int:
        return int(lib().bnn_mlp_workspace_bytes(ctypes.byref(desc), batch, int(host_io)))

    def mlp_forward(self, desc, X, batch, scores=None, hidden_out=None):
        n_out = desc.layers[desc.n_layers - 1].N
        if scores is None:
            scores = self.empty(batch, n_out, dtype=torch.float32)
        hp = None
        if hidden_out is not None:
            hp = (c_void_p * (desc.n_layers - 1))(*[t.data_ptr() if t is not None else None for t in hidden_out])
        self._ck(lib().bnn_mlp_forward(self._h, ctypes.byref(desc), _ptr(X), X.stride(0) if batch > 1 else X.shape[-1],
                                       batch, _ptr(scores), n_out, hp), "bnn_mlp_forward")
        return scores

    def mlp_forward_noalloc(self, desc, X, batch, scores):
        """bnn_mlp_forward_noalloc: the caller passes the output too, so that nothing is allocated here either."""
        n_out = desc.layers[desc.n_layers - 1].N
        self._ck(lib().bnn_mlp_forward_noalloc(self._h, ctypes.byref(desc), _ptr(X),
                                               X.stride(0) if batch > 1 else X.shape[-1], batch, _ptr(scores), n_out),
                 "bnn_mlp_forward_noalloc")
        return scores

    def mlp_forward_host(self, desc, X_host, batch, scores_host):
        n_out = desc.layers[desc.n_layers - 1].N
        self._ck(lib().bnn_mlp_forward_host(self._h, ctypes.byref(desc), _ptr(X_host), X_host.stride(0), batch,
                                            _ptr(scores_host), n_out), "bnn_mlp_forward_host")
        return scores_host


def debug_ring_position(stage: int, slots: int, step: int = 1) -> dict:
    """bnn_debug_ring_position: host-only view of the operand-ring arithmetic of the tensor-engine kernels."""
    o = [ctypes.c_uint32() for _ in range(3)] + [ctypes.c_int32()] + [ctypes.c_uint32() for _ in range(4)]
    st = lib().bnn_debug_ring_position(stage, slots, step, *[ctypes.byref(x) for x in o])
    if st:
        raise BnnError(st, "bnn_debug_ring_position")
    keys = ("slot", "barrier", "parity", "reuses", "prev_barrier", "prev_parity", "next_barrier", "next_parity")
    return {k: int(v.value) for k, v in zip(keys, o)}


def fold_batchnorm(gamma, beta, mean, var, eps: float, x_max: int):
    """Host helper bnn_fold_batchnorm: float32 CPU tensors in, (thr int32[n], flip packed int32[ceil(n/32)]) out."""
    n = gamma.numel()
    g, b, m, v = (t.detach().to(torch.float32).contiguous().cpu() for t in (gamma, beta, mean, var))
    thr = torch.empty(n, dtype=torch.int32)
    flip = torch.zeros(words(n), dtype=torch.int32)
    st = lib().bnn_fold_batchnorm(_ptr(g), _ptr(b), _ptr(m), _ptr(v), float(eps), n, int(x_max), _ptr(thr), _ptr(flip))
    if st:
        raise BnnError(st, "bnn_fold_batchnorm")
    return thr, flip
