"""ctypes binding of the C ABI declared in include/ais.h (argument marshalling only)."""

from __future__ import annotations

import ctypes as C
import math
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libais_b200.so")
_lib = None

FLAG_EMPTY, FLAG_TOKEN_RANGE, FLAG_NONFINITE, FLAG_TIMEOUT = 1, 2, 4, 8
NUM_MOMENTS = 12


class AisError(RuntimeError):
    pass


class Shape(C.Structure):
    _fields_ = [("T", C.c_int64), ("d", C.c_int32), ("V", C.c_int32), ("P", C.c_int32), ("G", C.c_int32),
                ("fp8_block", C.c_int32), ("P_total", C.c_int32), ("w_layout", C.c_int32), ("ldh", C.c_int64), ("ldw", C.c_int64)]


class Params(C.Structure):
    _fields_ = [("C", C.c_float), ("delta", C.c_float), ("gamma", C.c_float), ("eps", C.c_float),
                ("beta_var", C.c_float), ("clip_eps", C.c_float), ("alpha_override", C.c_float),
                ("adv_std_norm", C.c_int32), ("vocab_chunk", C.c_int32), ("beta_kl", C.c_float),
                ("seq_level_weights", C.c_int32)]


class Diag(C.Structure):
    _fields_ = [(n, C.c_double) for n in
                ("n_valid", "mean_w", "cv2", "ess", "ess_ratio", "alpha_ess", "d_bar", "alpha_mis", "std_A", "std_Aw",
                 "delta_sigma", "alpha_var", "alpha_adaptive", "alpha", "loss", "kl_k1", "mean_abs_dp", "kl_ref")] + \
               [("status_flags", C.c_uint32), ("reserved", C.c_uint32)]

    def as_dict(self) -> dict:
        return {n: getattr(self, n) for n, _ in self._fields_ if n != "reserved"}


def lib_path() -> str:
    return _LIB_PATH


def lib() -> C.CDLL:
    """Loads the CUDA library; raises if it has not been built (python -m paper_2605_13907_b200.build)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise AisError(f"{_LIB_PATH} is missing: build it with `python paper_2605_13907_b200/build.py`; "
                           "there is no CPU fallback")
        L = C.CDLL(_LIB_PATH)
        vp, i64, sz = C.c_void_p, C.c_int64, C.c_size_t
        L.ais_version.restype = C.c_int
        L.ais_strerror.restype = C.c_char_p
        L.ais_strerror.argtypes = [C.c_int]
        L.ais_default_params.restype = None
        L.ais_default_params.argtypes = [C.POINTER(Params)]
        for f in (L.ais_workspace_bytes, L.ais_workspace_min_bytes):
            f.restype = sz
            f.argtypes = [C.POINTER(Shape), C.POINTER(Params)]
        L.ais_quantize_fp8.restype = C.c_int
        L.ais_quantize_fp8.argtypes = [vp, i64, i64, i64, C.c_int, vp, i64, vp, i64, vp]
        L.ais_quantize_fp8_cols.restype = C.c_int
        L.ais_quantize_fp8_cols.argtypes = [vp, i64, i64, i64, C.c_int, vp, i64, vp, i64, vp]
        L.ais_quantize_fp8_tensor.restype = C.c_int
        L.ais_quantize_fp8_tensor.argtypes = [vp, i64, i64, i64, vp, i64, vp, vp]
        L.ais_mx_scale_bytes.restype = sz
        L.ais_mx_scale_bytes.argtypes = [i64, i64]
        L.ais_quantize_mxfp8.restype = C.c_int
        L.ais_quantize_mxfp8.argtypes = [vp, i64, i64, i64, vp, i64, vp, vp]
        L.ais_quantize_mxfp4.restype = C.c_int
        L.ais_quantize_mxfp4.argtypes = [vp, i64, i64, i64, vp, i64, vp, vp]
        L.ais_logprob_fwd.restype = C.c_int
        L.ais_logprob_fwd.argtypes = [C.POINTER(Shape), C.POINTER(Params), vp, vp, vp, vp, i64, vp, vp, i64, vp, vp,
                                      vp, vp, vp, vp, vp, vp, sz, vp]
        L.ais_diagnostics.restype = C.c_int
        L.ais_diagnostics.argtypes = [C.POINTER(Shape), C.POINTER(Params), vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.ais_loss_bwd.restype = C.c_int
        L.ais_loss_bwd.argtypes = [C.POINTER(Shape), C.POINTER(Params)] + [vp] * 15 + [i64, C.c_int] + [vp, vp, sz, vp]
        L.ais_diag_moments.restype = C.c_int
        L.ais_diag_moments.argtypes = [C.POINTER(Shape), C.POINTER(Params)] + [vp] * 9 + [vp, sz, vp]
        L.ais_diag_finalize.restype = C.c_int
        L.ais_diag_finalize.argtypes = [C.POINTER(Shape), C.POINTER(Params)] + [vp] * 10
        L.ais_compact_index.restype = C.c_int
        L.ais_compact_index.argtypes = [vp, vp, C.c_int32, vp, vp, vp, vp]
        L.ais_gather_rows.restype = C.c_int
        L.ais_gather_rows.argtypes = [vp, i64, vp, i64, i64, vp, i64, vp]
        L.ais_scatter_rows.restype = C.c_int
        L.ais_scatter_rows.argtypes = [vp, i64, vp, i64, i64, vp, i64, i64, vp]
        L.ais_gather_words.restype = C.c_int
        L.ais_gather_words.argtypes = [vp, vp, i64, vp, vp]
        L.ais_scatter_words.restype = C.c_int
        L.ais_scatter_words.argtypes = [vp, vp, i64, vp, i64, C.c_uint32, vp]
        L.ais_set_wait_cycles.restype = C.c_int
        L.ais_set_wait_cycles.argtypes = [i64]
        L.ais_logprob_train_static.restype = C.c_int
        L.ais_logprob_train_static.argtypes = [C.POINTER(Shape)] + [vp] * 8
        _lib = L
    return _lib


def set_wait_cycles(cycles: int) -> None:
    """Bound of the kernels' device-side waits in SM clock ticks; 0 restores the default (about two seconds)."""
    _check(lib().ais_set_wait_cycles(int(cycles)), "ais_set_wait_cycles")


def _check(status: int, what: str) -> None:
    if status != 0:
        raise AisError(f"{what}: {lib().ais_strerror(status).decode()} ({status})")


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(t: torch.Tensor):
    return C.c_void_p(torch.cuda.current_stream(t.device).cuda_stream)


def default_params(**overrides) -> Params:
    p = Params()
    lib().ais_default_params(C.byref(p))
    for k, v in overrides.items():
        if k == "alpha_override" and v is None:
            v = math.nan
        setattr(p, k, v)
    return p


W_VD, W_DV = 0, 1       # ais_shape.w_layout: W stored [V, d] (a torch lm_head.weight) or [d, V]


def make_shape(T: int, d: int, V: int, P: int, G: int, fp8_block: int, ldh: int | None = None, ldw: int | None = None,
               P_total: int = 0, w_layout: int = W_VD) -> Shape:
    return Shape(T=T, d=d, V=V, P=P, G=G, fp8_block=fp8_block, P_total=P_total, w_layout=w_layout, ldh=ldh or d,
                 ldw=ldw or (V if w_layout == W_DV else d))


def workspace_bytes(shape: Shape, params: Params) -> int:
    return int(lib().ais_workspace_bytes(C.byref(shape), C.byref(params)))


def workspace_min_bytes(shape: Shape, params: Params) -> int:
    return int(lib().ais_workspace_min_bytes(C.byref(shape), C.byref(params)))


def _require_cuda(*tensors):
    for t in tensors:
        if t is not None and not t.is_cuda:
            raise AisError("all tensors must live on a CUDA device; this library has no CPU path")


FP8_MX32 = -32          # fp8_block value: microscaling FP8 (E8M0 scale per 32 elements, hardware block-scaled MMA)
FP4_MX32 = -4           # fp8_block value: microscaling FP4 (E2M1 elements, two per byte)


def mx_scale_bytes(rows: int, cols: int) -> int:
    return int(lib().ais_mx_scale_bytes(rows, cols))


def quantize_fp8(x: torch.Tensor, block: int, codes: torch.Tensor | None = None, scales: torch.Tensor | None = None):
    """x [rows, cols] bf16 -> (codes [rows, cols] uint8, scales [cols/block, lds] float32, block-major);
    block = 0: one scale per tensor; block = FP8_MX32: packed E8M0 scale bytes (see include/ais.h)."""
    _require_cuda(x, codes, scales)
    rows, cols = x.shape
    if block == FP4_MX32:                            # 4-bit elements, two per byte, packed scale bytes
        if codes is None:
            codes = torch.empty(rows, cols // 2, dtype=torch.uint8, device=x.device)
        if scales is None:
            scales = torch.empty(mx_scale_bytes(rows, cols), dtype=torch.uint8, device=x.device)
        _check(lib().ais_quantize_mxfp4(_ptr(x), rows, cols, x.stride(0), _ptr(codes), codes.stride(0), _ptr(scales),
                                        _stream(x)), "ais_quantize_mxfp4")
        return codes, scales
    if codes is None:
        codes = torch.empty(rows, cols, dtype=torch.uint8, device=x.device)
    if block == FP8_MX32:                            # power-of-two scale per 32 elements, packed scale bytes
        if scales is None:
            scales = torch.empty(mx_scale_bytes(rows, cols), dtype=torch.uint8, device=x.device)
        _check(lib().ais_quantize_mxfp8(_ptr(x), rows, cols, x.stride(0), _ptr(codes), codes.stride(0), _ptr(scales),
                                        _stream(x)), "ais_quantize_mxfp8")
        return codes, scales
    if block == 0:                                   # one scale per tensor; scales holds it in its first element
        if scales is None:
            scales = torch.empty(1, 4, dtype=torch.float32, device=x.device)
        _check(lib().ais_quantize_fp8_tensor(_ptr(x), rows, cols, x.stride(0), _ptr(codes), codes.stride(0), _ptr(scales),
                                             _stream(x)), "ais_quantize_fp8_tensor")
        return codes, scales
    if scales is None:
        lds = (rows + 3) // 4 * 4
        scales = torch.empty(cols // block, max(lds, 4), dtype=torch.float32, device=x.device)
    _check(lib().ais_quantize_fp8(_ptr(x), rows, cols, x.stride(0), block, _ptr(codes), codes.stride(0), _ptr(scales),
                                  scales.stride(0), _stream(x)), "ais_quantize_fp8")
    return codes, scales


def quantize_fp8_cols(x: torch.Tensor, block: int, codes: torch.Tensor | None = None, scales: torch.Tensor | None = None):
    """x [K, N] bf16 with the blocks running down the columns (an LM head stored [d, V]) ->
    (codes [N, K] uint8, transposed; scales [K/block, lds] float32, block-major)."""
    _require_cuda(x, codes, scales)
    K, N = x.shape
    if codes is None:
        codes = torch.empty(N, K, dtype=torch.uint8, device=x.device)
    if scales is None:
        scales = torch.empty(K // block, max((N + 3) // 4 * 4, 4), dtype=torch.float32, device=x.device)
    _check(lib().ais_quantize_fp8_cols(_ptr(x), K, N, x.stride(0), block, _ptr(codes), codes.stride(0), _ptr(scales),
                                       scales.stride(0), _stream(x)), "ais_quantize_fp8_cols")
    return codes, scales


def logprob_fwd(shape: Shape, params: Params, H, W, qH, sH, qW, sW, tokens, mask, lp_train, lse_train, lp_roll, lse_roll,
                dev_status, workspace):
    _require_cuda(H, W, qH, sH, qW, sW, tokens, mask, lp_train, lse_train, lp_roll, lse_roll, dev_status, workspace)
    _check(lib().ais_logprob_fwd(C.byref(shape), C.byref(params), _ptr(H), _ptr(W), _ptr(qH), _ptr(sH),
                                 sH.stride(0) if sH is not None and sH.dim() == 2 else 0, _ptr(qW), _ptr(sW),
                                 sW.stride(0) if sW is not None and sW.dim() == 2 else 0, _ptr(tokens), _ptr(mask), _ptr(lp_train),
                                 _ptr(lse_train), _ptr(lp_roll), _ptr(lse_roll), _ptr(dev_status), _ptr(workspace),
                                 workspace.numel() * workspace.element_size(), _stream(workspace)), "ais_logprob_fwd")


def diagnostics(shape: Shape, params: Params, lp_train, lp_roll, mask, seq_offsets, rewards, adv, n_valid_seq, rho, w_tilde,
                diag, workspace):
    _require_cuda(lp_train, lp_roll, mask, seq_offsets, rewards, adv, n_valid_seq, rho, w_tilde, diag, workspace)
    _check(lib().ais_diagnostics(C.byref(shape), C.byref(params), _ptr(lp_train), _ptr(lp_roll), _ptr(mask), _ptr(seq_offsets),
                                 _ptr(rewards), _ptr(adv), _ptr(n_valid_seq), _ptr(rho), _ptr(w_tilde), _ptr(diag),
                                 _ptr(workspace), workspace.numel() * workspace.element_size(), _stream(workspace)),
           "ais_diagnostics")


def diag_moments(shape: Shape, params: Params, lp_train, lp_roll, mask, seq_offsets, rewards, adv, n_valid_seq, moments, workspace,
                 seq_logw=None):
    _require_cuda(lp_train, lp_roll, mask, seq_offsets, rewards, adv, n_valid_seq, moments, workspace, seq_logw)
    _check(lib().ais_diag_moments(C.byref(shape), C.byref(params), _ptr(lp_train), _ptr(lp_roll), _ptr(mask), _ptr(seq_offsets),
                                  _ptr(rewards), _ptr(adv), _ptr(n_valid_seq), _ptr(moments), _ptr(seq_logw), _ptr(workspace),
                                  workspace.numel() * workspace.element_size(), _stream(workspace)), "ais_diag_moments")


def diag_finalize(shape: Shape, params: Params, moments, lp_train, lp_roll, mask, rho, w_tilde, diag, seq_offsets=None,
                  seq_logw=None):
    _require_cuda(moments, lp_train, lp_roll, mask, rho, w_tilde, diag, seq_offsets, seq_logw)
    _check(lib().ais_diag_finalize(C.byref(shape), C.byref(params), _ptr(moments), _ptr(lp_train), _ptr(lp_roll), _ptr(mask),
                                   _ptr(rho), _ptr(w_tilde), _ptr(diag), _ptr(seq_offsets), _ptr(seq_logw), _stream(moments)),
           "ais_diag_finalize")


def loss_bwd(shape: Shape, params: Params, H, W, tokens, mask, seq_offsets, lse_train, lp_train, lp_old, adv, w_tilde, dH, loss,
             diag, dev_status, workspace, lp_ref=None, dW=None, dw_accumulate: bool = False):
    _require_cuda(H, W, tokens, mask, seq_offsets, lse_train, lp_train, lp_old, lp_ref, adv, w_tilde, dH, loss, diag, dev_status,
                  workspace, dW)
    _check(lib().ais_loss_bwd(C.byref(shape), C.byref(params), _ptr(H), _ptr(W), _ptr(tokens), _ptr(mask), _ptr(seq_offsets),
                              _ptr(lse_train), _ptr(lp_train), _ptr(lp_old), _ptr(lp_ref), _ptr(adv), _ptr(w_tilde), _ptr(dH), _ptr(loss),
                              _ptr(diag), _ptr(dW), dW.stride(0) if dW is not None else 0, 1 if dw_accumulate else 0,
                              _ptr(dev_status), _ptr(workspace), workspace.numel() * workspace.element_size(),
                              _stream(workspace)), "ais_loss_bwd")


def logprob_train_static(shape: Shape, H, W, tokens, mask, lp_train, lse_train=None, dev_status=None):
    """Trainer log-probs with the library's built-in scratch: no workspace argument and no allocation, for
    callers that only own their inputs and outputs.  At most STATIC_MAX_ROWS rows; calls must not overlap."""
    _require_cuda(H, W, tokens, mask, lp_train, lse_train, dev_status)
    _check(lib().ais_logprob_train_static(C.byref(shape), _ptr(H), _ptr(W), _ptr(tokens), _ptr(mask), _ptr(lp_train),
                                          _ptr(lse_train), _ptr(dev_status), _stream(H)), "ais_logprob_train_static")


STATIC_MAX_ROWS = 16384


class RowCompaction:
    """Packing of the valid rows of a batch with a scattered mask, and the way back.

    n_packed is the number of valid rows; pass it when known (the usual case: the caller made the mask), otherwise it
    is read back from the device, which synchronises once.
    """

    def __init__(self, mask: torch.Tensor, seq_offsets: torch.Tensor, n_packed: int | None = None):
        _require_cuda(mask, seq_offsets)
        self.T = mask.numel()
        S = seq_offsets.numel() - 1
        dev = mask.device
        self.n_valid_seq = torch.empty(S, dtype=torch.int32, device=dev)
        self.packed_offsets = torch.empty(S + 1, dtype=torch.int32, device=dev)
        self.row_index = torch.empty(max(self.T, 1), dtype=torch.int32, device=dev)
        _check(lib().ais_compact_index(_ptr(mask), _ptr(seq_offsets), S, _ptr(self.n_valid_seq), _ptr(self.packed_offsets),
                                       _ptr(self.row_index), _stream(mask)), "ais_compact_index")
        self.n = int(self.packed_offsets[-1].item()) if n_packed is None else int(n_packed)

    def gather_rows(self, src: torch.Tensor, dst: torch.Tensor | None = None) -> torch.Tensor:
        if dst is None:
            dst = torch.empty(max(self.n, 1), src.shape[1], dtype=src.dtype, device=src.device)
        es = src.element_size()
        _check(lib().ais_gather_rows(_ptr(src), src.stride(0) * es, _ptr(self.row_index), self.n, src.shape[1] * es, _ptr(dst),
                                     dst.stride(0) * es, _stream(src)), "ais_gather_rows")
        return dst

    def scatter_rows(self, src: torch.Tensor, dst: torch.Tensor) -> torch.Tensor:
        es = src.element_size()
        _check(lib().ais_scatter_rows(_ptr(src), src.stride(0) * es, _ptr(self.row_index), self.n, src.shape[1] * es, _ptr(dst),
                                      dst.stride(0) * es, dst.shape[0], _stream(src)), "ais_scatter_rows")
        return dst

    def gather(self, src: torch.Tensor) -> torch.Tensor:
        """1-D tensor of 32-bit elements (tokens, float vectors)."""
        dst = torch.empty(max(self.n, 1), dtype=src.dtype, device=src.device)
        _check(lib().ais_gather_words(_ptr(src), _ptr(self.row_index), self.n, _ptr(dst), _stream(src)), "ais_gather_words")
        return dst

    def scatter(self, src: torch.Tensor, fill: float = 0.0) -> torch.Tensor:
        import struct
        dst = torch.empty(self.T, dtype=src.dtype, device=src.device)
        bits = struct.unpack("<I", struct.pack("<f", fill))[0] if src.dtype == torch.float32 else int(fill) & 0xFFFFFFFF
        _check(lib().ais_scatter_words(_ptr(src), _ptr(self.row_index), self.n, _ptr(dst), self.T, bits, _stream(src)),
               "ais_scatter_words")
        return dst


def read_diag(diag_buf: torch.Tensor) -> dict:
    """Copies the device-side ais_diag back (synchronises the current stream)."""
    host = diag_buf.cpu().numpy().tobytes()
    return Diag.from_buffer_copy(host[:C.sizeof(Diag)]).as_dict()


class AisStep:
    """Buffers and call order of one pass of the whole path for a fixed shape.

    step() enqueues: quantise H (and W unless its codes are cached) -> trainer and rollout log-probs ->
    ratios / diagnostics / alpha / w_tilde -> loss and dH.  Nothing synchronises; results stay on the device.
    """

    def __init__(self, T: int, d: int, V: int, P: int, G: int, fp8_block: int, device="cuda", params: Params | None = None,
                 workspace_bytes_cap: int | None = None, want_grad: bool = True, group=None, P_total: int = 0,
                 ldh: int | None = None, ldw: int | None = None, w_layout: int = W_VD):
        self.device = torch.device(device)
        self.group = group                       # torch.distributed process group: alpha over all its ranks
        ldh = ldh or d                           # row strides of H / W; H's codes and dH use H's stride
        ldw = ldw or (V if w_layout == W_DV else d)
        self.shape = make_shape(T, d, V, P, G, fp8_block, ldh=ldh, ldw=ldw, P_total=P_total, w_layout=w_layout)
        self.w_layout = w_layout
        self.params = params or default_params()
        S = P * G
        dev = self.device
        nkb = d // fp8_block if fp8_block > 0 else 1
        ws = workspace_bytes(self.shape, self.params)
        if ws == 0:
            raise AisError("invalid shape or parameters")
        if workspace_bytes_cap is not None:
            # room for every row's backward scratch in one pass, limited by the cap, never below the minimum
            ws_min = workspace_min_bytes(self.shape, self.params)
            ld_u = (V + 63) // 64 * 64
            ws_all = ws_min + max(0, (T + 127) // 128 * 128 - 128) * ld_u * 2
            ws = max(ws_min, min(ws_all, workspace_bytes_cap))
        self.workspace = torch.empty(ws, dtype=torch.uint8, device=dev)
        if fp8_block == FP4_MX32:
            self.qH = torch.empty(max(T, 1), ldh // 2, dtype=torch.uint8, device=dev)[:, :d // 2]
            self.qW = torch.empty(V, ldw // 2, dtype=torch.uint8, device=dev)[:, :d // 2]
        else:
            self.qH = torch.empty(max(T, 1), ldh, dtype=torch.uint8, device=dev)[:, :d]
            # a [d, V] head is quantised into codes [V, d] of row stride d; a [V, d] head's codes share its stride
            self.qW = torch.empty(V, d if w_layout == W_DV else ldw, dtype=torch.uint8, device=dev)[:, :d]
        if fp8_block in (FP8_MX32, FP4_MX32):
            self.sH = torch.empty(mx_scale_bytes(T, d), dtype=torch.uint8, device=dev)
            self.sW = torch.empty(mx_scale_bytes(V, d), dtype=torch.uint8, device=dev)
        else:
            self.sH = torch.empty(nkb, max((T + 3) // 4 * 4, 4), dtype=torch.float32, device=dev)
            self.sW = torch.empty(nkb, (V + 3) // 4 * 4, dtype=torch.float32, device=dev)
        f32 = dict(dtype=torch.float32, device=dev)
        self.lp_train = torch.empty(max(T, 1), **f32)
        self.lse_train = torch.empty(max(T, 1), **f32)
        self.lp_roll = torch.empty(max(T, 1), **f32)
        self.lse_roll = torch.empty(max(T, 1), **f32)
        self.rho = torch.empty(max(T, 1), **f32)
        self.w_tilde = torch.empty(max(T, 1), **f32)
        self.adv = torch.empty(S, **f32)
        self.n_valid_seq = torch.empty(S, dtype=torch.int32, device=dev)
        self.loss = torch.zeros(1, **f32)
        self.diag = torch.zeros((C.sizeof(Diag) + 7) // 8, dtype=torch.float64, device=dev)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.moments = torch.zeros(NUM_MOMENTS, dtype=torch.float64, device=dev)
        self.seq_logw = torch.zeros(max(S, 1), **f32)        # sequence-level variant: log weight per sequence
        self.dH = torch.empty(max(T, 1), ldh, dtype=torch.bfloat16, device=dev)[:, :d] if want_grad else None
        self.w_quantized = False

    def quantize_weights(self, W: torch.Tensor) -> None:
        if self.w_layout == W_DV:
            quantize_fp8_cols(W, self.shape.fp8_block, self.qW, self.sW)
        else:
            quantize_fp8(W, self.shape.fp8_block, self.qW, self.sW)
        self.w_quantized = True

    def forward(self, H, W, tokens, mask, requantize_w: bool = True) -> None:
        if self.shape.T > 0:
            quantize_fp8(H, self.shape.fp8_block, self.qH, self.sH)
        if requantize_w or not self.w_quantized:
            self.quantize_weights(W)
        logprob_fwd(self.shape, self.params, H, W, self.qH, self.sH, self.qW, self.sW, tokens, mask, self.lp_train,
                    self.lse_train, self.lp_roll, self.lse_roll, self.status, self.workspace)

    def diagnose(self, mask, seq_offsets, rewards) -> None:
        if self.group is None:
            diagnostics(self.shape, self.params, self.lp_train, self.lp_roll, mask, seq_offsets, rewards, self.adv,
                        self.n_valid_seq, self.rho, self.w_tilde, self.diag, self.workspace)
            return
        # data parallel: this rank's masked sums, one all-reduce of 12 doubles, then alpha / w_tilde from the global sums
        from . import dist as _dist
        diag_moments(self.shape, self.params, self.lp_train, self.lp_roll, mask, seq_offsets, rewards, self.adv,
                     self.n_valid_seq, self.moments, self.workspace, seq_logw=self.seq_logw)
        _dist.allreduce_moments(self.moments, self.group)
        diag_finalize(self.shape, self.params, self.moments, self.lp_train, self.lp_roll, mask, self.rho, self.w_tilde, self.diag,
                      seq_offsets=seq_offsets, seq_logw=self.seq_logw)

    def backward(self, H, W, tokens, mask, seq_offsets, lp_old=None, lp_ref=None, dW=None, dw_accumulate: bool = False) -> None:
        loss_bwd(self.shape, self.params, H, W, tokens, mask, seq_offsets, self.lse_train, self.lp_train, lp_old, self.adv,
                 self.w_tilde, self.dH, self.loss, self.diag, self.status, self.workspace, lp_ref=lp_ref, dW=dW,
                 dw_accumulate=dw_accumulate)

    def step(self, H, W, tokens, mask, seq_offsets, rewards, lp_old=None, requantize_w: bool = True, lp_ref=None) -> None:
        self.forward(H, W, tokens, mask, requantize_w)
        self.diagnose(mask, seq_offsets, rewards)
        if self.dH is not None:
            self.backward(H, W, tokens, mask, seq_offsets, lp_old, lp_ref)

    def read_diag(self) -> dict:
        return read_diag(self.diag)
