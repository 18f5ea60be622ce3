"""ctypes binding of libfaar.so.  Argument marshalling only: every function
below has the name and the arguments of the C entry point it calls; tensors
are torch CUDA tensors whose `data_ptr()` is handed through.  There is no
fallback: if the library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
#: the library this process binds: libfaar.so next to this file, or the file FAAR_LIB names (the debug build)
LIB_PATH = os.environ.get("FAAR_LIB") or os.path.join(_HERE, "libfaar.so")

OK, ERR_INVALID_ARG, ERR_SHAPE, ERR_ALIGN, ERR_DTYPE, ERR_WORKSPACE, ERR_ARCH, ERR_CUDA, ERR_TIMEOUT = range(9)
BF16, F32 = 0, 1

_P, _I, _L, _F, _Z, _U = C.c_void_p, C.c_int, C.c_int64, C.c_float, C.c_size_t, C.c_uint

#: every exported function: (result type, argument types), as declared in include/faar.h
SIGNATURES = {
    "faar_create": (_I, [_P, _I, _P]),
    "faar_destroy": (_I, [_P]),
    "faar_set_stream": (_I, [_P, _P]),
    "faar_status_string": (C.c_char_p, [_I]),
    "faar_last_cuda_error": (_I, [_P]),
    "faar_tune_tile_n": (_I, [_P, _I]),
    "faar_tune_tail_split": (_I, [_P, _I]),
    "faar_last_tail_split": (_I, [_P, _P]),
    "faar_last_gemm_config": (_I, [_P, _P, _P]),
    "faar_workspace_size": (_I, [_P, _P]),
    "faar_workspace_init": (_I, [_P, _P, _Z]),
    "faar_check_status": (_I, [_P, _P, _P]),
    "faar_selftest_wait_timeout": (_I, [_P, _P, _Z, _U]),
    "faar_profile_begin": (_I, [_P]),
    "faar_profile_end": (_I, [_P, _P, _I, _P]),
    "faar_kernel_name": (C.c_char_p, [_I]),
    "faar_softquant_init": (_I, [_P, _P, _P, _F, _P, _P, _P, _P, _P, _Z]),
    "faar_softquant_eval": (_I, [_P, _P, _P, _P, _P, _P, _F, _P, _P, _P]),
    "faar_softquant_operand_f32": (_I, [_P, _P, _P, _P, _P, _P, _F, _P]),
    "faar_transpose_bf16": (_I, [_P, _I, _I, _P, _L, _P, _L]),
    "faar_act_fakequant": (_I, [_P, _I, _I, _P, _L, _F, _P, _L, _P, _P, _P, _P, _Z]),
    "faar_layer_ref": (_I, [_P, _P, _P, _P, _P, _P, _Z]),
    "faar_layer_fwd": (_I, [_P, _P, _P, _P, _P, _P, _P, _P, _P, _P, _P, _P, _P, _Z]),
    "faar_layer_dx": (_I, [_P, _P, _F, _P, _P, _P, _P, _P, _P, _P, _P, _Z]),
    "faar_layer_dx_operand": (_I, [_P, _P, _P, _P, _P, _P, _Z]),
    "faar_round_loss": (_I, [_P, _P, _L, _P, _P, _Z]),
    "faar_round_loss_static": (_I, [_P, _P, _L, _P]),
    "faar_round_loss_static_max_n": (_L, []),
    "faar_layer_bwd": (_I, [_P, _P, _P, _P, _P, _P, _P, _P, _P, _P, _P, _P, _P, _Z]),
    "faar_layer_bwd_rowmajor": (_I, [_P, _P, _P, _P, _P, _P, _P, _P, _P, _P, _P, _P, _P, _Z]),
    "faar_layer_step": (_I, [_P, _P, _P, _P, _P, _P, _P, _P, _P, _P, _P, _P, _P, _P, _Z]),
    "faar_layer_step_host": (_I, [_P, _P, _P, _P, _P, _P, _P, _P, _P, _P, _P, _P, _P, _P, _P, _P, _P, _P, _Z]),
    "faar_nvfp4_expand": (_I, [_P, _I, _I, _P, _P, _P, _L]),
    "faar_layer_step_host_nvfp4": (_I, [_P] * 19 + [_Z]),
    "faar_harden_pack": (_I, [_P, _P, _P, _P, _P, _P, _P, _P, _P, _P, _I]),
    "faar_align_loss_workspace_size": (_I, [_I, _I, _P]),
    "faar_align_loss": (_I, [_P, _I, _I, _I, _P, _P, _L, _P, _P, _L, _F, _F, _P, _P, _P, _P, _Z]),
    "faar_swizzle_scales": (_I, [_P, _I, _I, _P, _P, _Z]),
    "faar_silu_mul": (_I, [_P, _I, _I, _P, _L, _P, _L, _P, _L]),
    "faar_rmsnorm": (_I, [_P, _I, _I, _P, _L, _P, _F, _P, _L, _P]),
    "faar_rmsnorm_bwd": (_I, [_P, _I, _I, _P, _L, _P, _L, _P, _P, _P, _L, _P, _L]),
    "faar_add_rmsnorm": (_I, [_P, _I, _I, _P, _L, _P, _L, _P, _L, _P, _F, _P, _L, _P]),
    "faar_rmsnorm_bwd_sum": (_I, [_P, _I, _I, _P, _P, _P, _L, _P, _L, _P, _P, _P, _L, _P, _L]),
    "faar_rope": (_I, [_P, _I, _I, _I, _P, _L, _P, _F, _I, _P, _L]),
    "faar_silu_mul_bwd": (_I, [_P, _I, _I, _P, _L, _P, _L, _P, _L, _P, _L, _P, _L]),
    "faar_embedding": (_I, [_P, _I, _I, _I, _P, _L, _P, _P, _L]),
    "faar_add": (_I, [_P, _I, _I, _P, _L, _P, _L, _P, _L]),
    "faar_tune_attention": (_I, [_P, _I]),
    "faar_attention_status": (_I, [_P, _P]),
    "faar_tune_wide_tiles": (_I, [_P, _I]),
    "faar_attention_fwd": (_I, [_P, _I, _I, _I, _I, _I, _P, _L, _P, _P, _L, _P, _L, _P]),
    "faar_attention_bwd": (_I, [_P, _I, _I, _I, _I, _I, _P, _L, _P, _P, _L, _P, _P, _L, _P, _P, _P, _P, _P]),
    "faar_nvfp4_gemm": (_I, [_P, _I, _I, _I, _P, _P, _P, _P, _P, _P, _P, _L, _P, _Z]),
}
EXPORTS = list(SIGNATURES)


class HParams(C.Structure):
    _fields_ = [("beta", C.c_float), ("lambda_round", C.c_float), ("mse_scale", C.c_float), ("opt", C.c_int),
                ("lr", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float),
                ("step", C.c_int), ("act_scale", C.c_float), ("beta_next", C.c_float), ("wsoft_ready", C.c_int)]


class Shape(C.Structure):
    _fields_ = [("O", C.c_int), ("K", C.c_int), ("T", C.c_int), ("ldw", C.c_int64), ("ldx", C.c_int64),
                ("ldxt", C.c_int64), ("ldy", C.c_int64), ("w_dtype", C.c_int), ("yref_dtype", C.c_int),
                ("yref_transposed", C.c_int)]


class FaarError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


_lib = None


def lib() -> C.CDLL:
    """Loads libfaar.so (built in-tree by `paper_2603_22370_b200.build`)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(f"{LIB_PATH} is missing; run `python -m paper_2603_22370_b200.build`")
        l = C.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(l, name)
            fn.restype, fn.argtypes = res, args
        _lib = l
    return _lib


def status_string(status: int) -> str:
    return lib().faar_status_string(int(status)).decode()


def _p(t):
    if t is None:
        return C.c_void_p(0)
    if isinstance(t, int):
        return C.c_void_p(t)
    assert t.is_cuda, "device tensors only"
    return C.c_void_p(t.data_ptr())


def C_size(t) -> C.c_size_t:
    return C.c_size_t(t.numel())


def _check(status: int, where: str):
    if status != OK:
        raise FaarError(status, where)


def make_shape(O, K, T, ldw=None, ldx=None, ldxt=None, ldy=None, w_dtype=BF16, yref_dtype=BF16,
               yref_transposed=0) -> Shape:
    """yref_transposed: Y_ref (and the optional Y_q) are stored [O, ldy], ldy >= T rounded up to 16."""
    if ldy is None:
        ldy = (T + 15) // 16 * 16 if yref_transposed else O
    return Shape(O, K, T, ldw if ldw is not None else K, ldx if ldx is not None else K,
                 ldxt if ldxt is not None else (T + 7) // 8 * 8, ldy, w_dtype, yref_dtype, yref_transposed)


def make_hparams(beta=4.0, lambda_round=1.0, mse_scale=1.0, opt=1, lr=1e-2, beta1=0.9, beta2=0.999, eps=1e-8,
                 step=1, act_scale=0.0, beta_next=0.0, wsoft_ready=0) -> HParams:
    return HParams(beta, lambda_round, mse_scale, opt, lr, beta1, beta2, eps, step, act_scale, beta_next, wsoft_ready)


class Context:
    """Owns a faar_ctx bound to a device and a stream, plus (optionally) a workspace tensor."""

    def __init__(self, device: int = 0, stream: torch.cuda.Stream | None = None):
        self._h = C.c_void_p(0)
        self.device = device
        s = stream.cuda_stream if stream is not None else torch.cuda.current_stream(device).cuda_stream
        _check(lib().faar_create(C.byref(self._h), device, C.c_void_p(s)), "faar_create")
        self.ws = None

    def close(self):
        if self._h:
            lib().faar_destroy(self._h)
            self._h = C.c_void_p(0)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_stream(self, stream: torch.cuda.Stream):
        _check(lib().faar_set_stream(self._h, C.c_void_p(stream.cuda_stream)), "faar_set_stream")

    def last_cuda_error(self) -> int:
        return lib().faar_last_cuda_error(self._h)

    def workspace(self, shape: Shape) -> torch.Tensor:
        """Allocates (with torch) and initialises a workspace large enough for `shape`."""
        n = workspace_size(shape)
        if self.ws is None or self.ws.numel() < n:
            self.ws = torch.empty(n, dtype=torch.uint8, device=f"cuda:{self.device}")
            workspace_init(self, self.ws)
        return self.ws


def tune_tile_n(ctx: Context, bn: int):
    """Forces the GEMM tile width (multiple of 16 in [128, 256]); 0 restores the automatic choice."""
    _check(lib().faar_tune_tile_n(ctx._h, C.c_int(bn)), "faar_tune_tile_n")


def tune_tail_split(ctx: Context, columns: int):
    """Forces how many trailing tile columns are cut into half-width tiles (-1 = automatic, 0 = none)."""
    _check(lib().faar_tune_tail_split(ctx._h, C.c_int(columns)), "faar_tune_tail_split")


def last_tail_split(ctx: Context) -> int:
    n = C.c_int(0)
    _check(lib().faar_last_tail_split(ctx._h, C.byref(n)), "faar_last_tail_split")
    return n.value


def last_gemm_config(ctx: Context) -> tuple[int, int]:
    """(tile width, CTA pairs) of the most recent GEMM launch on this context."""
    bn, pairs = C.c_int(0), C.c_int(0)
    _check(lib().faar_last_gemm_config(ctx._h, C.byref(bn), C.byref(pairs)), "faar_last_gemm_config")
    return bn.value, pairs.value


def workspace_size(shape: Shape) -> int:
    n = C.c_size_t(0)
    _check(lib().faar_workspace_size(C.byref(shape), C.byref(n)), "faar_workspace_size")
    return n.value


def workspace_init(ctx: Context, ws: torch.Tensor):
    _check(lib().faar_workspace_init(ctx._h, _p(ws), C.c_size_t(ws.numel())), "faar_workspace_init")


def selftest_wait_timeout(ctx: Context, ws: torch.Tensor, limit_us: int = 1000):
    _check(lib().faar_selftest_wait_timeout(ctx._h, _p(ws), C.c_size_t(ws.numel()), C.c_uint(limit_us)),
           "faar_selftest_wait_timeout")


def check_status(ctx: Context, ws: torch.Tensor) -> int:
    d = C.c_uint32(0)
    st = lib().faar_check_status(ctx._h, _p(ws), C.byref(d))
    if st != OK:
        raise FaarError(st, f"faar_check_status (detail 0x{d.value:x})")
    return st


def softquant_init(ctx, shape, W, s_global_in, scales, s_global_out, code, V_init, ws):
    _check(lib().faar_softquant_init(ctx._h, C.byref(shape), _p(W), C.c_float(s_global_in), _p(scales),
                                     _p(s_global_out), _p(code), _p(V_init), _p(ws), C.c_size_t(ws.numel())),
           "faar_softquant_init")


def softquant_eval(ctx, shape, V, code, scales, s_global, beta, W_soft, h, W_soft_bf16=None):
    _check(lib().faar_softquant_eval(ctx._h, C.byref(shape), _p(V), _p(code), _p(scales), _p(s_global),
                                     C.c_float(beta), _p(W_soft), _p(h), _p(W_soft_bf16)), "faar_softquant_eval")


def softquant_operand_f32(ctx, shape, V, code, scales, s_global, beta, W_operand):
    _check(lib().faar_softquant_operand_f32(ctx._h, C.byref(shape), _p(V), _p(code), _p(scales), _p(s_global),
                                            C.c_float(beta), _p(W_operand)), "faar_softquant_operand_f32")


def act_fakequant(ctx, T, K, X, ldx, s_global_in, Xq_units, ldq, s_global_out, packed, scales, ws):
    _check(lib().faar_act_fakequant(ctx._h, T, K, _p(X), C.c_int64(ldx), C.c_float(s_global_in), _p(Xq_units),
                                    C.c_int64(ldq), _p(s_global_out), _p(packed), _p(scales), _p(ws),
                                    C.c_size_t(ws.numel())), "faar_act_fakequant")


def align_loss_workspace_size(T, vocab) -> int:
    n = C.c_size_t(0)
    _check(lib().faar_align_loss_workspace_size(T, vocab, C.byref(n)), "faar_align_loss_workspace_size")
    return n.value


def align_loss(ctx, T, vocab, hidden, Z_fp, Z_q, ldz, H_fp, H_q, ldh, tau, lambda_kl, dZ_q, dH_q, loss_out2, ws):
    _check(lib().faar_align_loss(ctx._h, T, vocab, hidden, _p(Z_fp), _p(Z_q), C.c_int64(ldz), _p(H_fp), _p(H_q),
                                 C.c_int64(ldh), C.c_float(tau), C.c_float(lambda_kl), _p(dZ_q), _p(dH_q), _p(loss_out2),
                                 _p(ws), C.c_size_t(ws.numel())), "faar_align_loss")


def swizzle_scales(ctx, rows, cols, scales, scales_tiled):
    _check(lib().faar_swizzle_scales(ctx._h, rows, cols, _p(scales), _p(scales_tiled), C.c_size_t(scales_tiled.numel())),
           "faar_swizzle_scales")


def silu_mul(ctx, rows, cols, gate, ldg, up, ldu, out, ldo):
    _check(lib().faar_silu_mul(ctx._h, rows, cols, _p(gate), ldg, _p(up), ldu, _p(out), ldo), "faar_silu_mul")


def rmsnorm(ctx, rows, cols, x, ldx, g, eps, y, ldy, rstd=None):
    _check(lib().faar_rmsnorm(ctx._h, rows, cols, _p(x), ldx, _p(g), eps, _p(y), ldy, _p(rstd)), "faar_rmsnorm")


def rmsnorm_bwd(ctx, rows, cols, dy, lddy, x, ldx, g, rstd, add, ldadd, dx, lddx):
    _check(lib().faar_rmsnorm_bwd(ctx._h, rows, cols, _p(dy), lddy, _p(x), ldx, _p(g), _p(rstd), _p(add), ldadd, _p(dx), lddx),
           "faar_rmsnorm_bwd")


def add_rmsnorm(ctx, rows, cols, a, lda, b, ldb, total, lds, g, eps, y, ldy, rstd=None):
    _check(lib().faar_add_rmsnorm(ctx._h, rows, cols, _p(a), C.c_int64(lda), _p(b), C.c_int64(ldb), _p(total), C.c_int64(lds),
                                  _p(g), C.c_float(eps), _p(y), C.c_int64(ldy), _p(rstd)), "faar_add_rmsnorm")


def rmsnorm_bwd_sum(ctx, rows, cols, dy, dy2, dy3, lddy, x, ldx, g, rstd, add, ldadd, dx, lddx):
    _check(lib().faar_rmsnorm_bwd_sum(ctx._h, rows, cols, _p(dy), _p(dy2), _p(dy3), C.c_int64(lddy), _p(x), C.c_int64(ldx),
                                      _p(g), _p(rstd), _p(add), C.c_int64(ldadd), _p(dx), C.c_int64(lddx)),
           "faar_rmsnorm_bwd_sum")


def rope(ctx, rows, n_heads, head_dim, x, ldx, positions, theta, inverse, y, ldy):
    _check(lib().faar_rope(ctx._h, rows, n_heads, head_dim, _p(x), ldx, _p(positions), theta, int(inverse), _p(y), ldy),
           "faar_rope")


def silu_mul_bwd(ctx, rows, cols, dout, ldd, gate, ldg, up, ldu, dgate, lddg, dup, lddu):
    _check(lib().faar_silu_mul_bwd(ctx._h, rows, cols, _p(dout), ldd, _p(gate), ldg, _p(up), ldu, _p(dgate), lddg, _p(dup),
                                   lddu), "faar_silu_mul_bwd")


def embedding(ctx, rows, cols, vocab, table, ldt, tokens, out, ldo):
    _check(lib().faar_embedding(ctx._h, rows, cols, vocab, _p(table), ldt, _p(tokens), _p(out), ldo), "faar_embedding")


def add(ctx, rows, cols, a, lda, b, ldb, out, ldo):
    _check(lib().faar_add(ctx._h, rows, cols, _p(a), lda, _p(b), ldb, _p(out), ldo), "faar_add")


def tune_wide_tiles(ctx, mode: int):
    """1: 256 x 512 GEMM tiles whenever the shape allows; 0 or -1 (the default): never."""
    _check(lib().faar_tune_wide_tiles(ctx._h, mode), "faar_tune_wide_tiles")


def attention_status(ctx):
    """Raises FaarError(TIMEOUT) if a wait of the tcgen05 attention kernel gave up (call after a synchronise)."""
    code = C.c_uint32(0)
    _check(lib().faar_attention_status(ctx._h, C.byref(code)), f"faar_attention_status (code {code.value:#x})")


def tune_attention(ctx, mode: int):
    """head_dim 64: 0 = tcgen05 kernels forward and backward (default), 2 = register-resident mma.sync kernels,
    1 = the shared-memory fragment kernels (as head_dim 128 always takes)."""
    _check(lib().faar_tune_attention(ctx._h, mode), "faar_tune_attention")


def attention_fwd(ctx, batch, seq, n_heads, n_kv_heads, head_dim, q, ldq, k, v, ldkv, out, ldo, lse):
    _check(lib().faar_attention_fwd(ctx._h, batch, seq, n_heads, n_kv_heads, head_dim, _p(q), ldq, _p(k), _p(v), ldkv,
                                    _p(out), ldo, _p(lse)), "faar_attention_fwd")


def attention_bwd(ctx, batch, seq, n_heads, n_kv_heads, head_dim, q, ldq, k, v, ldkv, out, dout, ldo, lse, dsum, dq, dk, dv):
    _check(lib().faar_attention_bwd(ctx._h, batch, seq, n_heads, n_kv_heads, head_dim, _p(q), ldq, _p(k), _p(v), ldkv,
                                    _p(out), _p(dout), ldo, _p(lse), _p(dsum), _p(dq), _p(dk), _p(dv)), "faar_attention_bwd")


def nvfp4_gemm(ctx, M, N, K, A_packed, A_scales_tiled, A_s_global, B_packed, B_scales_tiled, B_s_global, C, ldc, ws):
    _check(lib().faar_nvfp4_gemm(ctx._h, M, N, K, _p(A_packed), _p(A_scales_tiled), _p(A_s_global), _p(B_packed),
                                 _p(B_scales_tiled), _p(B_s_global), _p(C), ldc, _p(ws), C_size(ws)), "faar_nvfp4_gemm")


def transpose_bf16(ctx, rows, cols, inp, ld_in, out, ld_out):
    _check(lib().faar_transpose_bf16(ctx._h, rows, cols, _p(inp), C.c_int64(ld_in), _p(out), C.c_int64(ld_out)),
           "faar_transpose_bf16")


def layer_ref(ctx, shape, X, W, Y_ref, ws):
    _check(lib().faar_layer_ref(ctx._h, C.byref(shape), _p(X), _p(W), _p(Y_ref), _p(ws), C.c_size_t(ws.numel())),
           "faar_layer_ref")


def layer_fwd(ctx, shape, hp, X, Y_ref, V, code, scales, s_global, dYt, loss_mse, Y_q, ws):
    _check(lib().faar_layer_fwd(ctx._h, C.byref(shape), C.byref(hp), _p(X), _p(Y_ref), _p(V), _p(code), _p(scales),
                                _p(s_global), _p(dYt), _p(loss_mse), _p(Y_q), _p(ws), C.c_size_t(ws.numel())),
           "faar_layer_fwd")


def layer_dx(ctx, shape, beta, dY, V, code, scales, s_global, WsoftT, dX, ws):
    _check(lib().faar_layer_dx(ctx._h, C.byref(shape), C.c_float(beta), _p(dY), _p(V), _p(code), _p(scales),
                               _p(s_global), _p(WsoftT), _p(dX), _p(ws), C.c_size_t(ws.numel())), "faar_layer_dx")


def layer_dx_operand(ctx, shape, dY, Wsoft, dX, ws):
    _check(lib().faar_layer_dx_operand(ctx._h, C.byref(shape), _p(dY), _p(Wsoft), _p(dX), _p(ws), C.c_size_t(ws.numel())),
           "faar_layer_dx_operand")


def round_loss(ctx, V, N, loss_round, ws):
    _check(lib().faar_round_loss(ctx._h, _p(V), C.c_int64(N), _p(loss_round), _p(ws), C.c_size_t(ws.numel())),
           "faar_round_loss")


def round_loss_static(ctx, V, N, loss_round):
    """Round Loss without a workspace: for callers that may not allocate device memory.  The scratch
    is a fixed array inside libfaar.so; N is limited to round_loss_static_max_n()."""
    _check(lib().faar_round_loss_static(ctx._h, _p(V), C.c_int64(N), _p(loss_round)), "faar_round_loss_static")


def round_loss_static_max_n() -> int:
    return int(lib().faar_round_loss_static_max_n())


def layer_bwd(ctx, shape, hp, dYt, Xt, V, code, scales, s_global, adam_m, adam_u, dV, ws):
    _check(lib().faar_layer_bwd(ctx._h, C.byref(shape), C.byref(hp), _p(dYt), _p(Xt), _p(V), _p(code), _p(scales),
                                _p(s_global), _p(adam_m), _p(adam_u), _p(dV), _p(ws), C.c_size_t(ws.numel())),
           "faar_layer_bwd")


def layer_bwd_rowmajor(ctx, shape, hp, dY, X, V, code, scales, s_global, adam_m, adam_u, dV, ws):
    _check(lib().faar_layer_bwd_rowmajor(ctx._h, C.byref(shape), C.byref(hp), _p(dY), _p(X), _p(V), _p(code), _p(scales),
                                _p(s_global), _p(adam_m), _p(adam_u), _p(dV), _p(ws), C.c_size_t(ws.numel())),
           "faar_layer_bwd_rowmajor")


def layer_step(ctx, shape, hp, X, Xt, Y_ref, V, code, scales, s_global, adam_m, adam_u, loss_out2, ws):
    _check(lib().faar_layer_step(ctx._h, C.byref(shape), C.byref(hp), _p(X), _p(Xt), _p(Y_ref), _p(V), _p(code),
                                 _p(scales), _p(s_global), _p(adam_m), _p(adam_u), _p(loss_out2), _p(ws),
                                 C.c_size_t(ws.numel())), "faar_layer_step")


def harden_pack(ctx, shape, V, code, scales, s_global, packed, scales_out, decisions, W_final, wfinal_dtype=F32):
    _check(lib().faar_harden_pack(ctx._h, C.byref(shape), _p(V), _p(code), _p(scales), _p(s_global), _p(packed),
                                  _p(scales_out), _p(decisions), _p(W_final), C.c_int(wfinal_dtype)),
           "faar_harden_pack")


def layer_step_host(ctx, shape, hp, X_host, Y_ref_host, W, X_dev, Xt_dev, Yref_dev, V, code, scales, s_global, adam_m,
                    adam_u, loss_dev2, loss_host2, ws):
    """X_host, Y_ref_host, loss_host2 are (pinned) CPU tensors; the rest are device tensors.  Y_ref_host None:
    the target is computed on the device from the copied X and W."""
    _check(lib().faar_layer_step_host(ctx._h, C.byref(shape), C.byref(hp), C.c_void_p(X_host.data_ptr()),
                                      C.c_void_p(Y_ref_host.data_ptr() if Y_ref_host is not None else 0), _p(W),
                                      _p(X_dev), _p(Xt_dev), _p(Yref_dev), _p(V),
                                      _p(code), _p(scales), _p(s_global), _p(adam_m), _p(adam_u), _p(loss_dev2),
                                      C.c_void_p(loss_host2.data_ptr()), _p(ws), C.c_size_t(ws.numel())),
           "faar_layer_step_host")


def nvfp4_expand(ctx, rows, K, packed, scales, out, ld):
    _check(lib().faar_nvfp4_expand(ctx._h, rows, K, _p(packed), _p(scales), _p(out), C.c_int64(ld)), "faar_nvfp4_expand")


def layer_step_host_nvfp4(ctx, shape, hp, Xpacked_host, Xscales_host, Y_ref_host, Xpacked_dev, Xscales_dev, Xq_dev, Yref_dev,
                          V, code, scales, s_global, adam_m, adam_u, loss_dev2, loss_host2, ws):
    """Host tensors (pinned): packed codes, block scales, frozen target, the two-float loss."""
    _check(lib().faar_layer_step_host_nvfp4(
        ctx._h, C.byref(shape), C.byref(hp), C.c_void_p(Xpacked_host.data_ptr()), C.c_void_p(Xscales_host.data_ptr()),
        C.c_void_p(Y_ref_host.data_ptr()), _p(Xpacked_dev), _p(Xscales_dev), _p(Xq_dev), _p(Yref_dev), _p(V), _p(code),
        _p(scales), _p(s_global), _p(adam_m), _p(adam_u), _p(loss_dev2), C.c_void_p(loss_host2.data_ptr()), _p(ws),
        C.c_size_t(ws.numel())), "faar_layer_step_host_nvfp4")


class KernelTime(C.Structure):
    _fields_ = [("kernel", C.c_int), ("launches", C.c_int), ("total_ms", C.c_float)]


def profile_begin(ctx):
    _check(lib().faar_profile_begin(ctx._h), "faar_profile_begin")


def profile_end(ctx) -> dict:
    """{kernel name: (launches, total_ms)} for the kernels launched since profile_begin."""
    arr = (KernelTime * 32)()
    n = C.c_int(0)
    _check(lib().faar_profile_end(ctx._h, arr, 32, C.byref(n)), "faar_profile_end")
    l = lib()
    return {l.faar_kernel_name(arr[i].kernel).decode(): (arr[i].launches, arr[i].total_ms) for i in range(n.value)}
