"""ctypes binding of libunitscale: same names as the C ABI, argument marshalling only.

Tensors are torch CUDA tensors (device memory and streams come from torch); every
computation happens inside the library's kernels.  Importing this module needs the
compiled library: there is no fallback of any kind.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

US_OK, US_ERR_INVALID_ARG, US_ERR_UNSUPPORTED, US_ERR_ALIGNMENT, US_ERR_WORKSPACE, US_ERR_CUDA, US_ERR_TIMEOUT = range(7)
STATUS_NAMES = {
    0: "US_OK", 1: "US_ERR_INVALID_ARG", 2: "US_ERR_UNSUPPORTED", 3: "US_ERR_ALIGNMENT",
    4: "US_ERR_WORKSPACE", 5: "US_ERR_CUDA", 6: "US_ERR_TIMEOUT",
}
US_F32, US_BF16, US_F16, US_E4M3, US_E5M2 = range(5)
US_ACT_NONE, US_ACT_GELU, US_ACT_GELU_GRAD, US_ACT_RELU, US_ACT_RELU_GRAD, US_ACT_TANH, US_ACT_TANH_GRAD, US_ACT_SIGMOID, US_ACT_SIGMOID_GRAD = range(9)
US_FN_GELU, US_FN_RELU, US_FN_TANH, US_FN_SIGMOID = range(4)
FN_BY_NAME = {"gelu": US_FN_GELU, "relu": US_FN_RELU, "tanh": US_FN_TANH, "sigmoid": US_FN_SIGMOID}

_TORCH_DTYPES = {
    torch.float32: US_F32, torch.bfloat16: US_BF16, torch.float16: US_F16,
    torch.float8_e4m3fn: US_E4M3, torch.float8_e5m2: US_E5M2,
}


class us_mat(C.Structure):
    _fields_ = [("ptr", C.c_void_p), ("dtype", C.c_int32), ("rows", C.c_int64), ("cols", C.c_int64), ("ld", C.c_int64)]


class us_epilogue(C.Structure):
    _fields_ = [
        ("act", C.c_int32), ("act_in_scale", C.c_float), ("act_out_scale", C.c_float),
        ("aux", us_mat), ("skip", us_mat), ("skip_coef", C.c_float), ("out_coef", C.c_float),
    ]


class us_batch(C.Structure):
    _fields_ = [("count", C.c_int64 * 2), ("a_stride", C.c_int64 * 2), ("b_stride", C.c_int64 * 2), ("out_stride", C.c_int64 * 2)]


class us_attention_batch(C.Structure):
    _fields_ = [("count", C.c_int64 * 2), ("q_stride", C.c_int64 * 2), ("k_stride", C.c_int64 * 2),
                ("v_stride", C.c_int64 * 2), ("c_stride", C.c_int64 * 2), ("p_stride", C.c_int64 * 2)]


class us_attention_bwd_batch(C.Structure):
    _fields_ = [("count", C.c_int64 * 2), ("dc_stride", C.c_int64 * 2), ("p_stride", C.c_int64 * 2), ("k_stride", C.c_int64 * 2),
                ("v_stride", C.c_int64 * 2), ("ds_stride", C.c_int64 * 2), ("dq_stride", C.c_int64 * 2)]


class us_linear_call(C.Structure):
    _fields_ = [("op", C.c_int32), ("a", us_mat), ("b", us_mat), ("scale", C.c_float), ("ep", us_epilogue), ("out", us_mat)]


US_OP_FWD, US_OP_BWD_X, US_OP_BWD_W = 0, 1, 2


class UnitScaleError(RuntimeError):
    def __init__(self, fn: str, status: int):
        self.status = status
        super().__init__(f"{fn}: {STATUS_NAMES.get(status, status)}")


def library_path() -> str:
    return os.path.join(os.path.dirname(os.path.abspath(__file__)), "libunitscale.so")


def _load() -> C.CDLL:
    path = library_path()
    if not os.path.exists(path):
        raise ImportError(
            f"{path} is missing: build it with `python -m paper_2303_11257_b200.build` "
            "(there is no fallback implementation)")
    lib = C.CDLL(path)
    P, MP, EP, F, V, SZ = C.c_void_p, C.POINTER(us_mat), C.POINTER(us_epilogue), C.c_float, C.c_void_p, C.c_size_t
    for name in ("us_linear_fwd", "us_linear_bwd_x", "us_linear_bwd_w"):
        fn = getattr(lib, name)
        fn.argtypes = [MP, MP, F, EP, MP, V, SZ, V]
        fn.restype = C.c_int
    for name in ("us_linear_fwd_batched", "us_linear_bwd_x_batched", "us_linear_bwd_w_batched"):
        fn = getattr(lib, name)
        fn.argtypes = [MP, MP, F, MP, C.POINTER(us_batch), V, SZ, V]
        fn.restype = C.c_int
    lib.us_attention_fwd.argtypes = [MP, MP, MP, F, F, F, MP, MP, C.POINTER(us_attention_batch), V, SZ, V]
    lib.us_attention_fwd.restype = C.c_int
    lib.us_attention_bwd.argtypes = [MP, MP, MP, MP, F, F, F, F, MP, MP, C.POINTER(us_attention_bwd_batch), V, SZ, V]
    lib.us_attention_bwd.restype = C.c_int
    lib.us_linear_fwd_static_ws.argtypes = [MP, MP, F, EP, MP, C.POINTER(C.c_void_p), V]
    lib.us_linear_fwd_static_ws.restype = C.c_int
    lib.us_linear_fwd_check.argtypes = [MP, MP, EP, MP, V, SZ]
    lib.us_linear_fwd_check.restype = C.c_int
    lib.us_test_linear_fwd_starved.argtypes = [MP, MP, F, MP, V, SZ, C.c_uint, V]
    lib.us_test_linear_fwd_starved.restype = C.c_int
    lib.us_linear_group.argtypes = [C.c_int, C.POINTER(us_linear_call), V, SZ, V]
    lib.us_linear_group.restype = C.c_int
    lib.us_ffn_hidden.argtypes = [MP, MP, F, MP, MP, F, F, F, F, C.c_int32, MP, MP, MP, V, SZ, V]
    lib.us_ffn_hidden.restype = C.c_int
    lib.us_test_ffn_hidden_starved.argtypes = [MP, MP, MP, MP, MP, MP, V, SZ, C.c_uint, V]
    lib.us_test_ffn_hidden_starved.restype = C.c_int
    lib.us_workspace_bytes.argtypes = []
    lib.us_workspace_bytes.restype = SZ
    lib.us_workspace_status.argtypes = [V, V]
    lib.us_workspace_status.restype = C.c_int
    lib.us_gelu_fwd.argtypes = [MP, F, F, MP, V]
    lib.us_gelu_bwd.argtypes = [MP, MP, F, F, MP, V]
    lib.us_residual_add.argtypes = [MP, MP, F, MP, V]
    lib.us_cast_fp8.argtypes = [MP, F, MP, V]
    lib.us_activation_fwd.argtypes = [C.c_int, MP, F, F, MP, V]
    lib.us_activation_bwd.argtypes = [C.c_int, MP, MP, F, F, MP, V]
    lib.us_activation_fwd.restype = lib.us_activation_bwd.restype = C.c_int
    lib.us_cast_fp8_multi.argtypes = [C.c_int, MP, C.POINTER(C.c_float), MP, V]
    lib.us_weighted_add.argtypes = [C.c_int, MP, C.POINTER(C.c_float), F, MP, V]
    lib.us_weighted_add.restype = C.c_int
    lib.us_softmax_fwd.argtypes = [MP, F, MP, V]
    lib.us_softmax_bwd.argtypes = [MP, MP, F, F, MP, V]
    lib.us_softmax_xent_fwd.argtypes = [MP, V, V, V]
    lib.us_softmax_xent_bwd.argtypes = [MP, V, V, F, MP, V]
    lib.us_softmax_xent_fwd.restype = lib.us_softmax_xent_bwd.restype = C.c_int
    lib.us_layer_norm_fwd.argtypes = [MP, MP, MP, F, MP, V]
    lib.us_layer_norm_bwd.argtypes = [MP, MP, MP, F, F, F, MP, MP, MP, V, SZ, V]
    lib.us_layer_norm_fwd.restype = lib.us_layer_norm_bwd.restype = C.c_int
    lib.us_layer_norm_bwd_workspace_bytes.argtypes = [C.c_int64, C.c_int64]
    lib.us_layer_norm_bwd_workspace_bytes.restype = SZ
    lib.us_quant_stats_workspace_bytes.argtypes = []
    lib.us_quant_stats_workspace_bytes.restype = SZ
    lib.us_quant_stats.argtypes = [MP, F, C.c_int, C.c_int, C.c_int, V, V, V, SZ, V]
    lib.us_quant_stats.restype = C.c_int
    for name in ("us_gelu_fwd", "us_gelu_bwd", "us_residual_add", "us_cast_fp8", "us_cast_fp8_multi", "us_softmax_fwd", "us_softmax_bwd"):
        getattr(lib, name).restype = C.c_int
    FP = C.POINTER(C.c_float)
    lib.us_scales_linear.argtypes = [C.c_int64, C.c_int64, C.c_int64, C.c_int, FP, FP, FP]
    lib.us_scales_linear.restype = C.c_int
    lib.us_scales_gelu.argtypes = [C.c_int, FP, FP]
    lib.us_scales_activation.argtypes = [C.c_int, C.c_int, FP, FP]
    lib.us_scales_activation.restype = C.c_int
    lib.us_scales_gelu.restype = C.c_int
    lib.us_scales_residual.argtypes = [C.c_float, FP, FP]
    lib.us_scales_residual.restype = C.c_int
    lib.us_scales_attention.argtypes = [C.c_int64, C.c_int64, C.c_int, FP, FP, FP, FP, FP, FP]
    lib.us_scales_attention.restype = C.c_int
    lib.us_status_string.argtypes = [C.c_int]
    lib.us_status_string.restype = C.c_char_p
    lib.us_version.argtypes = []
    lib.us_version.restype = C.c_int
    return lib


_lib = _load()


def raw() -> C.CDLL:
    """The loaded CDLL, for callers that want to build us_mat structures themselves."""
    return _lib


def mat(t: torch.Tensor) -> us_mat:
    """Describe a 2-D row-major torch tensor (last stride 1) without copying it."""
    if t.dim() != 2 or (t.shape[1] > 1 and t.stride(1) != 1):
        raise ValueError("expected a 2-D tensor with unit column stride")
    ld = t.stride(0) if t.shape[0] > 1 else max(t.shape[1], t.stride(0))
    return us_mat(t.data_ptr(), _TORCH_DTYPES[t.dtype], t.shape[0], t.shape[1], ld)


def _stream(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _check(fn: str, status: int) -> None:
    if status != US_OK:
        raise UnitScaleError(fn, status)


def epilogue(act: int = US_ACT_NONE, act_in_scale: float = 1.0, act_out_scale: float = 1.0,
             aux: torch.Tensor | None = None, skip: torch.Tensor | None = None,
             skip_coef: float = 0.0, out_coef: float = 1.0) -> us_epilogue:
    ep = us_epilogue()
    ep.act, ep.act_in_scale, ep.act_out_scale = act, act_in_scale, act_out_scale
    if aux is not None:
        ep.aux = mat(aux)
    if skip is not None:
        ep.skip = mat(skip)
    ep.skip_coef, ep.out_coef = skip_coef, out_coef
    ep._keep_alive = (aux, skip)      # the struct holds raw pointers only
    return ep


def us_workspace_bytes() -> int:
    return int(_lib.us_workspace_bytes())


def new_workspace(device="cuda") -> torch.Tensor:
    """A zeroed workspace of the size the linear ops ask for."""
    return torch.zeros(us_workspace_bytes(), dtype=torch.uint8, device=device)


def us_workspace_status(ws: torch.Tensor, stream=None) -> int:
    return int(_lib.us_workspace_status(ws.data_ptr(), _stream(stream)))


def _linear(name, a, b, scale, ep, out, ws, stream):
    fn = getattr(_lib, name)
    epp = C.byref(ep) if ep is not None else None
    _check(name, fn(C.byref(mat(a)), C.byref(mat(b)), scale, epp, C.byref(mat(out)),
                    ws.data_ptr(), ws.numel() * ws.element_size(), _stream(stream)))
    return out


def us_linear_fwd(X, W, alpha, Y, ws, ep=None, stream=None):
    return _linear("us_linear_fwd", X, W, alpha, ep, Y, ws, stream)


def us_linear_bwd_x(G, W, beta_x, dX, ws, ep=None, stream=None):
    return _linear("us_linear_bwd_x", G, W, beta_x, ep, dX, ws, stream)


def us_linear_bwd_w(X, G, beta_w, dW, ws, ep=None, stream=None):
    return _linear("us_linear_bwd_w", X, G, beta_w, ep, dW, ws, stream)


def linear_call(op: int, a, b, scale: float, out, ep=None) -> us_linear_call:
    """One entry of a us_linear_group launch: op in (US_OP_FWD, US_OP_BWD_X, US_OP_BWD_W), operands in that op's order."""
    c = us_linear_call()
    c.op, c.a, c.b, c.scale, c.out = op, mat(a), mat(b), scale, mat(out)
    if ep is not None:
        c.ep = ep
    else:
        c.ep.out_coef = 1.0
    c._keep_alive = (a, b, out, ep)
    return c


def us_linear_group(calls, ws, stream=None):
    """Several independent linear ops in one launch (see the header for what this form covers)."""
    arr = (us_linear_call * len(calls))(*calls)
    _check("us_linear_group", _lib.us_linear_group(len(calls), arr, ws.data_ptr(), ws.numel() * ws.element_size(), _stream(stream)))


def batch(count, a_stride, b_stride, out_stride) -> us_batch:
    """us_batch from (outer, inner) pairs of counts and element strides."""
    b = us_batch()
    for i in range(2):
        b.count[i], b.a_stride[i], b.b_stride[i], b.out_stride[i] = count[i], a_stride[i], b_stride[i], out_stride[i]
    return b


def _linear_batched(name, a, b, scale, out, bt, ws, stream):
    fn = getattr(_lib, name)
    _check(name, fn(C.byref(mat(a)), C.byref(mat(b)), scale, C.byref(mat(out)), C.byref(bt),
                    ws.data_ptr(), ws.numel() * ws.element_size(), _stream(stream)))
    return out


def us_linear_fwd_batched(X, W, alpha, Y, bt, ws, stream=None):
    return _linear_batched("us_linear_fwd_batched", X, W, alpha, Y, bt, ws, stream)


def us_linear_bwd_x_batched(G, W, beta_x, dX, bt, ws, stream=None):
    return _linear_batched("us_linear_bwd_x_batched", G, W, beta_x, dX, bt, ws, stream)


def us_linear_bwd_w_batched(X, G, beta_w, dW, bt, ws, stream=None):
    return _linear_batched("us_linear_bwd_w_batched", X, G, beta_w, dW, bt, ws, stream)


def attention_batch(count, q_stride, k_stride, v_stride, c_stride, p_stride=(0, 0)) -> us_attention_batch:
    """us_attention_batch from (outer, inner) pairs of counts and element strides."""
    b = us_attention_batch()
    for i in range(2):
        b.count[i] = count[i]
        b.q_stride[i], b.k_stride[i], b.v_stride[i] = q_stride[i], k_stride[i], v_stride[i]
        b.c_stride[i], b.p_stride[i] = c_stride[i], p_stride[i]
    return b


def us_attention_fwd(Q, K, V, alpha_scores, softmax_scale, alpha_context, Cx, P, bt, ws, stream=None):
    """Fused scaled dot-product attention forward; P may be None (weights not stored)."""
    pp = C.byref(mat(P)) if P is not None else None
    _check("us_attention_fwd",
           _lib.us_attention_fwd(C.byref(mat(Q)), C.byref(mat(K)), C.byref(mat(V)), alpha_scores, softmax_scale,
                                 alpha_context, C.byref(mat(Cx)), pp, C.byref(bt), ws.data_ptr(),
                                 ws.numel() * ws.element_size(), _stream(stream)))
    return Cx


def attention_bwd_batch(count, dc_stride, p_stride, k_stride, v_stride, ds_stride, dq_stride) -> us_attention_bwd_batch:
    b = us_attention_bwd_batch()
    for i in range(2):
        b.count[i] = count[i]
        b.dc_stride[i], b.p_stride[i], b.k_stride[i] = dc_stride[i], p_stride[i], k_stride[i]
        b.v_stride[i], b.ds_stride[i], b.dq_stride[i] = v_stride[i], ds_stride[i], dq_stride[i]
    return b


def us_attention_bwd(dC, P, K, V, beta_p, softmax_alpha, softmax_beta, beta_q, dS, dQ, bt, ws, stream=None):
    """Attention backward down to the queries: dS (for the dK matmul) and dQ from dC, the stored P, K and V."""
    _check("us_attention_bwd",
           _lib.us_attention_bwd(C.byref(mat(dC)), C.byref(mat(P)), C.byref(mat(K)), C.byref(mat(V)), beta_p, softmax_alpha,
                                 softmax_beta, beta_q, C.byref(mat(dS)), C.byref(mat(dQ)), C.byref(bt), ws.data_ptr(),
                                 ws.numel() * ws.element_size(), _stream(stream)))
    return dQ


def us_linear_fwd_static_ws(X, W, alpha, Y, ep=None, stream=None) -> int:
    """us_linear_fwd without a caller workspace: the library's built-in scratch array is used and
    nothing is allocated.  For callers that cannot allocate device memory (see the header).
    Returns the device address of the built-in scratch, which us_workspace_status_ptr accepts."""
    ws = C.c_void_p()
    epp = C.byref(ep) if ep is not None else None
    _check("us_linear_fwd_static_ws",
           _lib.us_linear_fwd_static_ws(C.byref(mat(X)), C.byref(mat(W)), alpha, epp, C.byref(mat(Y)),
                                        C.byref(ws), _stream(stream)))
    return ws.value


def us_linear_fwd_check(X, W, Y, ws, ep=None) -> int:
    """Status us_linear_fwd would return from its host-side checks (0 = it would launch); launches nothing."""
    epp = C.byref(ep) if ep is not None else None
    return int(_lib.us_linear_fwd_check(C.byref(mat(X)), C.byref(mat(W)), epp, C.byref(mat(Y)),
                                        ws.data_ptr(), ws.numel() * ws.element_size()))


def us_test_linear_fwd_starved(X, W, alpha, Y, ws, wait_limit: int, stream=None):
    """The failure-path exercise of the header: a forward linear launch whose loads are withheld and
    whose waits give up after wait_limit polls; the status word in ws is raised and the kernel returns."""
    _check("us_test_linear_fwd_starved",
           _lib.us_test_linear_fwd_starved(C.byref(mat(X)), C.byref(mat(W)), alpha, C.byref(mat(Y)), ws.data_ptr(),
                                           ws.numel() * ws.element_size(), wait_limit, _stream(stream)))


def us_ffn_hidden(X, W1, alpha, G, W2, beta_x, act_in_scale, act_out_scale, grad_out_scale, A, dH, ws,
                  H=None, h_dtype=torch.bfloat16, stream=None):
    """Hidden layer of the FFN block, forward and backward, in one launch (see the header): A and dH are written,
    H (optional) receives the pre-activation rounded to h_dtype."""
    hp = C.byref(mat(H)) if H is not None else None
    _check("us_ffn_hidden",
           _lib.us_ffn_hidden(C.byref(mat(X)), C.byref(mat(W1)), alpha, C.byref(mat(G)), C.byref(mat(W2)), beta_x,
                              act_in_scale, act_out_scale, grad_out_scale, _TORCH_DTYPES[h_dtype], hp, C.byref(mat(A)),
                              C.byref(mat(dH)), ws.data_ptr(), ws.numel() * ws.element_size(), _stream(stream)))
    return A, dH


def us_test_ffn_hidden_starved(X, W1, G, W2, A, dH, ws, wait_limit: int, stream=None):
    """us_test_linear_fwd_starved for the kernel of us_ffn_hidden."""
    _check("us_test_ffn_hidden_starved",
           _lib.us_test_ffn_hidden_starved(C.byref(mat(X)), C.byref(mat(W1)), C.byref(mat(G)), C.byref(mat(W2)),
                                           C.byref(mat(A)), C.byref(mat(dH)), ws.data_ptr(),
                                           ws.numel() * ws.element_size(), wait_limit, _stream(stream)))


def us_workspace_status_ptr(ws_ptr: int, stream=None) -> int:
    """us_workspace_status for a raw device address."""
    return int(_lib.us_workspace_status(ws_ptr, _stream(stream)))


def us_gelu_fwd(H, s_in, alpha, A, stream=None):
    _check("us_gelu_fwd", _lib.us_gelu_fwd(C.byref(mat(H)), s_in, alpha, C.byref(mat(A)), _stream(stream)))
    return A


def us_gelu_bwd(H, dA, s_in, beta, dH, stream=None):
    _check("us_gelu_bwd", _lib.us_gelu_bwd(C.byref(mat(H)), C.byref(mat(dA)), s_in, beta, C.byref(mat(dH)), _stream(stream)))
    return dH


def us_activation_fwd(fn, H, s_in, alpha, A, stream=None):
    _check("us_activation_fwd", _lib.us_activation_fwd(FN_BY_NAME.get(fn, fn), C.byref(mat(H)), s_in, alpha, C.byref(mat(A)), _stream(stream)))
    return A


def us_activation_bwd(fn, H, dA, s_in, beta, dH, stream=None):
    _check("us_activation_bwd", _lib.us_activation_bwd(FN_BY_NAME.get(fn, fn), C.byref(mat(H)), C.byref(mat(dA)), s_in, beta,
                                                       C.byref(mat(dH)), _stream(stream)))
    return dH


def us_scales_activation(fn, constrained: bool = False):
    a, b = C.c_float(), C.c_float()
    _check("us_scales_activation", _lib.us_scales_activation(FN_BY_NAME.get(fn, fn), int(constrained), C.byref(a), C.byref(b)))
    return a.value, b.value


def us_residual_add(skip, branch, tau, out, stream=None):
    _check("us_residual_add", _lib.us_residual_add(C.byref(mat(skip)), C.byref(mat(branch)), tau, C.byref(mat(out)), _stream(stream)))
    return out


def us_cast_fp8(src, scale, dst, stream=None):
    _check("us_cast_fp8", _lib.us_cast_fp8(C.byref(mat(src)), scale, C.byref(mat(dst)), _stream(stream)))
    return dst


def us_weighted_add(srcs, gammas, alpha, out, stream=None):
    n = len(srcs)
    sm = (us_mat * n)(*[mat(t) for t in srcs])
    gm = (C.c_float * n)(*[float(g) for g in gammas])
    _check("us_weighted_add", _lib.us_weighted_add(n, sm, gm, alpha, C.byref(mat(out)), _stream(stream)))
    return out


def us_cast_fp8_multi(srcs, scales, dsts, stream=None):
    """One launch for len(srcs) casts; scales: one float per tensor."""
    n = len(srcs)
    sm = (us_mat * n)(*[mat(t) for t in srcs])
    dm = (us_mat * n)(*[mat(t) for t in dsts])
    sc = (C.c_float * n)(*[float(x) for x in scales])
    _check("us_cast_fp8_multi", _lib.us_cast_fp8_multi(n, sm, sc, dm, _stream(stream)))
    return dsts


def us_softmax_fwd(S, alpha, P, stream=None):
    _check("us_softmax_fwd", _lib.us_softmax_fwd(C.byref(mat(S)), alpha, C.byref(mat(P)), _stream(stream)))
    return P


def us_softmax_bwd(P, dP, alpha, beta, dS, stream=None):
    _check("us_softmax_bwd", _lib.us_softmax_bwd(C.byref(mat(P)), C.byref(mat(dP)), alpha, beta, C.byref(mat(dS)), _stream(stream)))
    return dS


def us_softmax_xent_fwd(X, targets, out, stream=None):
    """targets: int32 CUDA tensor [rows]; out: float32 CUDA tensor [rows]."""
    assert targets.dtype == torch.int32 and out.dtype == torch.float32 and targets.is_contiguous() and out.is_contiguous()
    _check("us_softmax_xent_fwd", _lib.us_softmax_xent_fwd(C.byref(mat(X)), targets.data_ptr(), out.data_ptr(), _stream(stream)))
    return out


def us_softmax_xent_bwd(X, targets, g, beta, dX, stream=None):
    """g: float32 CUDA tensor [rows] or None (ones)."""
    assert targets.dtype == torch.int32 and targets.is_contiguous() and (g is None or (g.dtype == torch.float32 and g.is_contiguous()))
    _check("us_softmax_xent_bwd", _lib.us_softmax_xent_bwd(C.byref(mat(X)), targets.data_ptr(), g.data_ptr() if g is not None else None,
                                                           beta, C.byref(mat(dX)), _stream(stream)))
    return dX


def us_quant_stats(src, scale, fmt, exp_lo, nbins, stream=None):
    """Returns (snr, sum v^2, sum err^2, hist) with hist a list of nbins + 2 counts; fmt: a torch dtype.
    Allocates its small outputs and the workspace with torch and synchronises to read them back."""
    sums = torch.empty(2, dtype=torch.float64, device=src.device)
    hist = torch.empty(nbins + 2, dtype=torch.int64, device=src.device)
    ws = torch.empty(int(_lib.us_quant_stats_workspace_bytes()), dtype=torch.uint8, device=src.device)
    _check("us_quant_stats", _lib.us_quant_stats(C.byref(mat(src)), scale, _TORCH_DTYPES[fmt], exp_lo, nbins, sums.data_ptr(),
                                                 hist.data_ptr(), ws.data_ptr(), ws.numel(), _stream(stream)))
    s = sums.cpu().tolist()
    return (s[0] / s[1] if s[1] > 0 else float("inf")), s[0], s[1], hist.cpu().tolist()


def _vec(t: torch.Tensor) -> us_mat:
    """A 1-D parameter tensor as a 1 x n us_mat."""
    return mat(t.view(1, -1))


def us_layer_norm_fwd(X, w, c, eps, Y, stream=None):
    _check("us_layer_norm_fwd", _lib.us_layer_norm_fwd(C.byref(mat(X)), C.byref(_vec(w)), C.byref(_vec(c)), eps,
                                                       C.byref(mat(Y)), _stream(stream)))
    return Y


def us_layer_norm_bwd_workspace_bytes(rows: int, cols: int) -> int:
    return int(_lib.us_layer_norm_bwd_workspace_bytes(rows, cols))


def us_layer_norm_bwd(X, w, G, eps, beta_x, beta_wc, dX, dw, dc, ws, stream=None):
    """ws: a uint8 CUDA tensor of at least us_layer_norm_bwd_workspace_bytes(rows, cols) bytes."""
    _check("us_layer_norm_bwd", _lib.us_layer_norm_bwd(
        C.byref(mat(X)), C.byref(_vec(w)), C.byref(mat(G)), eps, beta_x, beta_wc, C.byref(mat(dX)), C.byref(_vec(dw)),
        C.byref(_vec(dc)), ws.data_ptr(), ws.numel() * ws.element_size(), _stream(stream)))
    return dX, dw, dc


def us_scales_linear(b: int, m: int, n: int, constrained: bool = False):
    a, bx, bw = C.c_float(), C.c_float(), C.c_float()
    _check("us_scales_linear", _lib.us_scales_linear(b, m, n, int(constrained), C.byref(a), C.byref(bx), C.byref(bw)))
    return a.value, bx.value, bw.value


def us_scales_gelu(constrained: bool = False):
    a, b = C.c_float(), C.c_float()
    _check("us_scales_gelu", _lib.us_scales_gelu(int(constrained), C.byref(a), C.byref(b)))
    return a.value, b.value


def us_scales_residual(tau: float):
    """(sqrt(1 - tau), sqrt(tau)) as the float32 values the library uses."""
    a, b = C.c_float(), C.c_float()
    _check("us_scales_residual", _lib.us_scales_residual(tau, C.byref(a), C.byref(b)))
    return a.value, b.value


def us_scales_attention(s: int, d_head: int, constrained: bool = False) -> dict:
    """Factors of scaled dot-product attention (see the header), keyed as the encoder driver uses them."""
    v = [C.c_float() for _ in range(6)]
    _check("us_scales_attention", _lib.us_scales_attention(s, d_head, int(constrained), *[C.byref(x) for x in v]))
    a_s, b_s, sm, a_c, b_p, b_v = (x.value for x in v)
    return dict(alpha_s=a_s, beta_Q=b_s, beta_K=b_s, sm=sm, alpha_c=a_c, beta_P=b_p, beta_V=b_v)


def us_status_string(status: int) -> str:
    return _lib.us_status_string(status).decode()


def us_version() -> int:
    return int(_lib.us_version())
