"""ctypes binding of ``libpike.so``: argument marshalling only.

Every function has the name of the C entry point it calls.  torch is used for
device memory (outputs, workspaces) and the current CUDA stream; all arithmetic
runs in the library's kernels.  There is no fallback: if the shared library is
missing, loading raises.
"""
from __future__ import annotations

import contextlib
import ctypes
import os
import threading

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libpike.so")

PIKE_F32, PIKE_BF16, PIKE_F16 = 0, 1, 2
ACT = {"none": 0, "gelu_erf": 1, "gelu_tanh": 2, "silu": 3}
REDUCE = {"none": 0, "layernorm": 1, "softmax": 2}
FLAG_W_IS_NK, FLAG_CAUSAL, FLAG_ONE_PASS = 0x1, 0x2, 0x4

EXPORTS = (
    "pike_create", "pike_destroy", "pike_status_string", "pike_get_last_device_status",
    "pike_set_wait_limit_ns", "pike_test_withhold_loads", "pike_test_withhold_partials", "pike_profile_begin", "pike_profile_end", "pike_linear_epilogue_workspace", "pike_linear_epilogue",
    "pike_mlp_block_workspace", "pike_mlp_block", "pike_attention_chain_workspace",
    "pike_attention_chain", "pike_linear_softmax_noalloc", "pike_attention_block_workspace", "pike_attention_block",
    "pike_grouped_linear_epilogue", "pike_linear_softmax_shard_workspace", "pike_linear_softmax_shard_local",
    "pike_linear_softmax_shard_finish",
)


class PikeError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__(f"{what}: status {code} ({pike_status_string(code)})")
        self.code = code


class pike_tensor_t(ctypes.Structure):
    _fields_ = [("data", ctypes.c_void_p), ("dtype", ctypes.c_int), ("ndim", ctypes.c_int32),
                ("shape", ctypes.c_int64 * 4), ("stride", ctypes.c_int64 * 4)]


class pike_epilogue_t(ctypes.Structure):
    _fields_ = [("struct_size", ctypes.c_uint32), ("act", ctypes.c_int), ("scale", ctypes.c_float),
                ("reduce", ctypes.c_int), ("eps", ctypes.c_float), ("out_dtype", ctypes.c_int),
                ("flags", ctypes.c_uint32)]


class pike_kernel_profile_t(ctypes.Structure):
    _fields_ = [("launches", ctypes.c_uint64), ("device_ms", ctypes.c_double)]


KERNELS = ("fp32_chain", "gemm_bf16", "layernorm_bf16", "softmax_finish", "attention_bf16")

_lib = None
_lock = threading.Lock()
_handles: dict[int, ctypes.c_void_p] = {}


def library_path() -> str:
    return _LIB_PATH


def load_library() -> ctypes.CDLL:
    """dlopen libpike.so and declare the prototypes.  Raises if it was not built."""
    global _lib
    if _lib is not None:
        return _lib
    with _lock:
        if _lib is None:
            if not os.path.exists(_LIB_PATH):
                raise RuntimeError(
                    f"{_LIB_PATH} is missing: build it with `python -m paper_2511_16964_b200.build` "
                    "(there is no CPU or PyTorch fallback)")
            lib = ctypes.CDLL(_LIB_PATH)
            T, E = ctypes.POINTER(pike_tensor_t), ctypes.POINTER(pike_epilogue_t)
            vp, sz = ctypes.c_void_p, ctypes.c_size_t
            lib.pike_create.argtypes = [ctypes.POINTER(vp), ctypes.c_int]
            lib.pike_destroy.argtypes = [vp]
            lib.pike_status_string.argtypes = [ctypes.c_int]
            lib.pike_status_string.restype = ctypes.c_char_p
            lib.pike_get_last_device_status.argtypes = [vp, ctypes.POINTER(ctypes.c_int), ctypes.POINTER(ctypes.c_uint32)]
            lib.pike_set_wait_limit_ns.argtypes = [vp, ctypes.c_uint64]
            lib.pike_test_withhold_loads.argtypes = [vp]
            lib.pike_test_withhold_partials.argtypes = [vp]
            lib.pike_profile_begin.argtypes = [vp]
            lib.pike_profile_end.argtypes = [vp, ctypes.POINTER(pike_kernel_profile_t)]
            lib.pike_linear_epilogue_workspace.argtypes = [vp, T, T, E, ctypes.POINTER(sz)]
            lib.pike_linear_epilogue.argtypes = [vp, T, T, T, T, T, T, E, T, vp, sz, vp]
            lib.pike_linear_softmax_noalloc.argtypes = [vp, T, T, T, E, T, vp]
            lib.pike_linear_softmax_shard_workspace.argtypes = [vp, T, T, E, ctypes.POINTER(sz)]
            lib.pike_linear_softmax_shard_local.argtypes = [vp, T, T, T, E, T, vp, vp, sz, vp]
            lib.pike_linear_softmax_shard_finish.argtypes = [vp, T, vp, ctypes.c_int32, vp]
            lib.pike_mlp_block_workspace.argtypes = [vp, T, T, E, ctypes.POINTER(sz)]
            lib.pike_mlp_block.argtypes = [vp, T, T, T, T, T, T, T, E, T, vp, sz, vp]
            lib.pike_attention_chain_workspace.argtypes = [vp, T, E, ctypes.POINTER(sz)]
            lib.pike_attention_chain.argtypes = [vp, T, T, T, E, T, vp, sz, vp]
            lib.pike_grouped_linear_epilogue.argtypes = [vp, T, T, T, T, vp, E, T, vp]
            lib.pike_attention_block_workspace.argtypes = [vp, T, E, ctypes.POINTER(sz)]
            lib.pike_attention_block.argtypes = [vp, T, T, T, T, T, T, T, E, T, vp, sz, vp]
            for name in EXPORTS:
                if name != "pike_status_string":
                    getattr(lib, name).restype = ctypes.c_int
            _lib = lib
    return _lib


def pike_status_string(code: int) -> str:
    return load_library().pike_status_string(int(code)).decode()


def _handle(device: torch.device) -> ctypes.c_void_p:
    idx = device.index if device.index is not None else torch.cuda.current_device()
    h = _handles.get(idx)
    if h is None:
        lib = load_library()
        h = ctypes.c_void_p()
        rc = lib.pike_create(ctypes.byref(h), idx)
        if rc:
            raise PikeError(rc, "pike_create")
        with _lock:
            _handles[idx] = h
    return h


_DTYPE_CODE = {torch.float32: PIKE_F32, torch.bfloat16: PIKE_BF16, torch.float16: PIKE_F16}
_I64x4 = ctypes.c_int64 * 4
# Descriptors already built, keyed by everything they hold: a model calls the same chains on the same buffers over
# and over, and building a ctypes structure costs more host time than the small chains' kernels take.
_desc_cache: dict = {}
_epi_cache: dict = {}
_ws_bytes_cache: dict = {}
_CACHE_LIMIT = 4096


def _dtype_code(t: torch.Tensor) -> int:
    try:
        return _DTYPE_CODE[t.dtype]
    except KeyError:
        raise TypeError(f"unsupported dtype {t.dtype}") from None


def _tensor(t):
    """torch CUDA tensor -> pike_tensor_t (by reference); None -> NULL."""
    if t is None:
        return None
    shape, stride = t.shape, t.stride()
    key = (t.data_ptr(), shape, stride, t.dtype)
    ref = _desc_cache.get(key)
    if ref is not None:
        return ref
    if not t.is_cuda:
        raise ValueError("tensors must live in CUDA device memory")
    if len(shape) > 4:
        raise ValueError("at most four dimensions")
    if 1 in shape:
        # torch leaves the stride of an extent-1 dimension arbitrary (a [1, K] view of a [K, 1] array keeps stride
        # 1); the C ABI wants every outer stride to cover the dimensions inside it, so such strides are canonicalised
        stride, inner = list(stride), 1
        for i in reversed(range(len(shape))):
            if shape[i] == 1:
                stride[i] = max(inner, 1)
            inner = max(inner, stride[i] * shape[i])
    ref = ctypes.byref(pike_tensor_t(key[0], _dtype_code(t), len(shape), _I64x4(*shape), _I64x4(*stride)))
    if len(_desc_cache) >= _CACHE_LIMIT:
        _desc_cache.clear()
    _desc_cache[key] = ref
    return ref


def _epilogue(act, scale, reduce, eps, out_dtype, flags):
    """The epilogue descriptor, by reference."""
    key = (act, scale, reduce, eps, out_dtype, flags)
    ref = _epi_cache.get(key)
    if ref is None:
        e = pike_epilogue_t(ctypes.sizeof(pike_epilogue_t), ACT[act], float(scale), REDUCE[reduce], float(eps),
                            _DTYPE_CODE[out_dtype], flags)
        if len(_epi_cache) >= _CACHE_LIMIT:
            _epi_cache.clear()
        ref = _epi_cache[key] = ctypes.byref(e)
    return ref


def _stream(stream) -> ctypes.c_void_p:
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _on(stream):
    """Allocations made for a call belong to the stream the kernels are enqueued on: torch's caching
    allocator hands a freed block back to allocations of the SAME stream only, in stream order, so a
    temporary dropped right after the call cannot be reused while the kernels still read or write it."""
    return contextlib.nullcontext() if stream is None else torch.cuda.stream(stream)


def _workspace(query, device, workspace, stream, key=None):
    """(keep-alive, pointer, bytes) of the workspace: the caller's, or a temporary of the size `query()`
    returns, allocated on `stream` (nothing when the chain needs none).  The size depends on the shapes, types and
    flags in `key` only, so it is asked for once per key.  A caller-supplied workspace is sized by the C side's
    own check."""
    if workspace is None:
        need = _ws_bytes_cache.get(key) if key is not None else None
        if need is None:
            need = int(query())
            if key is not None:
                if len(_ws_bytes_cache) >= _CACHE_LIMIT:
                    _ws_bytes_cache.clear()
                _ws_bytes_cache[key] = need
        if need == 0:
            return None, None, 0
        with _on(stream):
            workspace = torch.empty(need, dtype=torch.uint8, device=device)
    return workspace, ctypes.c_void_p(workspace.data_ptr()), workspace.numel() * workspace.element_size()


def _check(rc: int, what: str):
    if rc:
        raise PikeError(rc, what)


def pike_set_wait_limit_ns(ns: int, device=None) -> None:
    dev = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
    _check(load_library().pike_set_wait_limit_ns(_handle(dev), int(ns)), "pike_set_wait_limit_ns")


def pike_test_withhold_loads(device=None) -> None:
    """Test hook: the next bf16 GEMM issues no loads, so a bounded wait runs out (see include/pike.h)."""
    dev = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
    _check(load_library().pike_test_withhold_loads(_handle(dev)), "pike_test_withhold_loads")


def pike_test_withhold_partials(device=None) -> None:
    """Test hook: in the next one-pass softmax one CTA never counts itself in, so the stripe waits run out."""
    dev = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
    _check(load_library().pike_test_withhold_partials(_handle(dev)), "pike_test_withhold_partials")


def pike_get_last_device_status(device=None) -> tuple[int, int]:
    """(status, where) of the device status word.  Does not wait for anybody's kernels: synchronise the
    streams whose status is wanted first (torch.cuda.synchronize() or stream.synchronize())."""
    dev = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
    st, where = ctypes.c_int(0), ctypes.c_uint32(0)
    _check(load_library().pike_get_last_device_status(_handle(dev), ctypes.byref(st), ctypes.byref(where)),
           "pike_get_last_device_status")
    return st.value, where.value


def pike_profile_begin(device=None) -> None:
    dev = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
    _check(load_library().pike_profile_begin(_handle(dev)), "pike_profile_begin")


def pike_profile_end(device=None) -> dict:
    """{kernel name: (launches, summed device ms)} since pike_profile_begin; synchronises."""
    dev = torch.device("cuda", torch.cuda.current_device()) if device is None else torch.device(device)
    out = (pike_kernel_profile_t * len(KERNELS))()
    _check(load_library().pike_profile_end(_handle(dev), out), "pike_profile_end")
    return {name: (int(out[i].launches), float(out[i].device_ms)) for i, name in enumerate(KERNELS)}


def pike_linear_epilogue_workspace(x, w, *, act="none", scale=1.0, reduce="none", eps=1e-5,
                                   out_dtype=None, w_is_nk=False, one_pass=False) -> int:
    out_dtype = x.dtype if out_dtype is None else out_dtype
    e = _epilogue(act, scale, reduce, eps, out_dtype, (FLAG_W_IS_NK if w_is_nk else 0) | (FLAG_ONE_PASS if one_pass else 0))
    n = ctypes.c_size_t(0)
    _check(load_library().pike_linear_epilogue_workspace(_handle(x.device), _tensor(x), _tensor(w),
                                                         e, ctypes.byref(n)),
           "pike_linear_epilogue_workspace")
    return n.value


def pike_linear_epilogue(x, w, bias=None, residual=None, gamma=None, beta=None, *, act="none", scale=1.0,
                         reduce="none", eps=1e-5, out_dtype=None, w_is_nk=False, one_pass=False, out=None,
                         workspace=None, stream=None):
    """out = reduce(scale*act(x @ w + bias) + residual); one_pass selects PIKE_FLAG_ONE_PASS; see include/pike.h."""
    out_dtype = (out.dtype if out is not None else x.dtype) if out_dtype is None else out_dtype
    N = w.shape[0] if w_is_nk else w.shape[1]
    if out is None:
        with _on(stream):
            out = torch.empty((x.shape[0], N), dtype=out_dtype, device=x.device)
    e = _epilogue(act, scale, reduce, eps, out_dtype, (FLAG_W_IS_NK if w_is_nk else 0) | (FLAG_ONE_PASS if one_pass else 0))
    ws, ws_ptr, ws_bytes = _workspace(
        lambda: pike_linear_epilogue_workspace(x, w, act=act, scale=scale, reduce=reduce, eps=eps, out_dtype=out_dtype,
                                               w_is_nk=w_is_nk, one_pass=one_pass), x.device, workspace, stream,
        ("linear", x.device, x.shape, w.shape, x.dtype, out_dtype, reduce, w_is_nk, one_pass))
    _check(load_library().pike_linear_epilogue(_handle(x.device), _tensor(x), _tensor(w), _tensor(bias),
                                               _tensor(residual), _tensor(gamma), _tensor(beta), e,
                                               _tensor(out), ws_ptr, ws_bytes, _stream(stream)),
           "pike_linear_epilogue")
    return out


def pike_linear_softmax_shard_workspace(x, w, *, act="none", scale=1.0, w_is_nk=False) -> int:
    e = _epilogue(act, scale, "softmax", 0.0, torch.float32, FLAG_W_IS_NK if w_is_nk else 0)
    n = ctypes.c_size_t(0)
    _check(load_library().pike_linear_softmax_shard_workspace(_handle(x.device), _tensor(x), _tensor(w),
                                                              e, ctypes.byref(n)),
           "pike_linear_softmax_shard_workspace")
    return n.value


def pike_linear_softmax_shard_local(x, w, bias=None, *, act="none", scale=1.0, w_is_nk=False, out=None,
                                    row_stats=None, workspace=None, stream=None):
    """First half of a softmax whose columns are split over GPUs: this GPU's un-normalised slice
    out [M,N_r] fp32 and row_stats [M,2] fp32 = (max, sum exp) of the slice; see include/pike.h."""
    N = w.shape[0] if w_is_nk else w.shape[1]
    with _on(stream):
        if out is None:
            out = torch.empty((x.shape[0], N), dtype=torch.float32, device=x.device)
        if row_stats is None:
            row_stats = torch.empty((x.shape[0], 2), dtype=torch.float32, device=x.device)
    if row_stats.dtype != torch.float32 or not row_stats.is_cuda or not row_stats.is_contiguous() \
            or row_stats.numel() != 2 * x.shape[0]:
        raise TypeError("row_stats must be a contiguous CUDA float32 tensor of M pairs")
    e = _epilogue(act, scale, "softmax", 0.0, torch.float32, FLAG_W_IS_NK if w_is_nk else 0)
    ws, ws_ptr, ws_bytes = _workspace(
        lambda: pike_linear_softmax_shard_workspace(x, w, act=act, scale=scale, w_is_nk=w_is_nk), x.device, workspace,
        stream, ("shard", x.device, x.shape, w.shape, x.dtype, w_is_nk))
    _check(load_library().pike_linear_softmax_shard_local(_handle(x.device), _tensor(x), _tensor(w), _tensor(bias),
                                                          e, _tensor(out),
                                                          ctypes.c_void_p(row_stats.data_ptr()), ws_ptr, ws_bytes,
                                                          _stream(stream)),
           "pike_linear_softmax_shard_local")
    return out, row_stats


def pike_linear_softmax_shard_finish(out, all_stats, *, stream=None):
    """Second half: all_stats [R,M,2] fp32 (every GPU's row_stats, gathered shard-major) normalises this
    GPU's slice `out` in place; see include/pike.h."""
    if all_stats.dtype != torch.float32 or not all_stats.is_cuda or not all_stats.is_contiguous() \
            or all_stats.dim() != 3 or all_stats.shape[1] != out.shape[0] or all_stats.shape[2] != 2:
        raise TypeError("all_stats must be a contiguous CUDA float32 tensor [R, M, 2]")
    _check(load_library().pike_linear_softmax_shard_finish(_handle(out.device), _tensor(out),
                                                           ctypes.c_void_p(all_stats.data_ptr()),
                                                           int(all_stats.shape[0]), _stream(stream)),
           "pike_linear_softmax_shard_finish")
    return out


NOALLOC_MAX_PARTIALS = 262144


def pike_linear_softmax_noalloc(x, w, bias=None, *, out, act="none", scale=1.0, w_is_nk=False, stream=None):
    """out = softmax(scale*act(x @ w + bias)) with the scratch inside the library.

    For callers that cannot hand the library a workspace because they cannot allocate
    device memory.  `out` (fp32, [M,N]) must be supplied: this wrapper allocates nothing
    either.  M*ceil(N/256) is limited to NOALLOC_MAX_PARTIALS; calls on different
    streams must not overlap (they share one scratch array).  See include/pike.h."""
    e = _epilogue(act, scale, "softmax", 0.0, torch.float32, FLAG_W_IS_NK if w_is_nk else 0)
    _check(load_library().pike_linear_softmax_noalloc(_handle(x.device), _tensor(x), _tensor(w), _tensor(bias),
                                                      e, _tensor(out), _stream(stream)),
           "pike_linear_softmax_noalloc")
    return out


def pike_mlp_block_workspace(x, w1, *, act="gelu_tanh", eps=1e-5, w_is_nk=False) -> int:
    e = _epilogue(act, 1.0, "none", eps, x.dtype, FLAG_W_IS_NK if w_is_nk else 0)
    n = ctypes.c_size_t(0)
    _check(load_library().pike_mlp_block_workspace(_handle(x.device), _tensor(x), _tensor(w1), e,
                                                   ctypes.byref(n)), "pike_mlp_block_workspace")
    return n.value


def pike_mlp_block(x, gamma, beta, w1, b1, w2, b2, *, act="gelu_tanh", eps=1e-5, w_is_nk=False, out=None,
                   workspace=None, stream=None):
    """out = x + act(LayerNorm(x) @ w1 + b1) @ w2 + b2; see include/pike.h."""
    if out is None:
        with _on(stream):
            out = torch.empty_like(x)
    e = _epilogue(act, 1.0, "none", eps, x.dtype, FLAG_W_IS_NK if w_is_nk else 0)
    ws, ws_ptr, ws_bytes = _workspace(lambda: pike_mlp_block_workspace(x, w1, act=act, eps=eps, w_is_nk=w_is_nk),
                                      x.device, workspace, stream, ("mlp", x.device, x.shape, w1.shape, x.dtype, w_is_nk))
    _check(load_library().pike_mlp_block(_handle(x.device), _tensor(x), _tensor(gamma), _tensor(beta), _tensor(w1),
                                         _tensor(b1), _tensor(w2), _tensor(b2), e, _tensor(out),
                                         ws_ptr, ws_bytes, _stream(stream)), "pike_mlp_block")
    return out


def pike_attention_chain_workspace(q, *, scale, causal=True) -> int:
    e = _epilogue("none", scale, "none", 0.0, q.dtype, FLAG_CAUSAL if causal else 0)
    n = ctypes.c_size_t(0)
    _check(load_library().pike_attention_chain_workspace(_handle(q.device), _tensor(q), e,
                                                         ctypes.byref(n)), "pike_attention_chain_workspace")
    return n.value


def pike_attention_chain(q, k, v, *, scale, causal=True, out=None, stream=None):
    """out = softmax(scale * q k^T [+ causal mask]) v per (batch, head); see include/pike.h."""
    if out is None:
        with _on(stream):
            out = torch.empty_like(q)
    e = _epilogue("none", scale, "none", 0.0, q.dtype, FLAG_CAUSAL if causal else 0)
    _check(load_library().pike_attention_chain(_handle(q.device), _tensor(q), _tensor(k), _tensor(v),
                                               e, _tensor(out), None, 0, _stream(stream)),
           "pike_attention_chain")
    return out


def pike_attention_block_workspace(x, *, scale, causal=True, eps=1e-5, w_is_nk=False) -> int:
    e = _epilogue("none", scale, "none", eps, x.dtype, (FLAG_CAUSAL if causal else 0) | (FLAG_W_IS_NK if w_is_nk else 0))
    n = ctypes.c_size_t(0)
    _check(load_library().pike_attention_block_workspace(_handle(x.device), _tensor(x), e, ctypes.byref(n)),
           "pike_attention_block_workspace")
    return n.value


def pike_attention_block(x, gamma, beta, w_qkv, b_qkv, w_o, b_o, *, scale, causal=True, eps=1e-5, w_is_nk=False,
                         out=None, workspace=None, stream=None):
    """out = x + attention(LayerNorm(x) @ w_qkv + b_qkv) @ w_o + b_o for x [B,S,E]; see include/pike.h."""
    if out is None:
        with _on(stream):
            out = torch.empty_like(x)
    e = _epilogue("none", scale, "none", eps, x.dtype, (FLAG_CAUSAL if causal else 0) | (FLAG_W_IS_NK if w_is_nk else 0))
    ws, ws_ptr, ws_bytes = _workspace(
        lambda: pike_attention_block_workspace(x, scale=scale, causal=causal, eps=eps, w_is_nk=w_is_nk), x.device,
        workspace, stream)
    _check(load_library().pike_attention_block(_handle(x.device), _tensor(x), _tensor(gamma), _tensor(beta),
                                               _tensor(w_qkv), _tensor(b_qkv), _tensor(w_o), _tensor(b_o),
                                               e, _tensor(out), ws_ptr, ws_bytes, _stream(stream)),
           "pike_attention_block")
    return out


def pike_grouped_linear_epilogue(x, w, bias, residual, group_offsets, *, act="none", scale=1.0, out_dtype=None,
                                 w_is_nk=False, out=None, stream=None):
    """out[r] = scale*act(x[r] @ w[g] + bias[g]) + residual[r] for rows r of group g; group_offsets is a CUDA
    int32 tensor with G+1 entries.  See include/pike.h."""
    if group_offsets.dtype != torch.int32 or not group_offsets.is_cuda or not group_offsets.is_contiguous():
        raise TypeError("group_offsets must be a contiguous CUDA int32 tensor")
    out_dtype = (out.dtype if out is not None else x.dtype) if out_dtype is None else out_dtype
    N = w.shape[1] if w_is_nk else w.shape[2]
    if out is None:
        with _on(stream):
            out = torch.zeros((x.shape[0], N), dtype=out_dtype, device=x.device)
    e = _epilogue(act, scale, "none", 0.0, out_dtype, FLAG_W_IS_NK if w_is_nk else 0)
    _check(load_library().pike_grouped_linear_epilogue(_handle(x.device), _tensor(x), _tensor(w), _tensor(bias),
                                                       _tensor(residual), ctypes.c_void_p(group_offsets.data_ptr()),
                                                       e, _tensor(out), _stream(stream)),
           "pike_grouped_linear_epilogue")
    return out
