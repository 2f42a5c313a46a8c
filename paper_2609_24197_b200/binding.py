"""Thin ctypes binding over libhspec.so: argument marshalling only.

Every function has the name of the C entry point it wraps (see include/hspec.h) and takes torch
tensors that already live on the CUDA device; torch is used for device memory and streams, nothing
else.  There is no fallback: if the library is missing or no CUDA device is present, calls raise.
"""
import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libhspec.so")

HSPEC_MAX_LAYERS = 16
HSPEC_BF16, HSPEC_F32, HSPEC_I32, HSPEC_F16 = 0, 1, 2, 3
_DT = {torch.bfloat16: 0, torch.float32: 1, torch.int32: 2, torch.float16: 3}

EXPORTS = [
    "hspec_init", "hspec_workspace_bytes", "hspec_load_weights", "hspec_draft_block", "hspec_destroy",
    "hspec_last_error", "hspec_get_stats", "hspec_set_profiling", "hspec_get_profile",
    "hspec_debug_wait_selftest", "hspec_clear_status", "hspec_op_gemm", "hspec_gemm_workspace_bytes",
    "hspec_op_lm_head_argmax", "hspec_op_lm_head_argmax_noalloc", "hspec_op_rmsnorm", "hspec_op_mamba_scan", "hspec_scan_workspace_bytes", "hspec_op_qk_norm_rope",
    "hspec_op_attention", "hspec_attention_workspace_bytes", "hspec_debug_gather_kv", "hspec_op_swiglu",
    "hspec_op_accept", "hspec_op_token_probs", "hspec_op_markov_head", "hspec_markov_workspace_bytes",
    "hspec_op_kv_inject_write", "hspec_op_device_status",
]


class HSpecError(RuntimeError):
    pass


class hspec_config(C.Structure):
    _fields_ = [
        ("D", C.c_int32), ("n_fuse", C.c_int32), ("r", C.c_int32), ("L", C.c_int32),
        ("has_attn", C.c_int32 * HSPEC_MAX_LAYERS), ("kv_slot", C.c_int32 * HSPEC_MAX_LAYERS),
        ("n_slots", C.c_int32), ("Di", C.c_int32), ("P", C.c_int32), ("N", C.c_int32), ("G", C.c_int32),
        ("d_conv", C.c_int32), ("dt_rank", C.c_int32), ("Hq", C.c_int32), ("Hkv", C.c_int32), ("dh", C.c_int32),
        ("rope_theta", C.c_float), ("window", C.c_int32), ("qk_norm", C.c_int32), ("F", C.c_int32),
        ("V", C.c_int32), ("V_draft", C.c_int32), ("mask_id", C.c_int32), ("rms_eps", C.c_float), ("page_size", C.c_int32),
        ("max_batch", C.c_int32), ("max_k", C.c_int32), ("max_pages_per_req", C.c_int32),
        ("markov_rank", C.c_int32), ("act_bf16", C.c_int32),
    ]


class hspec_tensor(C.Structure):
    _fields_ = [("name", C.c_char_p), ("data", C.c_void_p), ("dtype", C.c_int32), ("ndim", C.c_int32),
                ("shape", C.c_int64 * 2)]


class hspec_step(C.Structure):
    _fields_ = [
        ("B", C.c_int32), ("k", C.c_int32), ("page_table", C.c_void_p), ("page_table_stride", C.c_int32),
        ("ctx_lens", C.c_void_p), ("max_ctx", C.c_int32), ("last_hidden", C.c_void_p), ("last_token", C.c_void_p),
        ("k_pools", C.POINTER(C.c_void_p)), ("v_pools", C.POINTER(C.c_void_p)), ("num_pages", C.c_int64),
        ("stream", C.c_void_p), ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t),
    ]


class hspec_out(C.Structure):
    _fields_ = [("draft_ids", C.c_void_p), ("logits", C.c_void_p), ("hidden", C.c_void_p)]


class hspec_stats(C.Structure):
    _fields_ = [("kernel_launches", C.c_uint64), ("device_status", C.c_uint32), ("launches_last_step", C.c_uint32),
                ("attn_rescales", C.c_uint32), ("f16_range_events", C.c_uint32), ("bad_inputs", C.c_uint32)]


class hspec_prof_entry(C.Structure):
    _fields_ = [("name", C.c_char * 40), ("ms", C.c_float), ("flops", C.c_double), ("bytes", C.c_double),
                ("io_bytes", C.c_double)]


_lib = None


def load_library(path=None):
    """dlopen libhspec.so (built by paper_2609_24197_b200.build).  Raises if it is missing."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    path = path or LIB_PATH
    if not os.path.exists(path):
        raise HSpecError(f"{path} not found: build it with `python -m paper_2609_24197_b200.build` "
                         "(there is no fallback path)")
    lib = C.CDLL(path)
    lib.hspec_init.argtypes = [C.POINTER(hspec_config), C.POINTER(C.c_void_p)]
    lib.hspec_workspace_bytes.argtypes = [C.POINTER(hspec_config)]
    lib.hspec_workspace_bytes.restype = C.c_size_t
    lib.hspec_load_weights.argtypes = [C.c_void_p, C.POINTER(hspec_tensor), C.c_int32]
    lib.hspec_draft_block.argtypes = [C.c_void_p, C.POINTER(hspec_step), C.POINTER(hspec_out)]
    lib.hspec_destroy.argtypes = [C.c_void_p]
    lib.hspec_last_error.argtypes = [C.c_void_p]
    lib.hspec_last_error.restype = C.c_char_p
    lib.hspec_get_stats.argtypes = [C.c_void_p, C.POINTER(hspec_stats)]
    lib.hspec_set_profiling.argtypes = [C.c_void_p, C.c_int32]
    lib.hspec_debug_wait_selftest.argtypes = [C.c_void_p, C.c_int32, C.c_void_p]
    lib.hspec_clear_status.argtypes = [C.c_void_p]
    lib.hspec_get_profile.argtypes = [C.c_void_p, C.POINTER(hspec_prof_entry), C.c_int32]
    vp, i32, i64, f32, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_float, C.c_size_t
    lib.hspec_op_gemm.argtypes = [vp, vp, i32, vp, i32, i32, i32, i64, i32, i32, i32, vp, sz, vp]
    lib.hspec_gemm_workspace_bytes.argtypes = [i32, i32, i32]
    lib.hspec_gemm_workspace_bytes.restype = sz
    lib.hspec_op_lm_head_argmax.argtypes = [vp, vp, i32, vp, vp, i32, i32, i32, vp, sz, vp]
    lib.hspec_op_lm_head_argmax_noalloc.argtypes = [vp, vp, i32, vp, vp, i32, i32, i32, vp]
    lib.hspec_op_rmsnorm.argtypes = [vp, vp, vp, i32, i32, f32, vp]
    lib.hspec_op_accept.argtypes = [vp, vp, vp, vp, i32, i32, vp]
    lib.hspec_op_token_probs.argtypes = [vp, i64, vp, vp, i32, i32, vp]
    lib.hspec_op_markov_head.argtypes = [vp, i64, vp, vp, i32, vp, vp, vp, i32, i32, i32, i32, i32, vp, sz, vp]
    lib.hspec_markov_workspace_bytes.argtypes = [i32, i32, i32]
    lib.hspec_markov_workspace_bytes.restype = sz
    lib.hspec_op_kv_inject_write.argtypes = [vp, vp, vp, vp, vp, i32, vp, vp, i32, i32, i32, i32, f32, f32, i32, vp]
    lib.hspec_op_mamba_scan.argtypes = [vp, i64, vp, vp, vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, i32, vp, sz, vp]
    lib.hspec_scan_workspace_bytes.argtypes = [i32, i32, i32, i32, i32]
    lib.hspec_scan_workspace_bytes.restype = sz
    lib.hspec_op_qk_norm_rope.argtypes = [vp, vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, f32, f32, i32, vp]
    lib.hspec_op_attention.argtypes = [vp, vp, vp, vp, vp, i64, vp, i32, vp, i32, vp, i32, i32, i32, i32, i32, i32, i32,
                                       i32, vp, sz, vp]
    lib.hspec_attention_workspace_bytes.argtypes = [i32, i32, i32, i32, i32, i32, i32, i32]
    lib.hspec_attention_workspace_bytes.restype = sz
    lib.hspec_debug_gather_kv.argtypes = [vp, vp, i32, i32, i32, i32, vp, vp]
    lib.hspec_op_swiglu.argtypes = [vp, vp, i32, i32, vp]
    lib.hspec_op_device_status.argtypes = [C.POINTER(C.c_uint32), i32]
    if path == LIB_PATH:
        _lib = lib
    return lib


def _check(rc, handle=None, what=""):
    if rc != 0:
        msg = load_library().hspec_last_error(handle)
        raise HSpecError(f"{what} failed ({rc}): {msg.decode() if msg else ''}")


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _ptr(t, dtype=None):
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise HSpecError("expected a contiguous CUDA tensor")
    if dtype is not None and t.dtype != dtype:
        raise HSpecError(f"expected dtype {dtype}, got {t.dtype}")
    return C.c_void_p(t.data_ptr())


def make_config(cfg, max_batch=None, max_k=None, max_pages_per_req=None):
    """dict of shapes (see synth.configs) -> hspec_config."""
    c = hspec_config()
    for name in ("D", "n_fuse", "r", "L", "n_slots", "Di", "P", "N", "G", "d_conv", "dt_rank", "Hq", "Hkv", "dh",
                 "window", "qk_norm", "F", "V", "mask_id", "page_size"):
        setattr(c, name, int(cfg[name]))
    c.V_draft = int(cfg.get("V_draft", 0))
    c.markov_rank = int(cfg.get("markov_rank", 0))
    c.act_bf16 = int(cfg.get("act_bf16", 0))
    c.rope_theta = float(cfg["rope_theta"])
    c.rms_eps = float(cfg["rms_eps"])
    for l in range(int(cfg["L"])):
        c.has_attn[l] = int(cfg["has_attn"][l])
        c.kv_slot[l] = int(cfg["kv_slot"][l])
    c.max_batch = int(max_batch if max_batch is not None else cfg.get("B", 1))
    c.max_k = int(max_k if max_k is not None else cfg.get("k", 16))
    c.max_pages_per_req = int(max_pages_per_req if max_pages_per_req is not None else 1)
    return c


def hspec_init(config):
    h = C.c_void_p()
    _check(load_library().hspec_init(C.byref(config), C.byref(h)), None, "hspec_init")
    return h


def hspec_workspace_bytes(config):
    return int(load_library().hspec_workspace_bytes(C.byref(config)))


def hspec_load_weights(handle, tensors):
    """tensors: dict name -> CUDA tensor (bf16 matrices, fp32 vectors).  Borrowed, not copied."""
    arr = (hspec_tensor * len(tensors))()
    keep = []
    for i, (name, t) in enumerate(tensors.items()):
        if not t.is_cuda or not t.is_contiguous():
            raise HSpecError(f"weight {name} must be a contiguous CUDA tensor")
        bname = name.encode()
        keep.append(bname)
        arr[i].name = bname
        arr[i].data = t.data_ptr()
        arr[i].dtype = {torch.bfloat16: HSPEC_BF16, torch.float32: HSPEC_F32, torch.int32: HSPEC_I32}[t.dtype]
        arr[i].ndim = t.dim()
        for j in range(t.dim()):
            arr[i].shape[j] = t.shape[j]
    _check(load_library().hspec_load_weights(handle, arr, len(tensors)), handle, "hspec_load_weights")


def hspec_draft_block(handle, page_table, ctx_lens, last_hidden, last_token, k, k_pools, v_pools, workspace,
                      draft_ids, logits=None, hidden=None, max_ctx=0):
    """Enqueue one block-parallel draft step on the current torch stream (no synchronisation)."""
    B = int(ctx_lens.shape[0])
    step = hspec_step()
    step.B, step.k = B, int(k)
    step.page_table = _ptr(page_table, torch.int32)
    step.page_table_stride = int(page_table.shape[1])
    step.ctx_lens = _ptr(ctx_lens, torch.int32)
    step.max_ctx = int(max_ctx)
    step.last_hidden = _ptr(last_hidden, torch.bfloat16)
    step.last_token = _ptr(last_token, torch.int32)
    n = len(k_pools)
    kp = (C.c_void_p * max(n, 1))(*[p.data_ptr() for p in k_pools])
    vp = (C.c_void_p * max(n, 1))(*[p.data_ptr() for p in v_pools])
    step.k_pools, step.v_pools = kp, vp
    step.num_pages = int(k_pools[0].shape[0]) if n else 0
    step.stream = _stream()
    step.workspace = _ptr(workspace)
    step.workspace_bytes = workspace.numel() * workspace.element_size()
    out = hspec_out()
    out.draft_ids = _ptr(draft_ids, torch.int32)
    out.logits = _ptr(logits, torch.float32)
    out.hidden = _ptr(hidden, torch.float32)
    _check(load_library().hspec_draft_block(handle, C.byref(step), C.byref(out)), handle, "hspec_draft_block")


def hspec_destroy(handle):
    _check(load_library().hspec_destroy(handle), None, "hspec_destroy")


def hspec_get_stats(handle):
    s = hspec_stats()
    rc = load_library().hspec_get_stats(handle, C.byref(s))
    return dict(kernel_launches=int(s.kernel_launches), device_status=int(s.device_status),
                launches_last_step=int(s.launches_last_step), attn_rescales=int(s.attn_rescales),
                f16_range_events=int(s.f16_range_events), bad_inputs=int(s.bad_inputs), rc=rc)


def hspec_op_device_status(clear=False):
    """Status block of the handle-less hspec_op_* calls on the current device (synchronises it)."""
    w = (C.c_uint32 * 4)()
    rc = load_library().hspec_op_device_status(w, int(bool(clear)))
    return dict(device_status=int(w[0]), attn_rescales=int(w[1]), f16_range_events=int(w[2]), bad_inputs=int(w[3]), rc=rc)


def hspec_debug_wait_selftest(handle, limit_ms=100):
    _check(load_library().hspec_debug_wait_selftest(handle, int(limit_ms), _stream()), handle, "hspec_debug_wait_selftest")


def hspec_clear_status(handle):
    _check(load_library().hspec_clear_status(handle), handle, "hspec_clear_status")


def hspec_set_profiling(handle, on):
    _check(load_library().hspec_set_profiling(handle, int(on)), handle, "hspec_set_profiling")


def hspec_get_profile(handle, max_entries=512):
    """Per-launch (name, ms, flops, bytes) of the last step; needs hspec_set_profiling(handle, True) before it."""
    arr = (hspec_prof_entry * max_entries)()
    n = load_library().hspec_get_profile(handle, arr, max_entries)
    if n < 0:
        _check(n, handle, "hspec_get_profile")
    return [dict(name=arr[i].name.decode(), ms=float(arr[i].ms), flops=float(arr[i].flops), bytes=float(arr[i].bytes),
                 io_bytes=float(arr[i].io_bytes)) for i in range(n)]


# ----------------------------------------------------------------------------- single operations

def hspec_gemm_workspace_bytes(M, n_out, K):
    return int(load_library().hspec_gemm_workspace_bytes(M, n_out, K))


def hspec_op_gemm(x, W, y, accumulate=False, splits=0, workspace=None):
    M, K = x.shape
    n_out = W.shape[0]
    ws_bytes = workspace.numel() * workspace.element_size() if workspace is not None else 0
    _check(load_library().hspec_op_gemm(
        _ptr(x), _ptr(W, x.dtype), _DT[x.dtype], _ptr(y), M, n_out, K, y.stride(0),
        _DT[y.dtype], int(accumulate), int(splits),
        _ptr(workspace), ws_bytes, _stream()), None, "hspec_op_gemm")


def hspec_op_lm_head_argmax(x, W, ids, logits, workspace):
    M, K = x.shape
    _check(load_library().hspec_op_lm_head_argmax(
        _ptr(x), _ptr(W, x.dtype), _DT[x.dtype], _ptr(ids, torch.int32), _ptr(logits, torch.float32),
        M, W.shape[0], K, _ptr(workspace), workspace.numel() * workspace.element_size(), _stream()),
        None, "hspec_op_lm_head_argmax")


def hspec_op_lm_head_argmax_noalloc(x, W, ids, logits=None):
    """LM head + arg-max without any device allocation: the scratch is a fixed array inside the library (M <= 512 rows,
    V <= 262144).  For hosts that cannot allocate while drafting (pre-reserved HBM, no allocator handle)."""
    M, K = x.shape
    _check(load_library().hspec_op_lm_head_argmax_noalloc(
        _ptr(x), _ptr(W, x.dtype), _DT[x.dtype], _ptr(ids, torch.int32), _ptr(logits, torch.float32), M, W.shape[0], K,
        _stream()), None, "hspec_op_lm_head_argmax_noalloc")


def hspec_op_accept(p_target, p_draft, alpha, n_accept):
    """App. A acceptance rule on device fp32 [B, k] arrays -> n_accept int32 [B]."""
    B, k = p_target.shape
    _check(load_library().hspec_op_accept(_ptr(p_target, torch.float32), _ptr(p_draft, torch.float32), _ptr(alpha, torch.float32),
                                          _ptr(n_accept, torch.int32), B, k, _stream()), None, "hspec_op_accept")


def hspec_op_token_probs(logits, ids, p):
    """p[m] = softmax(logits[m])[ids[m]] for fp32 logits [M, V]."""
    M, V = logits.shape
    _check(load_library().hspec_op_token_probs(_ptr(logits, torch.float32), V, _ptr(ids, torch.int32), _ptr(p, torch.float32),
                                               M, V, _stream()), None, "hspec_op_token_probs")


def hspec_markov_workspace_bytes(B, Vd, r):
    return int(load_library().hspec_markov_workspace_bytes(B, Vd, r))


def hspec_op_markov_head(logits, W_in, W_out, last_token, id_map, ids, B, k, write_logits, workspace):
    """Sequential first-order correction of the block's fp32 logits [B*k, Vd] (Sec. 3.3.3) -> token ids [B*k]."""
    Vd, r = W_out.shape
    _check(load_library().hspec_op_markov_head(
        _ptr(logits, torch.float32), logits.shape[1], _ptr(W_in), _ptr(W_out, W_in.dtype), _DT[W_in.dtype],
        _ptr(last_token, torch.int32), _ptr(id_map, torch.int32), _ptr(ids, torch.int32), B, k, Vd, r, int(write_logits),
        _ptr(workspace), workspace.numel() * workspace.element_size(), _stream()), None, "hspec_op_markov_head")


def hspec_op_kv_inject_write(kv, k_norm_w, req, pos, page_table, k_pool, v_pool, theta, eps, k_norm=True):
    """The comparison drafters' cache write: fp32 rows [T, 2, Hkv, dh] -> bf16 paged pools, in place (Sec. 2.2)."""
    T, _, Hkv, dh = kv.shape
    _check(load_library().hspec_op_kv_inject_write(
        _ptr(kv, torch.float32), _ptr(k_norm_w, torch.float32), _ptr(req, torch.int32), _ptr(pos, torch.int32),
        _ptr(page_table, torch.int32), page_table.shape[1], _ptr(k_pool, torch.bfloat16), _ptr(v_pool, torch.bfloat16), T, Hkv,
        dh, k_pool.shape[1], float(theta), float(eps), int(bool(k_norm)), _stream()), None, "hspec_op_kv_inject_write")


def hspec_op_rmsnorm(x, w, y, eps):
    _check(load_library().hspec_op_rmsnorm(_ptr(x, torch.float32), _ptr(w, torch.float32), _ptr(y, torch.float16),
                                           x.shape[0], x.shape[1], float(eps), _stream()), None, "hspec_op_rmsnorm")


def hspec_scan_workspace_bytes(B, k, Di, N, G):
    return int(load_library().hspec_scan_workspace_bytes(B, k, Di, N, G))


def hspec_op_mamba_scan(zxbcdt, dt_raw, s_init, conv_w, conv_b, dt_bias, A_log, Dskip, y_gated, B, k, Di, P, N, G,
                        d_conv, workspace=None):
    _check(load_library().hspec_op_mamba_scan(
        _ptr(zxbcdt, torch.float32), zxbcdt.stride(0), _ptr(dt_raw, torch.float32), _ptr(s_init, torch.float16),
        _ptr(conv_w, torch.float32), _ptr(conv_b, torch.float32), _ptr(dt_bias, torch.float32),
        _ptr(A_log, torch.float32), _ptr(Dskip, torch.float32), _ptr(y_gated, torch.float32),
        B, k, Di, P, N, G, d_conv, _ptr(workspace), workspace.numel() * workspace.element_size() if workspace is not None else 0,
        _stream()), None, "hspec_op_mamba_scan")


def hspec_op_qk_norm_rope(qkv, q_norm_w, k_norm_w, ctx_lens, q, kb, vb, B, k, Hq, Hkv, dh, theta, eps, qk_norm=1):
    _check(load_library().hspec_op_qk_norm_rope(
        _ptr(qkv, torch.float32), _ptr(q_norm_w, torch.float32), _ptr(k_norm_w, torch.float32),
        _ptr(ctx_lens, torch.int32), _ptr(q, torch.bfloat16), _ptr(kb, torch.bfloat16), _ptr(vb, torch.bfloat16),
        B, k, Hq, Hkv, dh, float(theta), float(eps), int(qk_norm), _stream()), None, "hspec_op_qk_norm_rope")


def hspec_attention_workspace_bytes(B, k, Hq, Hkv, dh, max_ctx, window=0, chunk_tokens=0):
    return int(load_library().hspec_attention_workspace_bytes(B, k, Hq, Hkv, dh, max_ctx, window, chunk_tokens))


def hspec_op_attention(q, kb, vb, k_pool, v_pool, page_table, ctx_lens, max_ctx, o, B, k, Hq, Hkv, dh, page_size,
                       window, chunk_tokens, workspace):
    _check(load_library().hspec_op_attention(
        _ptr(q, torch.bfloat16), _ptr(kb, torch.bfloat16), _ptr(vb, torch.bfloat16), _ptr(k_pool, torch.bfloat16),
        _ptr(v_pool, torch.bfloat16), int(k_pool.shape[0]), _ptr(page_table, torch.int32), int(page_table.shape[1]),
        _ptr(ctx_lens, torch.int32), int(max_ctx), _ptr(o, torch.float16), B, k, Hq, Hkv, dh, page_size, window,
        chunk_tokens, _ptr(workspace), workspace.numel() * workspace.element_size(), _stream()),
        None, "hspec_op_attention")


def hspec_debug_gather_kv(pool, page_table_row, ctx_len, dst):
    _, page_size, Hkv, dh = pool.shape
    _check(load_library().hspec_debug_gather_kv(_ptr(pool, torch.bfloat16), _ptr(page_table_row, torch.int32),
                                                int(ctx_len), page_size, Hkv, dh, _ptr(dst, torch.bfloat16),
                                                _stream()), None, "hspec_debug_gather_kv")


def hspec_op_swiglu(gu, h):
    _check(load_library().hspec_op_swiglu(_ptr(gu, torch.float32), _ptr(h, torch.float16), gu.shape[0], h.shape[1],
                                          _stream()), None, "hspec_op_swiglu")


# ----------------------------------------------------------------------------- convenience wrapper

class Drafter:
    """Owns a handle, its borrowed weights and a workspace; `draft` is one call of hspec_draft_block."""

    def __init__(self, cfg, weights, max_batch, max_k, max_ctx):
        if not torch.cuda.is_available():
            raise HSpecError("no CUDA device: the H-Spec draft step has no CPU path")
        self.cfg = cfg
        self.weights = weights if cfg.get("act_bf16", 0) else None     # bf16 mode borrows the GEMM matrices: keep them alive
        ps = cfg["page_size"]
        self.max_pages = max(1, (max_ctx + ps - 1) // ps)
        self.config = make_config(cfg, max_batch, max_k, self.max_pages)
        self.handle = hspec_init(self.config)
        hspec_load_weights(self.handle, weights)
        nbytes = hspec_workspace_bytes(self.config)
        self.workspace = torch.empty(nbytes + 1024, dtype=torch.uint8, device="cuda")
        off = (-self.workspace.data_ptr()) % 1024
        self.workspace = self.workspace[off:off + nbytes]

    def draft(self, batch, k, want_logits=False, want_hidden=False, max_ctx=0):
        B = batch["ctx_lens"].shape[0]
        dev = batch["ctx_lens"].device
        ids = torch.empty((B, k), dtype=torch.int32, device=dev)
        v_out = self.cfg.get("V_draft", 0) or self.cfg["V"]
        logits = torch.empty((B, k, v_out), dtype=torch.float32, device=dev) if want_logits else None
        hidden = torch.empty((B, k, self.cfg["D"]), dtype=torch.float32, device=dev) if want_hidden else None
        hspec_draft_block(self.handle, batch["page_table"], batch["ctx_lens"], batch["last_hidden"],
                          batch["last_token"], k, batch["k_pools"], batch["v_pools"], self.workspace, ids, logits,
                          hidden, max_ctx=max_ctx)
        return ids, logits, hidden

    def stats(self):
        return hspec_get_stats(self.handle)

    def close(self):
        if self.handle is not None:
            hspec_destroy(self.handle)
            self.handle = None
