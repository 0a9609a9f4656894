"""ctypes binding of libhma.so: the same entry points as include/hma.h, argument marshalling only.

Tensors are torch CUDA tensors (torch provides device memory and streams); every step of the
path runs inside the library's kernels.  Loading fails loudly when the library has not been
built: there is no fallback of any kind.
"""
import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libhma.so")

HMA_OK = 0
HMA_ERR_INVALID_ARG, HMA_ERR_UNSUPPORTED_SHAPE, HMA_ERR_ALIGNMENT = 1, 2, 3
HMA_ERR_WORKSPACE_TOO_SMALL, HMA_ERR_CUDA = 4, 5
HMA_ERR_STATIC_LIMIT = 7
HMA_KV_BFP8, HMA_KV_BF16 = 0, 1
HMA_WIRE_TILE32, HMA_WIRE_ROWMAJOR, HMA_WIRE_BF16_ROWS = 0, 1, 2
HMA_OUT_BF16, HMA_OUT_F32 = 0, 1
HMA_KEYS_AS_QUERIES, HMA_KEYS_INTERLEAVED = 0, 1
HMA_FLAG_BAD_PAGE_ATTENTION, HMA_FLAG_BAD_PAGE_INGEST, HMA_FLAG_BAD_PAGE_DEQUANT, HMA_FLAG_WAIT_TIMEOUT = 1, 2, 4, 8
HMA_FLAG_BAD_VALUE_ENCODE, HMA_FLAG_EXPONENT_RANGE, HMA_FLAG_BAD_PLAN = 16, 32, 64


class CacheDesc(ctypes.Structure):
    _fields_ = [("num_layers", ctypes.c_int32), ("num_q_heads", ctypes.c_int32), ("num_kv_heads", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("page_tokens", ctypes.c_int32), ("bfp_block", ctypes.c_int32),
                ("num_pages", ctypes.c_int64), ("format", ctypes.c_int32), ("key_layout", ctypes.c_int32)]


class HmaError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        detail = ""
        if status == HMA_ERR_CUDA:
            detail = ": " + hma_last_cuda_error()
        super().__init__("%s: %s (status %d)%s" % (where, status_string(status), status, detail))


_lib = None


def lib():
    """The loaded C-ABI library.  Raises if libhma.so is missing (build it with build.py)."""
    global _lib
    if _lib is None:
        # HMA_LIBRARY selects another build of the same sources (the instrumented libhma_trace.so), nothing else
        path = os.environ.get("HMA_LIBRARY") or _LIB_PATH
        if not os.path.exists(path):
            raise ImportError("%s is not built: run `python -m paper_2606_29986_b200.build`" % os.path.basename(path))
        L = ctypes.CDLL(path)
        vp, i32, i64, f32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_float, ctypes.c_size_t
        L.hma_cache_layer_bytes.restype = sz
        L.hma_cache_layer_bytes.argtypes = [ctypes.POINTER(CacheDesc)]
        L.hma_cache_create.restype = i32
        L.hma_cache_create.argtypes = [ctypes.POINTER(CacheDesc), ctypes.POINTER(vp), ctypes.POINTER(vp)]
        L.hma_cache_destroy.restype = None
        L.hma_cache_destroy.argtypes = [vp]
        L.hma_kv_ingest_layer.restype = i32
        L.hma_kv_ingest_layer.argtypes = [vp, i32, vp, vp, i32, i32, i32, vp, i64, i64, vp]
        L.hma_kv_ingest_layer_shards.restype = i32
        L.hma_kv_ingest_layer_shards.argtypes = [vp, i32, i32, ctypes.POINTER(vp), ctypes.POINTER(vp), i32,
                                                 ctypes.POINTER(i32), ctypes.POINTER(i32), vp, i64, i64, vp]
        L.hma_kv_ingest_request_shards.restype = i32
        L.hma_kv_ingest_request_shards.argtypes = [vp, i32, ctypes.POINTER(vp), ctypes.POINTER(vp), sz, i32,
                                                   ctypes.POINTER(i32), ctypes.POINTER(i32), vp, i64, i64, vp]
        L.hma_decode_attention_workspace_bytes.restype = sz
        L.hma_decode_attention_workspace_bytes.argtypes = [ctypes.POINTER(CacheDesc), i32]
        L.hma_decode_attention_workspace_init.restype = i32
        L.hma_decode_attention_workspace_init.argtypes = [vp, sz, vp]
        L.hma_decode_attention.restype = i32
        L.hma_decode_attention.argtypes = [vp, i32, vp, vp, i32, vp, i32, vp, i32, f32, vp, sz, vp]
        L.hma_decode_attention_multi.restype = i32
        L.hma_decode_attention_multi.argtypes = [vp, i32, vp, vp, i32, vp, i32, vp, i32, i32, f32, vp, sz, vp]
        L.hma_decode_attention_plan_bytes.restype = sz
        L.hma_decode_attention_plan_bytes.argtypes = [i32]
        L.hma_decode_attention_plan.restype = i32
        L.hma_decode_attention_plan.argtypes = [vp, vp, i32, vp, i32, i32, vp, sz, vp]
        L.hma_decode_attention_planned.restype = i32
        L.hma_decode_attention_planned.argtypes = [vp, i32, vp, vp, i32, vp, i32, vp, i32, i32, f32, vp, vp, sz, vp]
        L.hma_decode_attention_static.restype = i32
        L.hma_decode_attention_static.argtypes = [vp, i32, vp, vp, i32, vp, i32, vp, i32, f32, vp]
        L.hma_decode_attention_static_limit_bytes.restype = sz
        L.hma_decode_attention_static_limit_bytes.argtypes = []
        L.hma_kv_read_probe.restype = i32
        L.hma_kv_read_probe.argtypes = [vp, i32, vp, i32, vp, i32, vp, sz, vp]
        L.hma_hbm_read_probe.restype = i32
        L.hma_hbm_read_probe.argtypes = [vp, sz, vp, vp]
        L.hma_hbm_copy_probe.restype = i32
        L.hma_hbm_copy_probe.argtypes = [vp, sz, vp, sz, vp]
        L.hma_attention_alu_probe.restype = i32
        L.hma_attention_alu_probe.argtypes = [vp, i32, vp, i32, vp, i32, vp, sz, vp]
        L.hma_decode_attention_mixed.restype = i32
        L.hma_decode_attention_mixed.argtypes = [vp, vp, i32, vp, vp, i32, vp, i32, vp, vp, i32, vp, i32, f32, vp, sz, vp]
        L.hma_decode_attention_mixed_planned.restype = i32
        L.hma_decode_attention_mixed_planned.argtypes = [vp, vp, i32, vp, vp, i32, vp, i32, vp, vp, i32, vp, i32, f32, vp, vp, vp, sz, vp]
        L.hma_decode_attention_simple.restype = i32
        L.hma_decode_attention_simple.argtypes = [vp, i32, vp, vp, i32, vp, i32, vp, i32, f32, vp]
        L.hma_bfp8_dequant_bf16.restype = i32
        L.hma_bfp8_dequant_bf16.argtypes = [vp, i32, i32, vp, i64, i64, vp, vp]
        L.hma_bfp8_dequant_bf16_naive.restype = i32
        L.hma_bfp8_dequant_bf16_naive.argtypes = [vp, i32, i32, vp, i64, i64, vp, vp]
        L.hma_bfp8_rebuild_request.restype = i32
        L.hma_bfp8_rebuild_request.argtypes = [vp, vp, i64, i64, vp, vp]
        L.hma_bfp8_encode_rows.restype = i32
        L.hma_bfp8_encode_rows.argtypes = [vp, vp, i32, i64, vp, vp]
        L.hma_bfp8_dequant_blocks_bf16.restype = i32
        L.hma_bfp8_dequant_blocks_bf16.argtypes = [vp, vp, i64, vp, vp]
        L.hma_error_flags.restype = i32
        L.hma_error_flags.argtypes = [vp, ctypes.POINTER(ctypes.c_uint32), vp]
        L.hma_status_string.restype = ctypes.c_char_p
        L.hma_status_string.argtypes = [i32]
        L.hma_last_cuda_error.restype = ctypes.c_char_p
        L.hma_last_cuda_error.argtypes = []
        L.hma_launch_count.restype = i64
        L.hma_launch_count.argtypes = []
        _lib = L
    return _lib


def status_string(status):
    return lib().hma_status_string(int(status)).decode()


def _check(status, where):
    if status != HMA_OK:
        raise HmaError(status, where)


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _ptr(t):
    return ctypes.c_void_p(t.data_ptr()) if t is not None else ctypes.c_void_p(0)


def make_desc(num_layers, num_q_heads, num_kv_heads, num_pages, fmt=HMA_KV_BFP8, head_dim=128, page_tokens=16, bfp_block=16,
              key_layout=0):
    return CacheDesc(num_layers, num_q_heads, num_kv_heads, head_dim, page_tokens, bfp_block, num_pages, fmt, key_layout)


def hma_cache_layer_bytes(desc):
    return int(lib().hma_cache_layer_bytes(ctypes.byref(desc)))


class KVCache:
    """Owns the torch uint8 layer buffers and the library's cache handle."""

    def __init__(self, desc, device="cuda", fill=None):
        self.desc = desc
        nbytes = hma_cache_layer_bytes(desc)
        if nbytes == 0:
            raise HmaError(HMA_ERR_UNSUPPORTED_SHAPE, "hma_cache_layer_bytes")
        self.layers = []
        for _ in range(desc.num_layers):
            t = torch.empty(nbytes, dtype=torch.uint8, device=device)
            if fill is not None:
                t.fill_(fill)
            self.layers.append(t)
        ptrs = (ctypes.c_void_p * desc.num_layers)(*[t.data_ptr() for t in self.layers])
        handle = ctypes.c_void_p()
        _check(lib().hma_cache_create(ctypes.byref(desc), ptrs, ctypes.byref(handle)), "hma_cache_create")
        self.handle = handle

    def close(self):
        if getattr(self, "handle", None):
            lib().hma_cache_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def hma_kv_ingest_layer(cache, layer, k_wire, v_wire, wire_layout, head_begin, head_count, page_ids,
                        token_begin, n_tokens, stream=None):
    _check(lib().hma_kv_ingest_layer(cache.handle, layer, _ptr(k_wire), _ptr(v_wire), wire_layout, head_begin,
                                     head_count, _ptr(page_ids), token_begin, n_tokens, _stream(stream)),
           "hma_kv_ingest_layer")


def hma_kv_ingest_layer_shards(cache, layer, k_wires, v_wires, wire_layout, head_begins, head_counts, page_ids,
                               token_begin, n_tokens, stream=None):
    """All producer shards of one layer in one launch; k_wires / v_wires are lists of tensors, one per shard."""
    n = len(k_wires)
    kp = (ctypes.c_void_p * n)(*[t.data_ptr() for t in k_wires])
    vp_ = (ctypes.c_void_p * n)(*[t.data_ptr() for t in v_wires])
    hb = (ctypes.c_int32 * n)(*head_begins)
    hc = (ctypes.c_int32 * n)(*head_counts)
    _check(lib().hma_kv_ingest_layer_shards(cache.handle, layer, n, kp, vp_, wire_layout, hb, hc, _ptr(page_ids),
                                            token_begin, n_tokens, _stream(stream)), "hma_kv_ingest_layer_shards")


def hma_kv_ingest_request_shards(cache, k_wires, v_wires, layer_stride_bytes, wire_layout, head_begins, head_counts, page_ids,
                                 token_begin, n_tokens, stream=None):
    """Every layer of the cache in one call: k_wires / v_wires are lists (one per shard) of layer 0's wire tensors; layer l's
    wire starts l * layer_stride_bytes further on in the same allocation."""
    n = len(k_wires)
    kp = (ctypes.c_void_p * n)(*[t.data_ptr() for t in k_wires])
    vp_ = (ctypes.c_void_p * n)(*[t.data_ptr() for t in v_wires])
    hb = (ctypes.c_int32 * n)(*head_begins)
    hc = (ctypes.c_int32 * n)(*head_counts)
    _check(lib().hma_kv_ingest_request_shards(cache.handle, n, kp, vp_, layer_stride_bytes, wire_layout, hb, hc, _ptr(page_ids),
                                              token_begin, n_tokens, _stream(stream)), "hma_kv_ingest_request_shards")


def hma_decode_attention_workspace_bytes(desc, batch):
    return int(lib().hma_decode_attention_workspace_bytes(ctypes.byref(desc), batch))


def hma_decode_attention_workspace_init(workspace, stream=None):
    """Zero-fills a workspace (required once before its first use; calls leave it ready for the next one)."""
    _check(lib().hma_decode_attention_workspace_init(_ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream)),
           "hma_decode_attention_workspace_init")


def new_workspace(desc, batch, device="cuda", copies=1):
    """A torch uint8 tensor sized for hma_decode_attention on `batch` sequences (`copies` = 2 for the two-cache call,
    each half rounded up to 256 bytes) and initialised through hma_decode_attention_workspace_init."""
    n = (hma_decode_attention_workspace_bytes(desc, batch) + 255) // 256 * 256
    ws = torch.empty(copies * n, dtype=torch.uint8, device=device)
    with torch.cuda.device(ws.device):
        hma_decode_attention_workspace_init(ws)
    return ws


def hma_decode_attention(cache, layer, q, out, block_table, context_lens, sm_scale, workspace, stream=None):
    out_dtype = HMA_OUT_F32 if out.dtype == torch.float32 else HMA_OUT_BF16
    _check(lib().hma_decode_attention(cache.handle, layer, _ptr(q), _ptr(out), out_dtype, _ptr(block_table),
                                      block_table.shape[1], _ptr(context_lens), q.shape[0], float(sm_scale),
                                      _ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream)),
           "hma_decode_attention")


def hma_decode_attention_multi(cache, layer, q, out, block_table, context_lens, sm_scale, workspace, stream=None):
    """q, out: [batch][q_len][Hq][128]; the last q_len cached tokens of each sequence are the query tokens (causal)."""
    out_dtype = HMA_OUT_F32 if out.dtype == torch.float32 else HMA_OUT_BF16
    _check(lib().hma_decode_attention_multi(cache.handle, layer, _ptr(q), _ptr(out), out_dtype, _ptr(block_table),
                                            block_table.shape[1], _ptr(context_lens), q.shape[0], q.shape[1], float(sm_scale),
                                            _ptr(workspace), workspace.numel() * workspace.element_size(), _stream(stream)),
           "hma_decode_attention_multi")


def hma_decode_attention_plan_bytes(rows):
    """Bytes of a plan for `rows` = sequences x query tokens per sequence."""
    return int(lib().hma_decode_attention_plan_bytes(rows))


def hma_decode_attention_plan(cache, block_table, context_lens, q_len=1, plan=None, stream=None):
    """Runs the attention kernel's set-up for this block table and these context lengths once and returns the plan (a uint8
    device tensor, reused when given); valid for every layer until the table or the lengths change."""
    batch = context_lens.shape[0]
    need = hma_decode_attention_plan_bytes(batch * q_len)
    if plan is None:
        plan = torch.empty(need, dtype=torch.uint8, device=context_lens.device)
    _check(lib().hma_decode_attention_plan(cache.handle, _ptr(block_table), block_table.shape[1], _ptr(context_lens), batch, q_len,
                                           _ptr(plan), plan.numel(), _stream(stream)), "hma_decode_attention_plan")
    return plan


def hma_decode_attention_planned(cache, layer, q, out, block_table, context_lens, sm_scale, plan, workspace, stream=None):
    """hma_decode_attention (q, out: [batch][Hq][128]) or hma_decode_attention_multi (q, out: [batch][q_len][Hq][128]) with the
    set-up taken from `plan` (hma_decode_attention_plan with the same table, lengths and q_len)."""
    out_dtype = HMA_OUT_F32 if out.dtype == torch.float32 else HMA_OUT_BF16
    q_len = q.shape[1] if q.dim() == 4 else 1
    _check(lib().hma_decode_attention_planned(cache.handle, layer, _ptr(q), _ptr(out), out_dtype, _ptr(block_table),
                                              block_table.shape[1], _ptr(context_lens), q.shape[0], q_len, float(sm_scale),
                                              _ptr(plan), _ptr(workspace), workspace.numel() * workspace.element_size(),
                                              _stream(stream)), "hma_decode_attention_planned")


def hma_decode_attention_static(cache, layer, q, out, block_table, context_lens, sm_scale, stream=None):
    """hma_decode_attention without a workspace argument, for callers that cannot allocate device memory.

    The scratch is an array inside the library (hma_decode_attention_static_limit_bytes() bytes on every GPU
    that loads it).  Raises HmaError(HMA_ERR_STATIC_LIMIT) when batch * kv heads is too large for it.  Calls
    on one device share the array: keep them on one stream.  Make the first call outside stream capture."""
    out_dtype = HMA_OUT_F32 if out.dtype == torch.float32 else HMA_OUT_BF16
    _check(lib().hma_decode_attention_static(cache.handle, layer, _ptr(q), _ptr(out), out_dtype, _ptr(block_table),
                                             block_table.shape[1], _ptr(context_lens), q.shape[0], float(sm_scale),
                                             _stream(stream)), "hma_decode_attention_static")


def hma_decode_attention_static_limit_bytes():
    return int(lib().hma_decode_attention_static_limit_bytes())


def hma_kv_read_probe(cache, layer, block_table, context_lens, workspace, stream=None):
    _check(lib().hma_kv_read_probe(cache.handle, layer, _ptr(block_table), block_table.shape[1], _ptr(context_lens),
                                   context_lens.shape[0], _ptr(workspace), workspace.numel() * workspace.element_size(),
                                   _stream(stream)), "hma_kv_read_probe")


def hma_attention_alu_probe(cache, layer, block_table, context_lens, workspace, stream=None):
    _check(lib().hma_attention_alu_probe(cache.handle, layer, _ptr(block_table), block_table.shape[1], _ptr(context_lens),
                                         context_lens.shape[0], _ptr(workspace), workspace.numel() * workspace.element_size(),
                                         _stream(stream)), "hma_attention_alu_probe")


def hma_hbm_read_probe(src, sink, stream=None):
    """Contiguous streaming read of the whole tensor `src` (a read-only memory ceiling); `sink` is a 4-byte device tensor."""
    _check(lib().hma_hbm_read_probe(_ptr(src), src.numel() * src.element_size(), _ptr(sink), _stream(stream)), "hma_hbm_read_probe")


def hma_hbm_copy_probe(src, read_bytes, dst, write_bytes, stream=None):
    """Streaming read of `read_bytes` of `src` mixed with a streaming write of `write_bytes` of `dst` (a copy-like ceiling)."""
    assert read_bytes <= src.numel() * src.element_size() and write_bytes <= dst.numel() * dst.element_size()
    _check(lib().hma_hbm_copy_probe(_ptr(src), read_bytes, _ptr(dst), write_bytes, _stream(stream)), "hma_hbm_copy_probe")


def hma_decode_attention_mixed(prefix, tail, layer, q, out, prefix_table, prefix_lens, tail_table, tail_lens, sm_scale,
                               workspace, stream=None):
    """Attention over a BFP8 prefix cache and a BF16 tail cache (see include/hma.h)."""
    out_dtype = HMA_OUT_F32 if out.dtype == torch.float32 else HMA_OUT_BF16
    _check(lib().hma_decode_attention_mixed(prefix.handle, tail.handle, layer, _ptr(q), _ptr(out), out_dtype,
                                            _ptr(prefix_table), prefix_table.shape[1], _ptr(prefix_lens),
                                            _ptr(tail_table), tail_table.shape[1], _ptr(tail_lens), q.shape[0],
                                            float(sm_scale), _ptr(workspace), workspace.numel() * workspace.element_size(),
                                            _stream(stream)), "hma_decode_attention_mixed")


def hma_decode_attention_mixed_planned(prefix, tail, layer, q, out, prefix_table, prefix_lens, tail_table, tail_lens, sm_scale,
                                       prefix_plan, tail_plan, workspace, stream=None):
    """hma_decode_attention_mixed with both launches' set-up taken from plans (one per cache, hma_decode_attention_plan)."""
    out_dtype = HMA_OUT_F32 if out.dtype == torch.float32 else HMA_OUT_BF16
    _check(lib().hma_decode_attention_mixed_planned(prefix.handle, tail.handle, layer, _ptr(q), _ptr(out), out_dtype,
                                                    _ptr(prefix_table), prefix_table.shape[1], _ptr(prefix_lens),
                                                    _ptr(tail_table), tail_table.shape[1], _ptr(tail_lens), q.shape[0],
                                                    float(sm_scale), _ptr(prefix_plan), _ptr(tail_plan), _ptr(workspace),
                                                    workspace.numel() * workspace.element_size(), _stream(stream)),
           "hma_decode_attention_mixed_planned")


def hma_decode_attention_simple(cache, layer, q, out, block_table, context_lens, sm_scale, stream=None):
    out_dtype = HMA_OUT_F32 if out.dtype == torch.float32 else HMA_OUT_BF16
    _check(lib().hma_decode_attention_simple(cache.handle, layer, _ptr(q), _ptr(out), out_dtype, _ptr(block_table),
                                             block_table.shape[1], _ptr(context_lens), q.shape[0], float(sm_scale),
                                             _stream(stream)), "hma_decode_attention_simple")


def hma_bfp8_dequant_bf16(cache, layer, which, page_ids, token_begin, n_tokens, out_bf16, stream=None):
    _check(lib().hma_bfp8_dequant_bf16(cache.handle, layer, which, _ptr(page_ids), token_begin, n_tokens,
                                       _ptr(out_bf16), _stream(stream)), "hma_bfp8_dequant_bf16")


def hma_bfp8_dequant_bf16_naive(cache, layer, which, page_ids, token_begin, n_tokens, out_bf16, stream=None):
    """Elementwise strawman of hma_bfp8_dequant_bf16 (same bits, one thread per element)."""
    _check(lib().hma_bfp8_dequant_bf16_naive(cache.handle, layer, which, _ptr(page_ids), token_begin, n_tokens,
                                             _ptr(out_bf16), _stream(stream)), "hma_bfp8_dequant_bf16_naive")


def hma_bfp8_rebuild_request(cache, page_ids, token_begin, n_tokens, out_bf16, stream=None):
    """Every layer, K and V, of one request in a single launch -> out_bf16 [layers][2][n_tokens][Hkv][128]."""
    _check(lib().hma_bfp8_rebuild_request(cache.handle, _ptr(page_ids), token_begin, n_tokens, _ptr(out_bf16), _stream(stream)),
           "hma_bfp8_rebuild_request")


def hma_bfp8_encode_rows(cache, x, wire_rowmajor, stream=None):
    """x: float32 or bfloat16 tensor [..., 128] -> ROWMAJOR BFP8 rows in wire_rowmajor (uint8 [..., 136])."""
    n_rows = x.numel() // 128
    _check(lib().hma_bfp8_encode_rows(cache.handle, _ptr(x), 1 if x.dtype == torch.bfloat16 else 0, n_rows,
                                      _ptr(wire_rowmajor), _stream(stream)), "hma_bfp8_encode_rows")


def hma_bfp8_dequant_blocks_bf16(exps, mants, n_blocks, out_bf16, stream=None):
    _check(lib().hma_bfp8_dequant_blocks_bf16(_ptr(exps), _ptr(mants), n_blocks, _ptr(out_bf16), _stream(stream)),
           "hma_bfp8_dequant_blocks_bf16")


def hma_error_flags(cache, stream=None):
    v = ctypes.c_uint32(0)
    _check(lib().hma_error_flags(cache.handle, ctypes.byref(v), _stream(stream)), "hma_error_flags")
    return int(v.value)


def hma_last_cuda_error():
    return lib().hma_last_cuda_error().decode()


def hma_launch_count():
    return int(lib().hma_launch_count())
