"""ctypes binding of include/san.h: same names, argument marshalling only.

Device arguments may be torch CUDA tensors (their ``data_ptr()`` is passed) or raw
integer addresses; ``stream`` may be a ``torch.cuda.Stream``, an integer handle or
None (torch's current stream).  Every function returns the library's status code;
``check`` turns a non-zero status into ``SanError``.

There is no CPU fallback: if the CUDA library has not been built, ``lib()`` raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libsan_b200.so")

SAN_OK = 0
SAN_ERR_NULL, SAN_ERR_SHAPE, SAN_ERR_POLICY, SAN_ERR_CAPACITY, SAN_ERR_DTYPE = 1, 2, 3, 4, 5
SAN_ERR_RANGE, SAN_ERR_CUDA, SAN_ERR_DEVICE_CHECK, SAN_ERR_TIMEOUT, SAN_ERR_UNSUPPORTED = 6, 7, 8, 9, 10
SAN_F32, SAN_BF16 = 0, 1
SAN_SELF, SAN_ENCDEC = 0, 1
SAN_MAX_LAYERS, SAN_MAX_BEAM = 64, 32

# every symbol include/san.h declares
EXPORTS = (
    "san_query_bytes", "san_create", "san_destroy",
    "san_policy_set_sizes", "san_policy_set_map", "san_policy_get_map",
    "san_cache_append", "san_attn_weights", "san_attn_apply", "san_aan_step", "san_seq_reset",
    "san_device_status", "san_status_string", "san_attn_weights_static", "san_decode_step",
    "san_decode_step_host", "san_step_kernel_select", "san_step_kernel_used", "san_full_block", "san_beam_reorder", "san_js_matrix", "san_block_similarity", "san_policy_search",
)


class san_config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in (
        "n_layers", "n_heads", "d_head", "max_sent", "beam", "max_tgt_len", "max_src_len",
        "dtype", "self_is_aan", "encdec_shared_context")]


class san_step_args(C.Structure):
    _fields_ = [
        ("d_q_self", C.c_void_p), ("d_k_new", C.c_void_p), ("d_v_new", C.c_void_p),
        ("d_seq_ids", C.c_void_p), ("d_pos", C.c_void_p), ("n_seqs", C.c_int32), ("max_len", C.c_int32),
        ("d_S_self", C.c_void_p), ("ld_t", C.c_int64), ("d_O_self", C.c_void_p),
        ("d_q_enc", C.c_void_p), ("d_sent_ids", C.c_void_p), ("d_src_lens", C.c_void_p),
        ("n_sent", C.c_int32), ("max_src", C.c_int32),
        ("d_S_enc", C.c_void_p), ("ld_s", C.c_int64), ("d_O_enc", C.c_void_p),
        ("d_x_aan", C.c_void_p), ("d_t", C.c_void_p),
    ]


class SanError(RuntimeError):
    def __init__(self, status: int, where: str = ""):
        self.status = status
        super().__init__(f"{where}: status {status} ({san_status_string(status)})")


_lib = None
_I32P = C.POINTER(C.c_int32)


def lib():
    """Load libsan_b200.so (built by ``paper_1906_11024_b200.build``); raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_1906_11024_b200.build` "
                          "(there is no CPU fallback)")
    L = C.CDLL(LIB_PATH)
    vp, i32, i64, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t
    L.san_query_bytes.argtypes = [C.POINTER(san_config), i32, i32, C.POINTER(sz), C.POINTER(sz)]
    L.san_create.argtypes = [C.POINTER(san_config), _I32P, i32, _I32P, i32, vp, sz, vp, sz, C.POINTER(vp)]
    L.san_destroy.argtypes = [vp]
    L.san_policy_set_sizes.argtypes = [vp, i32, _I32P, i32]
    L.san_policy_set_map.argtypes = [vp, i32, _I32P, i32]
    L.san_policy_get_map.argtypes = [vp, i32, _I32P, _I32P, _I32P]
    L.san_cache_append.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp, vp, i32, i32, vp]
    L.san_attn_weights.argtypes = [vp, i32, i32, vp, vp, vp, i32, i32, vp, i64, vp]
    L.san_attn_apply.argtypes = [vp, i32, i32, i32, i32, vp, i64, vp, vp, vp, i32, i32, vp, i32, vp]
    L.san_aan_step.argtypes = [vp, i32, i32, vp, vp, vp, i32, vp, vp]
    L.san_seq_reset.argtypes = [vp, vp, i32, vp]
    L.san_device_status.argtypes = [vp, _I32P, _I32P, vp]
    L.san_attn_weights_static.argtypes = [i32, i32, i32, vp, vp, i32, i32, vp, vp, i32, i32, vp, i64, vp, vp]
    L.san_decode_step.argtypes = [vp, C.POINTER(san_step_args), vp]
    L.san_step_kernel_select.argtypes = [vp, i32, i32, i32, i32, i32, i32]
    L.san_step_kernel_used.argtypes = [vp, _I32P, _I32P]
    L.san_decode_step_host.argtypes = [vp, C.POINTER(san_step_args), C.POINTER(san_step_args), vp]
    L.san_full_block.argtypes = [i32, i32, i32, i32, vp, vp, vp, vp, i32, i32, i32, vp, i64, vp, vp]
    L.san_beam_reorder.argtypes = [vp, vp, vp, vp, i32, i32, vp]
    L.san_js_matrix.argtypes = [i32, vp, i64, i64, i32, i32, vp, vp, vp]
    L.san_block_similarity.argtypes = [C.POINTER(C.c_double), i32, i32, i32, C.POINTER(C.c_double)]
    L.san_policy_search.argtypes = [C.POINTER(C.c_double), i32, C.c_double, _I32P, _I32P]
    L.san_status_string.argtypes = [i32]
    L.san_status_string.restype = C.c_char_p
    for name in EXPORTS:
        if name != "san_status_string":
            getattr(L, name).restype = i32
    _lib = L
    return L


def _ptr(x) -> Optional[int]:
    if x is None:
        return None
    if isinstance(x, int):
        return x
    return x.data_ptr()          # torch tensor


def _stream(s) -> Optional[int]:
    if s is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(s, int):
        return s
    return s.cuda_stream


def _i32_array(v: Sequence[int]):
    return (C.c_int32 * len(v))(*[int(x) for x in v])


def check(status: int, where: str = "san") -> None:
    if status != SAN_OK:
        raise SanError(status, where)


def san_status_string(status: int) -> str:
    return lib().san_status_string(int(status)).decode()


def san_query_bytes(cfg: san_config, n_self_blocks: int, n_encdec_blocks: int):
    """Returns (status, cache_bytes, workspace_bytes)."""
    cb, wb = C.c_size_t(0), C.c_size_t(0)
    rc = lib().san_query_bytes(C.byref(cfg), n_self_blocks, n_encdec_blocks, C.byref(cb), C.byref(wb))
    return rc, cb.value, wb.value


def san_create(cfg: san_config, self_sizes, encdec_sizes, d_cache, cache_bytes, d_workspace, workspace_bytes):
    """Returns (status, ctx handle)."""
    h = C.c_void_p(None)
    ss = _i32_array(self_sizes) if self_sizes is not None else None
    es = _i32_array(encdec_sizes) if encdec_sizes is not None else None
    rc = lib().san_create(C.byref(cfg), ss, len(self_sizes) if self_sizes is not None else 0,
                          es, len(encdec_sizes) if encdec_sizes is not None else 0,
                          _ptr(d_cache), cache_bytes, _ptr(d_workspace), workspace_bytes, C.byref(h))
    return rc, h.value


def san_destroy(ctx) -> int:
    return lib().san_destroy(ctx)


def san_policy_set_sizes(ctx, kind: int, sizes) -> int:
    return lib().san_policy_set_sizes(ctx, kind, _i32_array(sizes), len(sizes))


def san_policy_set_map(ctx, kind: int, block_of_layer) -> int:
    return lib().san_policy_set_map(ctx, kind, _i32_array(block_of_layer), len(block_of_layer))


def san_policy_get_map(ctx, kind: int):
    """Returns (status, block_of_layer list, first_layer_of_block list)."""
    bol = (C.c_int32 * SAN_MAX_LAYERS)(*([-1] * SAN_MAX_LAYERS))   # the library fills n_layers entries
    first = (C.c_int32 * SAN_MAX_LAYERS)()
    nb = C.c_int32(0)
    rc = lib().san_policy_get_map(ctx, kind, bol, first, C.byref(nb))
    if rc != SAN_OK:
        return rc, [], []
    return rc, [b for b in bol if b >= 0], list(first[:nb.value])


def san_cache_append(ctx, kind, layer_begin, layer_end, d_k_new, d_v_new, d_ids, d_pos, d_nrows,
                     n_items, rows_per_item=1, stream=None) -> int:
    return lib().san_cache_append(ctx, kind, layer_begin, layer_end, _ptr(d_k_new), _ptr(d_v_new), _ptr(d_ids),
                                  _ptr(d_pos), _ptr(d_nrows), n_items, rows_per_item, _stream(stream))


def san_attn_weights(ctx, kind, block, d_q, d_ids, d_lens, n_items, max_len, d_S, ld_s, stream=None) -> int:
    return lib().san_attn_weights(ctx, kind, block, _ptr(d_q), _ptr(d_ids), _ptr(d_lens), n_items, max_len,
                                  _ptr(d_S), ld_s, _stream(stream))


def san_attn_apply(ctx, kind, block, layer_begin, layer_end, d_S, ld_s, d_ids, d_pos_begin, d_pos_end,
                   n_items, max_len, d_out, accumulate=0, stream=None) -> int:
    return lib().san_attn_apply(ctx, kind, block, layer_begin, layer_end, _ptr(d_S), ld_s, _ptr(d_ids),
                                _ptr(d_pos_begin), _ptr(d_pos_end), n_items, max_len, _ptr(d_out),
                                int(accumulate), _stream(stream))


def san_aan_step(ctx, layer_begin, layer_end, d_x, d_ids, d_t, n_items, d_out, stream=None) -> int:
    return lib().san_aan_step(ctx, layer_begin, layer_end, _ptr(d_x), _ptr(d_ids), _ptr(d_t), n_items,
                              _ptr(d_out), _stream(stream))


def san_seq_reset(ctx, d_seq_ids, n, stream=None) -> int:
    """Zero the running sums of the listed sequences in every layer (average attention only)."""
    return lib().san_seq_reset(ctx, _ptr(d_seq_ids), n, _stream(stream))


def san_device_status(ctx, stream=None):
    """Returns (status, first_error, detail[4]).  Synchronises the stream."""
    fe = C.c_int32(0)
    det = (C.c_int32 * 4)()
    rc = lib().san_device_status(ctx, C.byref(fe), det, _stream(stream))
    return rc, fe.value, list(det)


def san_attn_weights_static(dtype, n_heads, n_queries, d_q, d_K, max_ids, cap_len, d_ids, d_lens, n_items,
                            max_len, d_S, ld_s, d_status=None, stream=None) -> int:
    """The weights step without a context or workspace, for callers that cannot allocate
    device memory (see include/san.h).  ``d_K`` is the device address of a key plane."""
    return lib().san_attn_weights_static(dtype, n_heads, n_queries, _ptr(d_q), _ptr(d_K), max_ids, cap_len,
                                         _ptr(d_ids), _ptr(d_lens), n_items, max_len, _ptr(d_S), ld_s,
                                         _ptr(d_status), _stream(stream))


def san_decode_step(ctx, *, d_q_self=None, d_k_new=None, d_v_new=None, d_seq_ids=None, d_pos=None, n_seqs=0,
                    max_len=0, d_S_self=None, ld_t=0, d_O_self=None, d_q_enc=None, d_sent_ids=None,
                    d_src_lens=None, n_sent=0, max_src=0, d_S_enc=None, ld_s=0, d_O_enc=None, d_x_aan=None,
                    d_t=None, stream=None) -> int:
    """One whole decode step in one launch (see include/san.h)."""
    a = san_step_args(_ptr(d_q_self), _ptr(d_k_new), _ptr(d_v_new), _ptr(d_seq_ids), _ptr(d_pos), n_seqs, max_len,
                      _ptr(d_S_self), ld_t, _ptr(d_O_self), _ptr(d_q_enc), _ptr(d_sent_ids), _ptr(d_src_lens),
                      n_sent, max_src, _ptr(d_S_enc), ld_s, _ptr(d_O_enc), _ptr(d_x_aan), _ptr(d_t))
    return lib().san_decode_step(ctx, C.byref(a), _stream(stream))


def san_step_kernel_select(ctx, which=0, spans_log2=-1, heads_per_unit=4, tile_pos=64, layers_per_unit=0, grab_mult=1) -> int:
    """Choose the kernel behind san_decode_step (0 automatic, 1 per-warp, 2 team pipeline) and its cut."""
    return lib().san_step_kernel_select(ctx, which, spans_log2, heads_per_unit, tile_pos, layers_per_unit, grab_mult)


def san_step_kernel_used(ctx):
    """Returns (status, kernel of the last san_decode_step: 0 none / 1 per-warp / 2 team, [heads per unit self, enc-dec])."""
    which = C.c_int32(0)
    rpu = (C.c_int32 * 2)()
    rc = lib().san_step_kernel_used(ctx, C.byref(which), rpu)
    return rc, which.value, list(rpu)


def san_beam_reorder(ctx, d_sent_ids, d_parent, d_lens, n_sent, max_len=0, stream=None) -> int:
    """Beam-search cache reorder: every beam slot takes over its parent's cached rows, in place."""
    return lib().san_beam_reorder(ctx, _ptr(d_sent_ids), _ptr(d_parent), _ptr(d_lens), n_sent, max_len,
                                  _stream(stream))


def san_js_matrix(n_layers, d_S, layer_stride, ld_s, n_rows, n_heads, d_lens, d_js, stream=None) -> int:
    """Pairwise Jensen-Shannon divergence of the layers' attention weights into d_js [M][M] float64."""
    return lib().san_js_matrix(n_layers, _ptr(d_S), layer_stride, ld_s, n_rows, n_heads, _ptr(d_lens), _ptr(d_js),
                               _stream(stream))


def _f64_matrix(js, n_layers):
    flat = [float(x) for row in js for x in row] if not isinstance(js, (bytes, bytearray)) else js
    if len(flat) != n_layers * n_layers:
        raise ValueError("js must be n_layers x n_layers")
    return (C.c_double * len(flat))(*flat)


def san_block_similarity(js, n_layers, m, n):
    """Eq. 6 on a host matrix (nested sequences).  Returns (status, sim)."""
    out = C.c_double(0.0)
    rc = lib().san_block_similarity(_f64_matrix(js, n_layers), n_layers, m, n, C.byref(out))
    return rc, out.value


def san_policy_search(js, n_layers, theta):
    """Section 3.3 search on a host matrix.  Returns (status, block sizes bottom-up)."""
    sizes = (C.c_int32 * max(n_layers, 1))()
    nb = C.c_int32(0)
    rc = lib().san_policy_search(_f64_matrix(js, n_layers), n_layers, float(theta), sizes, C.byref(nb))
    return rc, list(sizes[:nb.value]) if rc == SAN_OK else []


def step_args(**kw) -> san_step_args:
    """A san_step_args block from keyword arguments named like its fields (tensors, addresses or None)."""
    a = san_step_args()
    for name, _ in san_step_args._fields_:
        v = kw.pop(name, None)
        if name in ("n_seqs", "max_len", "n_sent", "max_src", "ld_t", "ld_s"):
            setattr(a, name, int(v or 0))
        else:
            setattr(a, name, _ptr(v))
    if kw:
        raise TypeError(f"unknown san_step_args fields: {sorted(kw)}")
    return a


def san_decode_step_host(ctx, host: san_step_args, dev: san_step_args, stream=None) -> int:
    """san_decode_step with host-resident inputs and outputs: copies in, one launch, copies out."""
    return lib().san_decode_step_host(ctx, C.byref(host), C.byref(dev), _stream(stream))


def san_full_block(dtype, n_heads, n_layers, causal, d_q, d_k, d_v, d_lens, n_seq, cap_len, max_len, d_S, ld_s,
                   d_out, stream=None) -> int:
    """Full-sequence shared attention: S once per block, applied to every layer's values."""
    return lib().san_full_block(dtype, n_heads, n_layers, int(causal), _ptr(d_q), _ptr(d_k), _ptr(d_v), _ptr(d_lens),
                                n_seq, cap_len, max_len, _ptr(d_S), ld_s, _ptr(d_out), _stream(stream))
