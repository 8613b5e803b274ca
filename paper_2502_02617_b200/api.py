"""Thin ctypes binding of the C ABI declared in include/polarquant.h.

Argument marshalling only: every step of the path (rotation, polar transform, quantisation,
packing, decode attention) runs inside the CUDA library.  PyTorch supplies device memory and
streams.  There is no CPU fallback: if the shared library is missing the import of any entry
point raises.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import c_char_p, c_double, c_float, c_int32, c_int64, c_uint64, c_void_p, POINTER

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpolarquant.so")

OK = 0
ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_ALIGNMENT, ERR_CAPACITY = -1, -2, -3, -4
ERR_CUDA, ERR_TIMEOUT, ERR_NONFINITE, ERR_EMPTY, ERR_SCRATCH = -5, -6, -7, -8, -9
DTYPE_F32, DTYPE_BF16 = 0, 1
STATUS_WORDS = 4
N_CENTROIDS, N_BOUNDARIES = 28, 24
N_LEVELS, HIST_MAX_BINS = 4, 1024
DEFAULT_BITS = (4, 2, 2, 2)

# name -> (restype, argtypes); must list every symbol of include/polarquant.h
_SIGNATURES = {
    "pq_status_string": (c_char_p, [c_int32]),
    "pq_last_cuda_error": (c_char_p, []),
    "pq_token_block": (c_int32, []),
    "pq_make_rotation": (c_int32, [c_int32, c_uint64, c_void_p]),
    "pq_make_structured_rotation": (c_int32, [c_int32, c_int32, c_void_p, c_void_p]),
    "pq_fit_codebooks": (c_int32, [POINTER(c_int32), POINTER(c_double), POINTER(c_double)]),
    "pq_angle_histograms": (c_int32, [c_int32, c_int32, c_void_p, c_void_p, c_void_p, c_int32, c_int64, c_int64, c_int32,
                                      c_int32, c_void_p, c_void_p, c_void_p]),
    "pq_fit_codebooks_from_histograms": (c_int32, [c_void_p, c_int32, c_void_p, c_void_p, c_void_p]),
    "pq_tables_bytes": (c_int64, []),
    "pq_build_tables": (c_int32, [POINTER(c_double), POINTER(c_double), c_void_p]),
    "pq_cache_bytes": (c_int64, [c_int32, c_int32, c_int32, c_int32]),
    "pq_workspace_bytes": (c_int64, [c_int32, c_int32, c_int32, c_int32, c_int32]),
    "pq_encode_kv": (c_int32, [c_int32, c_int32, c_void_p, c_void_p, c_void_p, c_void_p, c_int32, c_int64, c_int64,
                               c_void_p, c_int32, c_int32, c_void_p, c_void_p, c_int32, c_void_p, c_void_p]),
    "pq_append_kv": (c_int32, [c_int32, c_int32, c_void_p, c_void_p, c_void_p, c_void_p, c_int32, c_int32,
                               c_void_p, c_void_p, c_int32, c_void_p, c_void_p]),
    "pq_decode_attention": (c_int32, [c_int32, c_int32, c_int32, c_void_p, c_void_p, c_void_p, c_int32, c_void_p,
                                      c_void_p, c_int32, c_int32, c_int32, c_float, c_void_p, c_void_p, c_void_p,
                                      c_void_p]),
    "pq_multi_query_attention": (c_int32, [c_int32, c_int32, c_int32, c_void_p, c_void_p, c_void_p, c_int32, c_void_p,
                                           c_void_p, c_int32, c_int32, c_int32, c_int32, c_float, c_void_p, c_void_p,
                                           c_void_p, c_void_p]),
    "pq_static_scratch_bytes": (c_int64, []),
    "pq_decode_attention_static": (c_int32, [c_int32, c_int32, c_int32, c_void_p, c_void_p, c_void_p, c_int32, c_void_p,
                                             c_void_p, c_int32, c_int32, c_int32, c_float, c_void_p, c_void_p,
                                             c_void_p]),
    "pq_debug_fail_next_wait": (c_int32, [c_int32]),
    "pq_unpack_codes": (c_int32, [c_int32, c_int32, c_void_p, c_int32, c_int32, c_int32, c_void_p, c_void_p, c_void_p]),
    "pq_dequant_kv": (c_int32, [c_int32, c_int32, c_void_p, c_void_p, c_void_p, c_int32, c_int32, c_int32, c_void_p,
                                c_void_p]),
    "pq_decode_attention_lse": (c_int32, [c_int32, c_int32, c_int32, c_void_p, c_void_p, c_void_p, c_int32, c_void_p,
                                          c_void_p, c_int32, c_int32, c_void_p, c_int32, c_float, c_void_p, c_void_p,
                                          c_void_p, c_void_p, c_void_p]),
    "pq_merge_attention": (c_int32, [c_int32, c_int32, c_int32, c_int32, c_void_p, c_int32, c_void_p, c_void_p, c_int32,
                                     c_void_p, c_void_p, c_void_p]),
    "pq_tail_attention": (c_int32, [c_int32, c_int32, c_int32, c_void_p, c_int32, c_void_p, c_void_p, c_int32, c_void_p,
                                    c_int32, c_int32, c_int32, c_float, c_void_p, c_void_p, c_void_p, c_void_p]),
    "pq_general_sizes": (c_int32, [c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]),
    "pq_general_fit_codebooks": (c_int32, [c_void_p, c_void_p, c_void_p]),
    "pq_general_cache_bytes": (c_int64, [c_void_p, c_int32, c_int32, c_int32]),
    "pq_general_encode_kv": (c_int32, [c_void_p, c_int32, c_void_p, c_void_p, c_void_p, c_void_p, c_int32, c_int64, c_int64,
                                       c_void_p, c_int32, c_int32, c_void_p, c_void_p, c_int32, c_void_p, c_void_p]),
    "pq_general_decode_attention": (c_int32, [c_void_p, c_int32, c_int32, c_void_p, c_void_p, c_void_p, c_int32, c_void_p,
                                              c_void_p, c_int32, c_int32, c_float, c_void_p, c_void_p, c_void_p]),
    "pq_general_unpack_codes": (c_int32, [c_void_p, c_int32, c_void_p, c_int32, c_int32, c_int32, c_void_p, c_void_p,
                                          c_void_p]),
    "pq_general_dequant_kv": (c_int32, [c_void_p, c_int32, c_void_p, c_void_p, c_void_p, c_int32, c_int32, c_int32,
                                        c_void_p, c_void_p]),
    "pq_paged_cache_bytes": (c_int64, [c_int32, c_int32, c_int32, c_int32]),
    "pq_encode_kv_paged": (c_int32, [c_int32, c_int32, c_void_p, c_void_p, c_void_p, c_void_p, c_int32, c_int64, c_int64,
                                     c_void_p, c_int32, c_int32, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]),
    "pq_append_kv_paged": (c_int32, [c_int32, c_int32, c_void_p, c_void_p, c_void_p, c_void_p, c_int32, c_int32,
                                     c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]),
    "pq_decode_attention_paged": (c_int32, [c_int32, c_int32, c_int32, c_void_p, c_void_p, c_void_p, c_int32, c_void_p,
                                            c_void_p, c_int32, c_void_p, c_int32, c_float, c_void_p, c_void_p, c_void_p,
                                            c_void_p]),
    "pq_multi_query_attention_paged": (c_int32, [c_int32, c_int32, c_int32, c_void_p, c_void_p, c_void_p, c_int32, c_void_p,
                                                 c_void_p, c_int32, c_int32, c_void_p, c_int32, c_float, c_void_p,
                                                 c_void_p, c_void_p, c_void_p]),
    "pq_unpack_codes_paged": (c_int32, [c_int32, c_int32, c_void_p, c_int32, c_void_p, c_int32, c_void_p, c_void_p, c_void_p]),
    "pq_dequant_kv_paged": (c_int32, [c_int32, c_int32, c_void_p, c_void_p, c_void_p, c_int32, c_void_p, c_int32, c_void_p,
                                      c_void_p]),
}


class Paging(ctypes.Structure):
    """struct pq_paging of include/polarquant.h."""
    _fields_ = [("page_table_dev", c_void_p), ("page_tokens", c_int32), ("pages_per_seq", c_int32), ("n_pages", c_int32)]

    @classmethod
    def of(cls, page_table: torch.Tensor, page_tokens: int, n_pages: int) -> "Paging":
        assert page_table.dtype == torch.int32 and page_table.is_contiguous() and page_table.dim() == 2
        return cls(page_table.data_ptr(), page_tokens, page_table.shape[1], n_pages)

_lib = None


class PolarQuantError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        detail = lib().pq_last_cuda_error().decode() if status == ERR_CUDA else ""
        super().__init__(f"{where}: {status_string(status)} ({status})" + (f": {detail}" if detail else ""))


def lib() -> ctypes.CDLL:
    """Load the CUDA library (built in-tree by __graft_entry__.build()).  Raises if absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -c 'import __graft_entry__ as g; g.build()'`"
                              " -- there is no CPU fallback")
        handle = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(handle, name)
            fn.restype, fn.argtypes = res, args
        _lib = handle
    return _lib


def status_string(status: int) -> str:
    return lib().pq_status_string(int(status)).decode()


def _check(status: int, where: str):
    if status != OK:
        raise PolarQuantError(int(status), where)


def _ptr(t) -> int:
    return 0 if t is None else t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return DTYPE_F32
    if t.dtype == torch.bfloat16:
        return DTYPE_BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def token_block() -> int:
    return int(lib().pq_token_block())


def pq_make_rotation(d: int, seed: int) -> torch.Tensor:
    """Seeded random rotation S (float32 CPU tensor [d, d], y = x @ S)."""
    S = torch.empty((d, d), dtype=torch.float32)
    _check(lib().pq_make_rotation(d, seed, S.data_ptr()), "pq_make_rotation")
    return S



ROTATION_IDENTITY, ROTATION_HADAMARD = 0, 1


def pq_make_structured_rotation(d: int, kind: int, signs=None) -> torch.Tensor:
    """S = I, or diag(signs) . H_d / sqrt(d) with the Sylvester Hadamard matrix; `signs`: d values of +1 / -1 (int8)."""
    S = torch.empty((d, d), dtype=torch.float32)
    sg = None if signs is None else torch.as_tensor(signs).to(torch.int8).contiguous()
    if sg is not None and sg.numel() != d:
        raise ValueError("signs must have head_dim entries")
    _check(lib().pq_make_structured_rotation(d, kind, 0 if sg is None else sg.data_ptr(), S.data_ptr()), "pq_make_structured_rotation")
    return S

def pq_fit_codebooks(bits=DEFAULT_BITS):
    """Analytic Lloyd-Max codebooks: (centroids float64[28], boundaries float64[24]) CPU tensors."""
    cen = torch.empty(N_CENTROIDS, dtype=torch.float64)
    bnd = torch.empty(N_BOUNDARIES, dtype=torch.float64)
    arr = (c_int32 * 4)(*bits)
    _check(lib().pq_fit_codebooks(arr, ctypes.cast(cen.data_ptr(), POINTER(c_double)),
                                  ctypes.cast(bnd.data_ptr(), POINTER(c_double))), "pq_fit_codebooks")
    return cen, bnd


def pq_angle_histograms(S, K, V, hist, status, stream=None):
    """Add the angles of the rows of K and V [total_tokens, Hkv, d] to hist (int64 device tensor [4, n_bins])."""
    total, n_kv_heads, d = K.shape
    assert V.shape == K.shape and V.dtype == K.dtype and K.stride(2) == 1 and V.stride() == K.stride()
    assert hist.dtype == torch.int64 and hist.is_contiguous() and hist.shape[0] == N_LEVELS
    _check(lib().pq_angle_histograms(d, n_kv_heads, _ptr(S), _ptr(K), _ptr(V), _dtype_code(K), K.stride(0), K.stride(1),
                                     total, hist.shape[1], _ptr(hist), _ptr(status), _stream(stream)),
           "pq_angle_histograms")


def pq_fit_codebooks_from_histograms(hist: torch.Tensor, init_centroids: torch.Tensor = None):
    """k-means on the binned angles (hist: int64 CPU tensor [4, n_bins]): (centroids float64[28], boundaries
    float64[24]) CPU tensors, started from init_centroids (None: the analytic codebook)."""
    hist = hist.to(torch.int64).cpu().contiguous()
    init = None if init_centroids is None else init_centroids.to(torch.float64).cpu().contiguous()
    cen = torch.empty(N_CENTROIDS, dtype=torch.float64)
    bnd = torch.empty(N_BOUNDARIES, dtype=torch.float64)
    _check(lib().pq_fit_codebooks_from_histograms(hist.data_ptr(), hist.shape[1], _ptr(init), cen.data_ptr(),
                                                  bnd.data_ptr()), "pq_fit_codebooks_from_histograms")
    return cen, bnd


def pq_build_tables(centroids: torch.Tensor, boundaries: torch.Tensor) -> torch.Tensor:
    """Compiled device tables as a CPU uint8 tensor; move it to the GPU unchanged."""
    centroids = centroids.to(torch.float64).contiguous()
    boundaries = boundaries.to(torch.float64).contiguous()
    out = torch.zeros(int(lib().pq_tables_bytes()), dtype=torch.uint8)
    _check(lib().pq_build_tables(ctypes.cast(centroids.data_ptr(), POINTER(c_double)),
                                 ctypes.cast(boundaries.data_ptr(), POINTER(c_double)), out.data_ptr()),
           "pq_build_tables")
    return out


def pq_cache_bytes(d: int, batch: int, n_kv_heads: int, capacity: int) -> int:
    n = int(lib().pq_cache_bytes(d, batch, n_kv_heads, capacity))
    if n < 0:
        raise PolarQuantError(n, "pq_cache_bytes")
    return n


def pq_workspace_bytes(d: int, batch: int, n_q_heads: int, n_kv_heads: int, max_len: int) -> int:
    n = int(lib().pq_workspace_bytes(d, batch, n_q_heads, n_kv_heads, max_len))
    if n < 0:
        raise PolarQuantError(n, "pq_workspace_bytes")
    return n


def pq_encode_kv(S, tables, K, V, cu_seqlens, cache, cache_lens, capacity, status, stream=None):
    """Encode packed ragged K, V [total_tokens, Hkv, d] into `cache`; cache_lens advances."""
    total, n_kv_heads, d = K.shape
    assert V.shape == K.shape and V.dtype == K.dtype and K.stride(2) == 1 and V.stride() == K.stride()
    _check(lib().pq_encode_kv(d, n_kv_heads, _ptr(S), _ptr(tables), _ptr(K), _ptr(V), _dtype_code(K), K.stride(0),
                              K.stride(1), _ptr(cu_seqlens), cu_seqlens.numel() - 1, total, _ptr(cache),
                              _ptr(cache_lens), capacity, _ptr(status), _stream(stream)), "pq_encode_kv")


def pq_append_kv(S, tables, k_new, v_new, cache, cache_lens, capacity, status, stream=None):
    """Append one token per sequence: k_new, v_new [B, Hkv, d] contiguous."""
    batch, n_kv_heads, d = k_new.shape
    assert k_new.is_contiguous() and v_new.is_contiguous() and v_new.shape == k_new.shape
    _check(lib().pq_append_kv(d, n_kv_heads, _ptr(S), _ptr(tables), _ptr(k_new), _ptr(v_new), _dtype_code(k_new),
                              batch, _ptr(cache), _ptr(cache_lens), capacity, _ptr(status), _stream(stream)),
           "pq_append_kv")


def pq_decode_attention(S, tables, q, cache, cache_lens, n_kv_heads, capacity, max_len, scale, out, workspace,
                        status, stream=None):
    """Eq. 3 for one query per sequence: q, out [B, Hq, d] (bf16 or f32)."""
    batch, n_q_heads, d = q.shape
    assert q.is_contiguous() and out.is_contiguous() and out.shape == q.shape and out.dtype == q.dtype
    _check(lib().pq_decode_attention(d, n_q_heads, n_kv_heads, _ptr(S), _ptr(tables), _ptr(q), _dtype_code(q),
                                     _ptr(cache), _ptr(cache_lens), batch, capacity, max_len, float(scale),
                                     _ptr(out), _ptr(workspace), _ptr(status), _stream(stream)),
           "pq_decode_attention")


def pq_multi_query_attention(S, tables, q, cache, cache_lens, n_kv_heads, capacity, max_len, scale, out, workspace,
                             status, stream=None):
    """Eq. 2 / 3 for the last n_q positions of every sequence: q, out [B, n_q, Hq, d]; query j sees the cached
    tokens before and at its own position.  `workspace` must hold pq_workspace_bytes(d, B * n_q, Hq, Hkv, max_len)."""
    batch, n_q, n_q_heads, d = q.shape
    assert q.is_contiguous() and out.is_contiguous() and out.shape == q.shape and out.dtype == q.dtype
    _check(lib().pq_multi_query_attention(d, n_q_heads, n_kv_heads, _ptr(S), _ptr(tables), _ptr(q), _dtype_code(q),
                                          _ptr(cache), _ptr(cache_lens), batch, n_q, capacity, max_len, float(scale),
                                          _ptr(out), _ptr(workspace), _ptr(status), _stream(stream)),
           "pq_multi_query_attention")


def pq_static_scratch_bytes() -> int:
    return int(lib().pq_static_scratch_bytes())


def pq_decode_attention_static(S, tables, q, cache, cache_lens, n_kv_heads, capacity, max_len, scale, out, status,
                               stream=None):
    """pq_decode_attention on the library's built-in scratch buffer, for callers that cannot allocate
    or pass a workspace.  Raises PolarQuantError(ERR_SCRATCH) if the problem needs more scratch than
    pq_static_scratch_bytes().  Calls on one device share that buffer: keep them stream-ordered."""
    batch, n_q_heads, d = q.shape
    assert q.is_contiguous() and out.is_contiguous() and out.shape == q.shape and out.dtype == q.dtype
    _check(lib().pq_decode_attention_static(d, n_q_heads, n_kv_heads, _ptr(S), _ptr(tables), _ptr(q), _dtype_code(q),
                                            _ptr(cache), _ptr(cache_lens), batch, capacity, max_len, float(scale),
                                            _ptr(out), _ptr(status), _stream(stream)), "pq_decode_attention_static")


def pq_debug_fail_next_wait(which: int) -> None:
    """Test support: 1 = the next tensor-core encode launch, 2 = the next head_dim-128 decode-attention
    launch runs its give-up path (PQ_ERR_TIMEOUT in status word 0); 0 disarms."""
    _check(lib().pq_debug_fail_next_wait(int(which)), "pq_debug_fail_next_wait")


def pq_unpack_codes(d, n_kv_heads, cache, batch, capacity, n_tokens, stream=None):
    """Canonical codes uint8 [B, Hkv, 2, n_tokens, 15d/16] and radii fp16 [B, Hkv, 2, n_tokens, d/16]."""
    codes = torch.empty((batch, n_kv_heads, 2, n_tokens, 15 * d // 16), dtype=torch.uint8, device=cache.device)
    radii = torch.empty((batch, n_kv_heads, 2, n_tokens, d // 16), dtype=torch.float16, device=cache.device)
    _check(lib().pq_unpack_codes(d, n_kv_heads, _ptr(cache), batch, capacity, n_tokens, _ptr(codes), _ptr(radii),
                                 _stream(stream)), "pq_unpack_codes")
    return codes, radii


def pq_dequant_kv(d, n_kv_heads, S, tables, cache, batch, capacity, n_tokens, stream=None):
    """DeQuant of the first n_tokens positions: float32 [B, Hkv, 2, n_tokens, d] (original basis)."""
    out = torch.empty((batch, n_kv_heads, 2, n_tokens, d), dtype=torch.float32, device=cache.device)
    _check(lib().pq_dequant_kv(d, n_kv_heads, _ptr(S), _ptr(tables), _ptr(cache), batch, capacity, n_tokens,
                               _ptr(out), _stream(stream)), "pq_dequant_kv")
    return out


def pq_decode_attention_lse(S, tables, q, cache, cache_lens, n_kv_heads, capacity, max_len, scale, out, lse, workspace,
                            status, paging=None, stream=None):
    """pq_decode_attention that also writes lse float32 [B, Hq] (log of the softmax denominator); `paging`: a Paging
    for a paged cache, else the contiguous cache of `capacity` tokens."""
    batch, n_q_heads, d = q.shape
    assert q.is_contiguous() and out.is_contiguous() and out.shape == q.shape and out.dtype == q.dtype
    assert lse.dtype == torch.float32 and lse.is_contiguous() and lse.shape == (batch, n_q_heads)
    _check(lib().pq_decode_attention_lse(d, n_q_heads, n_kv_heads, _ptr(S), _ptr(tables), _ptr(q), _dtype_code(q),
                                         _ptr(cache), _ptr(cache_lens), batch, capacity,
                                         None if paging is None else ctypes.addressof(paging), max_len, float(scale),
                                         _ptr(out), _ptr(lse), _ptr(workspace), _ptr(status), _stream(stream)),
           "pq_decode_attention_lse")


def pq_merge_attention(parts_out, parts_lse, out, status, lse_out=None, stream=None):
    """Merge partial attentions: parts_out [P, B, Hq, d] (float32 or bf16), parts_lse float32 [P, B, Hq] -> out [B, Hq, d]."""
    n_parts, batch, n_q_heads, d = parts_out.shape
    assert parts_out.is_contiguous() and parts_lse.is_contiguous() and out.is_contiguous()
    assert parts_lse.shape == (n_parts, batch, n_q_heads) and parts_lse.dtype == torch.float32 and out.shape == parts_out.shape[1:]
    _check(lib().pq_merge_attention(d, n_q_heads, batch, n_parts, _ptr(parts_out), _dtype_code(parts_out), _ptr(parts_lse),
                                    _ptr(out), _dtype_code(out), _ptr(lse_out), _ptr(status), _stream(stream)),
           "pq_merge_attention")
    return out


def pq_tail_attention(q, k_tail, v_tail, tail_lens, scale, out, lse, status, n_splits=1, stream=None):
    """Exact attention of q [B, Hq, d] over an uncompressed window k_tail, v_tail [B, T, Hkv, d] (first tail_lens[b] rows),
    as n_splits partial attentions: out [n_splits, B, Hq, d] (or [B, Hq, d] for one), lse [n_splits, B, Hq]."""
    batch, n_q_heads, d = q.shape
    assert k_tail.is_contiguous() and v_tail.is_contiguous() and k_tail.shape == v_tail.shape and k_tail.dtype == v_tail.dtype
    assert k_tail.shape[0] == batch and k_tail.shape[3] == d and q.is_contiguous() and out.is_contiguous() and out.dtype == q.dtype
    assert out.numel() == n_splits * q.numel() and (lse is None or lse.numel() == n_splits * batch * n_q_heads)
    _check(lib().pq_tail_attention(d, n_q_heads, k_tail.shape[2], _ptr(q), _dtype_code(q), _ptr(k_tail), _ptr(v_tail),
                                   _dtype_code(k_tail), _ptr(tail_lens), batch, k_tail.shape[1], n_splits, float(scale),
                                   _ptr(out), _ptr(lse), _ptr(status), _stream(stream)), "pq_tail_attention")


def sharded_decode_attention(cache, q, dist, group=None, scale=None, stream=None):
    """Decode attention over a cache whose tokens are sharded over the ranks of `group` (each rank's `cache` holds its
    own tokens): local partial attention with its log-sum-exp in float32, one all-gather of [B, Hq, d + 1] floats per
    rank, merge on every rank.  Returns out in q's dtype."""
    from .sharding import gather_partials
    out32, lse = cache.attend_lse(q.float(), scale=scale, stream=stream)
    parts_out, parts_lse = gather_partials(out32, lse, dist, group)
    return pq_merge_attention(parts_out, parts_lse, torch.empty_like(q), cache.status, stream=stream)


def pq_paged_cache_bytes(d: int, n_kv_heads: int, page_tokens: int, n_pages: int) -> int:
    n = int(lib().pq_paged_cache_bytes(d, n_kv_heads, page_tokens, n_pages))
    if n < 0:
        raise PolarQuantError(n, "pq_paged_cache_bytes")
    return n


class PolarQuantCache:
    """Convenience owner of the device buffers one (layer's) compressed KV cache needs."""

    def __init__(self, batch, n_q_heads, n_kv_heads, d, capacity, seed=0, device="cuda", S=None, codebooks=None):
        self.batch, self.n_q_heads, self.n_kv_heads, self.d, self.capacity = batch, n_q_heads, n_kv_heads, d, capacity
        self.device = torch.device(device)
        self.S_host = pq_make_rotation(d, seed) if S is None else S.to(torch.float32).cpu().contiguous()
        self.centroids, self.boundaries = pq_fit_codebooks() if codebooks is None else codebooks
        self.S = self.S_host.to(self.device)
        self.tables = pq_build_tables(self.centroids, self.boundaries).to(self.device)
        self.cache = torch.empty(pq_cache_bytes(d, batch, n_kv_heads, capacity), dtype=torch.uint8, device=self.device)
        self.lens = torch.zeros(batch, dtype=torch.int32, device=self.device)
        self.status = torch.zeros(STATUS_WORDS, dtype=torch.int32, device=self.device)
        self.workspace = torch.empty(pq_workspace_bytes(d, batch, n_q_heads, n_kv_heads, capacity), dtype=torch.uint8,
                                     device=self.device)

    def fit_online_codebooks(self, K, V, n_bins=HIST_MAX_BINS, stream=None):
        """Replace the codebooks of this cache by the ones clustered on the angles of K, V ([tokens, Hkv, d], the
        prompt's keys and values): histogram on the device, clustering on the host, new tables.  To be called
        before anything is encoded (codes already in the cache belong to the previous codebooks)."""
        hist = torch.zeros((N_LEVELS, n_bins), dtype=torch.int64, device=self.device)
        pq_angle_histograms(self.S, K, V, hist, self.status, stream)
        self.set_codebooks(*pq_fit_codebooks_from_histograms(hist.cpu()))
        return hist

    def set_codebooks(self, centroids, boundaries):
        self.centroids, self.boundaries = centroids, boundaries
        self.tables = pq_build_tables(centroids, boundaries).to(self.device)

    def encode(self, K, V, cu_seqlens, stream=None):
        pq_encode_kv(self.S, self.tables, K, V, cu_seqlens, self.cache, self.lens, self.capacity, self.status, stream)

    def append(self, k_new, v_new, stream=None):
        pq_append_kv(self.S, self.tables, k_new, v_new, self.cache, self.lens, self.capacity, self.status, stream)

    def attend(self, q, out=None, scale=None, max_len=None, stream=None):
        out = torch.empty_like(q) if out is None else out
        scale = self.d ** -0.5 if scale is None else scale
        pq_decode_attention(self.S, self.tables, q, self.cache, self.lens, self.n_kv_heads, self.capacity,
                            self.capacity if max_len is None else max_len, scale, out, self.workspace, self.status,
                            stream)
        return out

    def _paging(self):
        return None

    def attend_lse(self, q, scale=None, max_len=None, stream=None):
        """Partial attention for merging: (out like q, lse float32 [B, Hq]); an empty sequence gives zeros and -inf."""
        out = torch.empty_like(q)
        lse = torch.empty(q.shape[:2], dtype=torch.float32, device=q.device)
        pq_decode_attention_lse(self.S, self.tables, q, self.cache, self.lens, self.n_kv_heads, self.capacity,
                                self.capacity if max_len is None else max_len, self.d ** -0.5 if scale is None else scale,
                                out, lse, self.workspace, self.status, paging=self._paging(), stream=stream)
        return out, lse

    def attend_with_tail(self, q, k_tail, v_tail, tail_lens, scale=None, stream=None):
        """Attention over the compressed cache followed by an uncompressed window (k_tail, v_tail [B, T, Hkv, d], the
        first tail_lens[b] rows): both partial attentions in float32, merged into q's dtype."""
        scale = self.d ** -0.5 if scale is None else scale
        q32 = q.float()
        n_splits = max(1, min(16, (k_tail.shape[1] + 127) // 128))   # enough thread blocks for the window
        parts_out = torch.empty((1 + n_splits,) + q32.shape, dtype=torch.float32, device=q.device)
        parts_lse = torch.empty((1 + n_splits,) + q32.shape[:2], dtype=torch.float32, device=q.device)
        pq_decode_attention_lse(self.S, self.tables, q32, self.cache, self.lens, self.n_kv_heads, self.capacity, self.capacity,
                                scale, parts_out[0], parts_lse[0], self.workspace, self.status, paging=self._paging(),
                                stream=stream)
        pq_tail_attention(q32, k_tail, v_tail, tail_lens, scale, parts_out[1:], parts_lse[1:], self.status, n_splits, stream)
        return pq_merge_attention(parts_out, parts_lse, torch.empty_like(q), self.status, stream=stream)

    def attend_multi(self, q, out=None, scale=None, max_len=None, stream=None):
        """q [B, n_q, Hq, d]: the last n_q positions of every sequence (already in the cache), causal."""
        out = torch.empty_like(q) if out is None else out
        scale = self.d ** -0.5 if scale is None else scale
        need = pq_workspace_bytes(self.d, self.batch * q.shape[1], self.n_q_heads, self.n_kv_heads, self.capacity)
        if getattr(self, "_multi_ws", None) is None or self._multi_ws.numel() < need:
            self._multi_ws = torch.empty(need, dtype=torch.uint8, device=self.device)
        pq_multi_query_attention(self.S, self.tables, q, self.cache, self.lens, self.n_kv_heads, self.capacity,
                                 self.capacity if max_len is None else max_len, scale, out, self._multi_ws, self.status,
                                 stream)
        return out

    def unpack(self, n_tokens):
        return pq_unpack_codes(self.d, self.n_kv_heads, self.cache, self.batch, self.capacity, n_tokens)

    def dequant(self, n_tokens):
        return pq_dequant_kv(self.d, self.n_kv_heads, self.S, self.tables, self.cache, self.batch, self.capacity,
                             n_tokens)

    def check_status(self):
        st = self.status.cpu().tolist()
        if st[0] != OK:
            raise PolarQuantError(st[0], "device status")
        return st


class PagedPolarQuantCache(PolarQuantCache):
    """The same cache behind a block table: a pool of `n_pages` pages of `page_tokens` tokens (all kv heads), and
    page_table int32 [batch, pages_per_seq] naming the physical page of every logical page of every sequence."""

    def __init__(self, batch, n_q_heads, n_kv_heads, d, page_tokens, n_pages, page_table, seed=0, device="cuda", S=None,
                 codebooks=None):
        self.batch, self.n_q_heads, self.n_kv_heads, self.d = batch, n_q_heads, n_kv_heads, d
        self.page_tokens, self.n_pages = page_tokens, n_pages
        self.device = torch.device(device)
        self.page_table = page_table.to(torch.int32).to(self.device).contiguous()
        assert self.page_table.shape[0] == batch
        self.capacity = page_tokens * self.page_table.shape[1]
        self.S_host = pq_make_rotation(d, seed) if S is None else S.to(torch.float32).cpu().contiguous()
        self.centroids, self.boundaries = pq_fit_codebooks() if codebooks is None else codebooks
        self.S = self.S_host.to(self.device)
        self.tables = pq_build_tables(self.centroids, self.boundaries).to(self.device)
        self.cache = torch.empty(pq_paged_cache_bytes(d, n_kv_heads, page_tokens, n_pages), dtype=torch.uint8, device=self.device)
        self.lens = torch.zeros(batch, dtype=torch.int32, device=self.device)
        self.status = torch.zeros(STATUS_WORDS, dtype=torch.int32, device=self.device)
        self.workspace = torch.empty(pq_workspace_bytes(d, batch, n_q_heads, n_kv_heads, self.capacity), dtype=torch.uint8,
                                     device=self.device)

    def _paging(self):
        return Paging.of(self.page_table, self.page_tokens, self.n_pages)

    def encode(self, K, V, cu_seqlens, stream=None):
        total, n_kv_heads, d = K.shape
        assert V.shape == K.shape and V.dtype == K.dtype and K.stride(2) == 1 and V.stride() == K.stride()
        pg = self._paging()
        _check(lib().pq_encode_kv_paged(d, n_kv_heads, _ptr(self.S), _ptr(self.tables), _ptr(K), _ptr(V), _dtype_code(K),
                                        K.stride(0), K.stride(1), _ptr(cu_seqlens), cu_seqlens.numel() - 1, total,
                                        _ptr(self.cache), _ptr(self.lens), ctypes.addressof(pg), _ptr(self.status),
                                        _stream(stream)), "pq_encode_kv_paged")

    def append(self, k_new, v_new, stream=None):
        batch, n_kv_heads, d = k_new.shape
        assert k_new.is_contiguous() and v_new.is_contiguous() and v_new.shape == k_new.shape
        pg = self._paging()
        _check(lib().pq_append_kv_paged(d, n_kv_heads, _ptr(self.S), _ptr(self.tables), _ptr(k_new), _ptr(v_new),
                                        _dtype_code(k_new), batch, _ptr(self.cache), _ptr(self.lens), ctypes.addressof(pg),
                                        _ptr(self.status), _stream(stream)), "pq_append_kv_paged")

    def attend(self, q, out=None, scale=None, max_len=None, stream=None):
        out = torch.empty_like(q) if out is None else out
        batch, n_q_heads, d = q.shape
        assert q.is_contiguous() and out.is_contiguous() and out.shape == q.shape and out.dtype == q.dtype
        pg = self._paging()
        _check(lib().pq_decode_attention_paged(d, n_q_heads, self.n_kv_heads, _ptr(self.S), _ptr(self.tables), _ptr(q),
                                               _dtype_code(q), _ptr(self.cache), _ptr(self.lens), batch,
                                               ctypes.addressof(pg), self.capacity if max_len is None else max_len,
                                               float(self.d ** -0.5 if scale is None else scale), _ptr(out),
                                               _ptr(self.workspace), _ptr(self.status), _stream(stream)),
               "pq_decode_attention_paged")
        return out

    def attend_multi(self, q, out=None, scale=None, max_len=None, stream=None):
        out = torch.empty_like(q) if out is None else out
        batch, n_q, n_q_heads, d = q.shape
        assert q.is_contiguous() and out.is_contiguous() and out.shape == q.shape and out.dtype == q.dtype
        need = pq_workspace_bytes(self.d, self.batch * n_q, self.n_q_heads, self.n_kv_heads, self.capacity)
        if getattr(self, "_multi_ws", None) is None or self._multi_ws.numel() < need:
            self._multi_ws = torch.empty(need, dtype=torch.uint8, device=self.device)
        pg = self._paging()
        _check(lib().pq_multi_query_attention_paged(d, n_q_heads, self.n_kv_heads, _ptr(self.S), _ptr(self.tables), _ptr(q),
                                                    _dtype_code(q), _ptr(self.cache), _ptr(self.lens), batch, n_q,
                                                    ctypes.addressof(pg), self.capacity if max_len is None else max_len,
                                                    float(self.d ** -0.5 if scale is None else scale), _ptr(out),
                                                    _ptr(self._multi_ws), _ptr(self.status), _stream(stream)),
               "pq_multi_query_attention_paged")
        return out

    def unpack(self, n_tokens):
        codes = torch.zeros((self.batch, self.n_kv_heads, 2, n_tokens, 15 * self.d // 16), dtype=torch.uint8, device=self.device)
        radii = torch.zeros((self.batch, self.n_kv_heads, 2, n_tokens, self.d // 16), dtype=torch.float16, device=self.device)
        pg = self._paging()
        _check(lib().pq_unpack_codes_paged(self.d, self.n_kv_heads, _ptr(self.cache), self.batch, ctypes.addressof(pg),
                                           n_tokens, _ptr(codes), _ptr(radii), _stream(None)), "pq_unpack_codes_paged")
        return codes, radii

    def dequant(self, n_tokens):
        out = torch.zeros((self.batch, self.n_kv_heads, 2, n_tokens, self.d), dtype=torch.float32, device=self.device)
        pg = self._paging()
        _check(lib().pq_dequant_kv_paged(self.d, self.n_kv_heads, _ptr(self.S), _ptr(self.tables), _ptr(self.cache),
                                         self.batch, ctypes.addressof(pg), n_tokens, _ptr(out), _stream(None)),
               "pq_dequant_kv_paged")
        return out


class GeneralConfig(ctypes.Structure):
    """struct pq_general_config of include/polarquant.h: any recursion depth and bits per level."""
    _fields_ = [("head_dim", c_int32), ("n_levels", c_int32), ("bits", c_int32 * 8)]

    @classmethod
    def of(cls, head_dim: int, bits) -> "GeneralConfig":
        arr = (c_int32 * 8)(*(list(bits) + [0] * (8 - len(bits))))
        return cls(head_dim, len(bits), arr)

    def sizes(self):
        """(n_centroids, n_boundaries, n_codes, n_radii, row_bytes)"""
        out = [c_int32() for _ in range(5)]
        _check(lib().pq_general_sizes(ctypes.addressof(self), *[ctypes.addressof(o) for o in out]), "pq_general_sizes")
        return tuple(o.value for o in out)


def pq_general_fit_codebooks(cfg: GeneralConfig):
    """Lloyd-Max codebooks of the analytic densities for every level of `cfg`: (centroids, boundaries) float64 CPU tensors."""
    n_cen, n_bnd = cfg.sizes()[:2]
    cen, bnd = torch.empty(n_cen, dtype=torch.float64), torch.empty(n_bnd, dtype=torch.float64)
    _check(lib().pq_general_fit_codebooks(ctypes.addressof(cfg), cen.data_ptr(), bnd.data_ptr()), "pq_general_fit_codebooks")
    return cen, bnd


class GeneralPolarQuantCache:
    """A contiguous cache for any recursion depth and bit table (pq_general_*): reference-speed kernels."""

    def __init__(self, batch, n_q_heads, n_kv_heads, d, bits, capacity, seed=0, device="cuda", S=None, codebooks=None):
        self.batch, self.n_q_heads, self.n_kv_heads, self.d, self.capacity = batch, n_q_heads, n_kv_heads, d, capacity
        self.bits = tuple(bits)
        self.cfg = GeneralConfig.of(d, bits)
        _, _, self.n_codes, self.n_radii, self.row_bytes = self.cfg.sizes()
        self.device = torch.device(device)
        self.S_host = pq_make_rotation(d, seed) if S is None else S.to(torch.float32).cpu().contiguous()
        self.centroids, self.boundaries = pq_general_fit_codebooks(self.cfg) if codebooks is None else codebooks
        self.S = self.S_host.to(self.device)
        self.centroids_dev, self.boundaries_dev = self.centroids.to(self.device), self.boundaries.to(self.device)
        n = int(lib().pq_general_cache_bytes(ctypes.addressof(self.cfg), batch, n_kv_heads, capacity))
        if n < 0:
            raise PolarQuantError(n, "pq_general_cache_bytes")
        self.cache = torch.empty(n, dtype=torch.uint8, device=self.device)
        self.lens = torch.zeros(batch, dtype=torch.int32, device=self.device)
        self.status = torch.zeros(STATUS_WORDS, dtype=torch.int32, device=self.device)

    def encode(self, K, V, cu_seqlens, stream=None):
        total, n_kv_heads, d = K.shape
        assert V.shape == K.shape and V.dtype == K.dtype and K.stride(2) == 1 and V.stride() == K.stride() and d == self.d
        _check(lib().pq_general_encode_kv(ctypes.addressof(self.cfg), n_kv_heads, _ptr(self.S), _ptr(self.boundaries_dev), _ptr(K),
                                          _ptr(V), _dtype_code(K), K.stride(0), K.stride(1), _ptr(cu_seqlens),
                                          cu_seqlens.numel() - 1, total, _ptr(self.cache), _ptr(self.lens), self.capacity,
                                          _ptr(self.status), _stream(stream)), "pq_general_encode_kv")

    def attend(self, q, out=None, scale=None, stream=None):
        out = torch.empty_like(q) if out is None else out
        batch, n_q_heads, d = q.shape
        assert q.is_contiguous() and out.is_contiguous() and out.dtype == q.dtype and d == self.d
        _check(lib().pq_general_decode_attention(ctypes.addressof(self.cfg), n_q_heads, self.n_kv_heads, _ptr(self.S),
                                                 _ptr(self.centroids_dev), _ptr(q), _dtype_code(q), _ptr(self.cache),
                                                 _ptr(self.lens), batch, self.capacity,
                                                 float(self.d ** -0.5 if scale is None else scale), _ptr(out),
                                                 _ptr(self.status), _stream(stream)), "pq_general_decode_attention")
        return out

    def unpack(self, n_tokens):
        codes = torch.empty((self.batch, self.n_kv_heads, 2, n_tokens, self.n_codes), dtype=torch.uint8, device=self.device)
        radii = torch.empty((self.batch, self.n_kv_heads, 2, n_tokens, self.n_radii), dtype=torch.float16, device=self.device)
        _check(lib().pq_general_unpack_codes(ctypes.addressof(self.cfg), self.n_kv_heads, _ptr(self.cache), self.batch,
                                             self.capacity, n_tokens, _ptr(codes), _ptr(radii), _stream(None)),
               "pq_general_unpack_codes")
        return codes, radii

    def dequant(self, n_tokens):
        out = torch.empty((self.batch, self.n_kv_heads, 2, n_tokens, self.d), dtype=torch.float32, device=self.device)
        _check(lib().pq_general_dequant_kv(ctypes.addressof(self.cfg), self.n_kv_heads, _ptr(self.S), _ptr(self.centroids_dev),
                                           _ptr(self.cache), self.batch, self.capacity, n_tokens, _ptr(out), _stream(None)),
               "pq_general_dequant_kv")
        return out

    def check_status(self):
        st = self.status.cpu().tolist()
        if st[0] != OK:
            raise PolarQuantError(st[0], "device status")
        return st
