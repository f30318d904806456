"""ctypes binding of libwushkv.so: the same entry points as ``include/wushkv.h``, argument
marshalling only.  Every step of the hot path runs inside the library's CUDA kernels; PyTorch is
used here for device memory and streams and nothing else.  There is no CPU fallback: importing
this module without the built library raises."""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libwushkv.so")

OK, EINVAL, ENOTPD, ECUDA, ECAPACITY = 0, 1, 2, 3, 4
QUANTIZER_AFFINE, QUANTIZER_QUEST = 0, 1
DEV_PAGE_TABLE_FULL, DEV_BAD_PAGE_ID, DEV_BAD_SLOT, DEV_COPY_TIMEOUT, DEV_BAD_COUNT, DEV_VALUE_RANGE = 1, 2, 4, 8, 16, 32
DEV_ROPE_RANGE = 64

EXPORTS = (
    "wushkv_page_bytes", "wushkv_status_string", "wushkv_accumulate_gram", "wushkv_build_transforms",
    "wushkv_append", "wushkv_decode_workspace_bytes", "wushkv_decode_attn", "wushkv_unpack_debug",
    "wushkv_decode_step", "wushkv_step_staging_bytes", "wushkv_decode_step_host", "wushkv_set_profile_events",
    "wushkv_decode_attn_static", "wushkv_set_test_option", "wushkv_prefill_workspace_bytes", "wushkv_prefill_attn",
    "wushkv_accumulate_gram_device", "wushkv_build_transforms_workspace_bytes", "wushkv_build_transforms_device",
    "wushkv_build_rope_table", "wushkv_append_projected", "wushkv_decode_attn_projected",
    "wushkv_attention_hessians_workspace_bytes", "wushkv_accumulate_attention_hessians_device",
    "wushkv_prefill_attn_projected",
)
STATIC_SCRATCH_BYTES = 8 << 20


class WushkvError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: status {status} ({status_string(status)})")


class wushkv_cache(C.Structure):
    """Mirror of ``struct wushkv_cache``."""
    _fields_ = [
        ("n_q", C.c_int32), ("n_kv", C.c_int32), ("d", C.c_int32), ("bits", C.c_int32),
        ("page_tokens", C.c_int32), ("s_sink", C.c_int32), ("s_keep", C.c_int32), ("s_flush", C.c_int32),
        ("boundary_lag", C.c_int32),
        ("n_slots", C.c_int32), ("max_pages", C.c_int32), ("ring_cap", C.c_int32),
        ("kappa_k", C.c_float), ("kappa_v", C.c_float), ("sm_scale", C.c_float),
        ("quantizer", C.c_int32),
        ("n_pages", C.c_int64),
        ("pages", C.c_void_p), ("page_table", C.c_void_p), ("sink_kv", C.c_void_p), ("ring_kv", C.c_void_p),
        ("T_K", C.c_void_p), ("T_K_invT", C.c_void_p), ("dev_status", C.c_void_p),
    ]


class wushkv_prologue(C.Structure):
    """Mirror of ``struct wushkv_prologue`` (device pointers)."""
    _fields_ = [("rope_table", C.c_void_p), ("rope_positions", C.c_int32), ("normalise", C.c_int32),
                ("k_norm_weight", C.c_void_p), ("q_norm_weight", C.c_void_p), ("norm_eps", C.c_float)]


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2609_38121_b200.build` "
            "(nvcc, sm_100a).  There is no fallback path.")
    lib = C.CDLL(LIB_PATH)
    lib.wushkv_page_bytes.restype = C.c_size_t
    lib.wushkv_page_bytes.argtypes = [C.c_int32] * 4
    lib.wushkv_status_string.restype = C.c_char_p
    lib.wushkv_status_string.argtypes = [C.c_int]
    lib.wushkv_accumulate_gram.restype = C.c_int
    lib.wushkv_accumulate_gram.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.c_int64, C.c_void_p, C.c_void_p,
                                           C.c_void_p, C.c_void_p]
    lib.wushkv_build_transforms.restype = C.c_int
    lib.wushkv_build_transforms.argtypes = [C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_double,
                                            C.c_void_p, C.c_void_p]
    lib.wushkv_append.restype = C.c_int
    lib.wushkv_append.argtypes = [C.POINTER(wushkv_cache), C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p,
                                  C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]
    lib.wushkv_decode_workspace_bytes.restype = C.c_size_t
    lib.wushkv_decode_workspace_bytes.argtypes = [C.POINTER(wushkv_cache), C.c_int32, C.c_int32]
    lib.wushkv_decode_attn.restype = C.c_int
    lib.wushkv_decode_attn.argtypes = [C.POINTER(wushkv_cache), C.c_int32, C.c_void_p, C.c_void_p, C.c_int32,
                                       C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
    lib.wushkv_unpack_debug.restype = C.c_int
    lib.wushkv_unpack_debug.argtypes = [C.POINTER(wushkv_cache), C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                                        C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    lib.wushkv_decode_step.restype = C.c_int
    lib.wushkv_decode_step.argtypes = [C.POINTER(wushkv_cache), C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32,
                                       C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
    lib.wushkv_step_staging_bytes.restype = C.c_size_t
    lib.wushkv_step_staging_bytes.argtypes = [C.POINTER(wushkv_cache), C.c_int32]
    lib.wushkv_decode_step_host.restype = C.c_int
    lib.wushkv_decode_step_host.argtypes = [C.POINTER(wushkv_cache), C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p,
                                            C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                            C.c_void_p, C.c_size_t, C.c_void_p, C.c_size_t, C.c_void_p]
    lib.wushkv_decode_attn_static.restype = C.c_int
    lib.wushkv_decode_attn_static.argtypes = [C.POINTER(wushkv_cache), C.c_int32, C.c_void_p, C.c_void_p, C.c_int32,
                                              C.c_void_p, C.c_void_p, C.c_void_p]
    lib.wushkv_set_profile_events.restype = C.c_int
    lib.wushkv_set_profile_events.argtypes = [C.c_void_p, C.c_void_p]
    lib.wushkv_prefill_workspace_bytes.restype = C.c_size_t
    lib.wushkv_prefill_workspace_bytes.argtypes = [C.POINTER(wushkv_cache), C.c_int32, C.c_int32]
    lib.wushkv_prefill_attn.restype = C.c_int
    lib.wushkv_prefill_attn.argtypes = [C.POINTER(wushkv_cache), C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32,
                                        C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
    lib.wushkv_accumulate_gram_device.restype = C.c_int
    lib.wushkv_accumulate_gram_device.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p,
                                                  C.c_void_p, C.c_void_p]
    lib.wushkv_build_transforms_workspace_bytes.restype = C.c_size_t
    lib.wushkv_build_transforms_workspace_bytes.argtypes = [C.c_int32, C.c_int32]
    lib.wushkv_build_transforms_device.restype = C.c_int
    lib.wushkv_build_transforms_device.argtypes = [C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_double, C.c_void_p, C.c_void_p,
                                                   C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
    lib.wushkv_build_rope_table.restype = C.c_int
    lib.wushkv_build_rope_table.argtypes = [C.c_double, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p]
    lib.wushkv_append_projected.restype = C.c_int
    lib.wushkv_append_projected.argtypes = [C.POINTER(wushkv_cache), C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p,
                                            C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.POINTER(wushkv_prologue), C.c_void_p]
    lib.wushkv_decode_attn_projected.restype = C.c_int
    lib.wushkv_decode_attn_projected.argtypes = [C.POINTER(wushkv_cache), C.c_int32, C.c_void_p, C.c_void_p, C.c_int32,
                                                 C.c_void_p, C.POINTER(wushkv_prologue), C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
    lib.wushkv_prefill_attn_projected.restype = C.c_int
    lib.wushkv_prefill_attn_projected.argtypes = [C.POINTER(wushkv_cache), C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32,
                                                  C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(wushkv_prologue), C.c_void_p, C.c_void_p,
                                                  C.c_size_t, C.c_void_p]
    lib.wushkv_attention_hessians_workspace_bytes.restype = C.c_size_t
    lib.wushkv_attention_hessians_workspace_bytes.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.c_int64]
    lib.wushkv_accumulate_attention_hessians_device.restype = C.c_int
    lib.wushkv_accumulate_attention_hessians_device.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int64, C.c_void_p,
                                                                C.c_void_p, C.c_void_p, C.c_void_p, C.c_double, C.c_void_p,
                                                                C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
    lib.wushkv_set_test_option.restype = C.c_int
    lib.wushkv_set_test_option.argtypes = [C.c_char_p, C.c_longlong]
    return lib


lib = _load()


def _check(status: int, where: str):
    if status != OK:
        raise WushkvError(status, where)


def _ptr(t):
    """Device or host pointer of a torch tensor / numpy array (None -> NULL)."""
    if t is None:
        return None
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    return t.data_ptr()


def _stream_ptr(stream):
    import torch
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def status_string(status: int) -> str:
    return lib.wushkv_status_string(int(status)).decode()


def page_bytes(n_kv: int, d: int, bits: int, page_tokens: int) -> int:
    return int(lib.wushkv_page_bytes(n_kv, d, bits, page_tokens))


def accumulate_gram(K_bits: np.ndarray, Q_bits: np.ndarray, M: np.ndarray, H: np.ndarray):
    """wushkv_accumulate_gram: K_bits uint16 [n_tok][n_kv][d], Q_bits uint16 [n_tok][n_q][d] (bf16
    patterns), M and H float64 [n_kv][d][d] updated in place."""
    K_bits = np.ascontiguousarray(K_bits, dtype=np.uint16)
    Q_bits = np.ascontiguousarray(Q_bits, dtype=np.uint16)
    assert M.dtype == np.float64 and H.dtype == np.float64 and M.flags.c_contiguous and H.flags.c_contiguous
    n_tok, n_kv, d = K_bits.shape
    _check(lib.wushkv_accumulate_gram(n_kv, Q_bits.shape[1], d, n_tok, K_bits.ctypes.data, Q_bits.ctypes.data,
                                      M.ctypes.data, H.ctypes.data), "wushkv_accumulate_gram")


def build_transforms(M: np.ndarray, H: np.ndarray, gamma: float):
    """wushkv_build_transforms: returns (T, T_invT) as float32 [n_heads][d][d]."""
    M = np.ascontiguousarray(M, dtype=np.float64)
    H = np.ascontiguousarray(H, dtype=np.float64)
    n, d, _ = M.shape
    T = np.empty((n, d, d), dtype=np.float32)
    TinvT = np.empty((n, d, d), dtype=np.float32)
    _check(lib.wushkv_build_transforms(n, d, M.ctypes.data, H.ctypes.data, float(gamma), T.ctypes.data,
                                       TinvT.ctypes.data), "wushkv_build_transforms")
    return T, TinvT


def accumulate_gram_device(K_bits, Q_bits, M, H, stream=None):
    """wushkv_accumulate_gram_device: K_bits int16/uint16 [n_tok][n_kv][d], Q_bits [n_tok][n_q][d] (bf16 patterns) and
    M, H float64 [n_kv][d][d], all CUDA tensors; M and H are updated in place."""
    n_tok, n_kv, d = K_bits.shape
    _check(lib.wushkv_accumulate_gram_device(n_kv, Q_bits.shape[1], d, n_tok, _ptr(K_bits), _ptr(Q_bits), _ptr(M), _ptr(H),
                                             _stream_ptr(stream)), "wushkv_accumulate_gram_device")


def build_transforms_device(M, H, gamma: float, stream=None):
    """wushkv_build_transforms_device: M, H float64 CUDA tensors [n_heads][d][d]; returns (T, T_invT) fp32 CUDA tensors.
    Raises with status ENOTPD if a damped matrix is not positive definite (this wrapper synchronises to find out)."""
    import torch
    n, d, _ = M.shape
    T = torch.empty((n, d, d), dtype=torch.float32, device=M.device)
    Ti = torch.empty_like(T)
    status = torch.zeros(1, dtype=torch.int32, device=M.device)
    nbytes = int(lib.wushkv_build_transforms_workspace_bytes(n, d))
    ws = torch.empty(nbytes, dtype=torch.uint8, device=M.device)
    _check(lib.wushkv_build_transforms_device(n, d, _ptr(M), _ptr(H), float(gamma), _ptr(T), _ptr(Ti), _ptr(status), _ptr(ws),
                                              nbytes, _stream_ptr(stream)), "wushkv_build_transforms_device")
    st = int(status.item())
    if st != 0:
        raise WushkvError(st, "wushkv_build_transforms_device")
    return T, Ti


def append(cache: wushkv_cache, batch, slot, seq_len, cu_new, total_new, max_new, K_new, V_new, stream=None):
    _check(lib.wushkv_append(C.byref(cache), batch, _ptr(slot), _ptr(seq_len), _ptr(cu_new), total_new, max_new,
                             _ptr(K_new), _ptr(V_new), _stream_ptr(stream)), "wushkv_append")


def accumulate_attention_hessians_device(K_bits, Q_bits, V_bits, W_O, tau: float, H_K, H_V, stream=None):
    """wushkv_accumulate_attention_hessians_device: K_bits / V_bits [n_tok][n_kv][d], Q_bits [n_tok][n_q][d] (bf16 patterns),
    W_O fp32 [n_q][d][d_model], H_K / H_V float64 [n_kv][d][d] (accumulated), all CUDA tensors; the scratch is allocated here."""
    import torch
    n_tok, n_kv, d = K_bits.shape
    n_q, d_model = Q_bits.shape[1], W_O.shape[2]
    nbytes = int(lib.wushkv_attention_hessians_workspace_bytes(n_kv, n_q, d, n_tok))
    if nbytes == 0:
        raise WushkvError(EINVAL, "wushkv_attention_hessians_workspace_bytes")
    ws = torch.empty(nbytes, dtype=torch.uint8, device=K_bits.device)
    _check(lib.wushkv_accumulate_attention_hessians_device(n_kv, n_q, d, d_model, n_tok, _ptr(K_bits), _ptr(Q_bits), _ptr(V_bits),
                                                           _ptr(W_O), float(tau), _ptr(H_K), _ptr(H_V), _ptr(ws), nbytes,
                                                           _stream_ptr(stream)), "wushkv_accumulate_attention_hessians_device")


class Prologue:
    """Holds the device tensors a ``wushkv_prologue`` points to (rotary table from wushkv_build_rope_table, optional
    normalisation weights [n_kv][d] / [n_q][d]) and the struct itself."""

    def __init__(self, theta: float, n_positions: int, normalise: bool = False, k_weight=None, q_weight=None,
                 eps: float = 0.0, device="cuda", d: int = 128):
        import torch
        self.table = torch.empty((n_positions, d // 2, 2), dtype=torch.float32, device=device)
        _check(lib.wushkv_build_rope_table(float(theta), n_positions, d, _ptr(self.table), _stream_ptr(None)),
               "wushkv_build_rope_table")
        as_dev = lambda w: None if w is None else torch.as_tensor(np.ascontiguousarray(w, dtype=np.float32)).to(device)
        self.k_weight, self.q_weight = as_dev(k_weight), as_dev(q_weight)
        self.desc = wushkv_prologue(_ptr(self.table), n_positions, 1 if normalise else 0, _ptr(self.k_weight),
                                    _ptr(self.q_weight), float(eps))


def append_projected(cache: wushkv_cache, batch, slot, seq_len, cu_new, total_new, max_new, K_proj, V_new,
                     prologue: wushkv_prologue, stream=None):
    """wushkv_append_projected: wushkv_append on projected keys (Norm and RoPE applied inside the kernels)."""
    _check(lib.wushkv_append_projected(C.byref(cache), batch, _ptr(slot), _ptr(seq_len), _ptr(cu_new), total_new, max_new,
                                       _ptr(K_proj), _ptr(V_new), C.byref(prologue), _stream_ptr(stream)),
           "wushkv_append_projected")


def decode_attn_projected(cache: wushkv_cache, batch, slot, seq_len, max_seq_len, Q_proj, prologue: wushkv_prologue, O,
                          workspace, workspace_bytes, stream=None):
    """wushkv_decode_attn_projected: wushkv_decode_attn on projected queries."""
    _check(lib.wushkv_decode_attn_projected(C.byref(cache), batch, _ptr(slot), _ptr(seq_len), max_seq_len, _ptr(Q_proj),
                                            C.byref(prologue), _ptr(O), _ptr(workspace), workspace_bytes,
                                            _stream_ptr(stream)), "wushkv_decode_attn_projected")


def prefill_attn_projected(cache: wushkv_cache, batch, slot, seq_len, cu_new, total_new, max_new, K_proj, V_new, Q_proj,
                           prologue: wushkv_prologue, O, workspace, workspace_bytes, stream=None):
    """wushkv_prefill_attn_projected: wushkv_prefill_attn on projected keys and queries."""
    _check(lib.wushkv_prefill_attn_projected(C.byref(cache), batch, _ptr(slot), _ptr(seq_len), _ptr(cu_new), total_new, max_new,
                                             _ptr(K_proj), _ptr(V_new), _ptr(Q_proj), C.byref(prologue), _ptr(O), _ptr(workspace),
                                             workspace_bytes, _stream_ptr(stream)), "wushkv_prefill_attn_projected")


def decode_workspace_bytes(cache: wushkv_cache, batch: int, max_seq_len: int) -> int:
    return int(lib.wushkv_decode_workspace_bytes(C.byref(cache), batch, max_seq_len))


def decode_attn(cache: wushkv_cache, batch, slot, seq_len, max_seq_len, Q, O, workspace, workspace_bytes, stream=None):
    _check(lib.wushkv_decode_attn(C.byref(cache), batch, _ptr(slot), _ptr(seq_len), max_seq_len, _ptr(Q), _ptr(O),
                                  _ptr(workspace), workspace_bytes, _stream_ptr(stream)), "wushkv_decode_attn")


def unpack_debug(cache: wushkv_cache, slot, kv_head, which, pos0, n, codes, scale, zero, stream=None):
    _check(lib.wushkv_unpack_debug(C.byref(cache), slot, kv_head, which, pos0, n, _ptr(codes), _ptr(scale),
                                   _ptr(zero), _stream_ptr(stream)), "wushkv_unpack_debug")


def decode_attn_static(cache: wushkv_cache, batch, slot, seq_len, max_seq_len, Q, O, stream=None):
    """wushkv_decode_attn_static: decode attention for callers that cannot allocate device memory
    (the workspace is a fixed array inside the library; requests needing more than
    STATIC_SCRATCH_BYTES raise with status ECAPACITY; overlapping calls on one GPU race)."""
    _check(lib.wushkv_decode_attn_static(C.byref(cache), batch, _ptr(slot), _ptr(seq_len), max_seq_len, _ptr(Q),
                                         _ptr(O), _stream_ptr(stream)), "wushkv_decode_attn_static")


def decode_step(cache: wushkv_cache, batch, slot, seq_len, cu_new, max_seq_len, K_new, V_new, Q, O, workspace,
                workspace_bytes, stream=None):
    """wushkv_decode_step: append one token per sequence, then decode over the extended cache (device tensors)."""
    _check(lib.wushkv_decode_step(C.byref(cache), batch, _ptr(slot), _ptr(seq_len), _ptr(cu_new), max_seq_len,
                                  _ptr(K_new), _ptr(V_new), _ptr(Q), _ptr(O), _ptr(workspace), workspace_bytes,
                                  _stream_ptr(stream)), "wushkv_decode_step")


def step_staging_bytes(cache: wushkv_cache, batch: int) -> int:
    return int(lib.wushkv_step_staging_bytes(C.byref(cache), batch))


def decode_step_host(cache: wushkv_cache, batch, slot, seq_len, cu_new, max_seq_len, K_new_host, V_new_host, Q_host,
                     O_host, staging, staging_bytes, workspace, workspace_bytes, stream=None):
    """wushkv_decode_step_host: the *_host tensors are (pinned) CPU tensors, everything else device."""
    _check(lib.wushkv_decode_step_host(C.byref(cache), batch, _ptr(slot), _ptr(seq_len), _ptr(cu_new), max_seq_len,
                                       _ptr(K_new_host), _ptr(V_new_host), _ptr(Q_host), _ptr(O_host),
                                       _ptr(staging), staging_bytes, _ptr(workspace), workspace_bytes,
                                       _stream_ptr(stream)), "wushkv_decode_step_host")


def set_profile_events(start=None, stop=None):
    """wushkv_set_profile_events with torch.cuda.Event objects (already recorded once so that their
    handles exist) or None to switch the hook off."""
    a = C.c_void_p(start.cuda_event) if start is not None else None
    b = C.c_void_p(stop.cuda_event) if stop is not None else None
    _check(lib.wushkv_set_profile_events(a, b), "wushkv_set_profile_events")


def prefill_workspace_bytes(cache: wushkv_cache, batch: int, total_new: int) -> int:
    return int(lib.wushkv_prefill_workspace_bytes(C.byref(cache), batch, total_new))


def prefill_attn(cache: wushkv_cache, batch, slot, seq_len, cu_new, total_new, max_new, K_new, V_new, Q_new, O, workspace,
                 workspace_bytes, stream=None):
    """wushkv_prefill_attn: attention outputs of an appended chunk over the mixed cache (device tensors)."""
    _check(lib.wushkv_prefill_attn(C.byref(cache), batch, _ptr(slot), _ptr(seq_len), _ptr(cu_new), total_new, max_new,
                                   _ptr(K_new), _ptr(V_new), _ptr(Q_new), _ptr(O), _ptr(workspace), workspace_bytes,
                                   _stream_ptr(stream)), "wushkv_prefill_attn")


def set_test_option(name: str, value: int):
    """wushkv_set_test_option: process-wide testing aids (see the header for the names)."""
    _check(lib.wushkv_set_test_option(name.encode(), int(value)), "wushkv_set_test_option")


class PagedCache:
    """Owns the device buffers of one layer's cache (torch tensors) and the filled ``wushkv_cache``
    descriptor.  Pure bookkeeping: page-table assignment and allocation, no arithmetic."""

    def __init__(self, n_q, n_kv, bits, n_slots, max_seq_len, s_sink, s_keep, s_flush, kappa_k, kappa_v,
                 T_K, T_K_invT, sm_scale=None, boundary_lag=0, ring_cap=None, device="cuda", page_order=None, quantizer=0):
        import torch
        d, page_tokens = 128, 64
        self.torch = torch
        self.device = torch.device(device)
        self.n_q, self.n_kv, self.bits, self.n_slots = n_q, n_kv, bits, n_slots
        self.max_pages = (max_seq_len + page_tokens - 1) // page_tokens
        n_pages = n_slots * self.max_pages
        self.page_bytes = page_bytes(n_kv, d, bits, page_tokens)
        self.pages = torch.zeros(n_pages * self.page_bytes, dtype=torch.uint8, device=self.device)
        order = np.arange(n_pages) if page_order is None else np.asarray(page_order)
        self.page_table = torch.from_numpy(order.reshape(n_slots, self.max_pages).astype(np.int32)).to(self.device)
        self.ring_cap = ring_cap if ring_cap is not None else s_keep + s_flush - 1 + boundary_lag
        self.sink_kv = torch.zeros((n_slots, n_kv, 2, max(s_sink, 1), d), dtype=torch.bfloat16, device=self.device)
        self.ring_kv = torch.zeros((n_slots, n_kv, 2, self.ring_cap, d), dtype=torch.bfloat16, device=self.device)
        self.T_K = torch.as_tensor(np.ascontiguousarray(T_K, dtype=np.float32)).to(self.device)
        self.T_K_invT = torch.as_tensor(np.ascontiguousarray(T_K_invT, dtype=np.float32)).to(self.device)
        self.dev_status = torch.zeros(1, dtype=torch.int32, device=self.device)
        self.desc = wushkv_cache(
            n_q=n_q, n_kv=n_kv, d=d, bits=bits, page_tokens=page_tokens, s_sink=s_sink, s_keep=s_keep, s_flush=s_flush,
            boundary_lag=boundary_lag, n_slots=n_slots, max_pages=self.max_pages, ring_cap=self.ring_cap,
            kappa_k=kappa_k, kappa_v=kappa_v, sm_scale=(sm_scale if sm_scale is not None else 1.0 / np.sqrt(d)),
            quantizer=quantizer, n_pages=n_pages, pages=self.pages.data_ptr(), page_table=self.page_table.data_ptr(),
            sink_kv=self.sink_kv.data_ptr(), ring_kv=self.ring_kv.data_ptr(), T_K=self.T_K.data_ptr(),
            T_K_invT=self.T_K_invT.data_ptr(), dev_status=self.dev_status.data_ptr())

    def status(self) -> int:
        return int(self.dev_status.item())
