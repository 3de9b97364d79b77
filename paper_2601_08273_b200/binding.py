"""Thin ctypes binding of libhippo.so: same names as the C ABI (include/hippo.h), argument marshalling only.

Every step of the hot path runs in the CUDA library; there is no CPU or PyTorch fallback.  Importing this module
fails loudly if the library has not been built (`python -m paper_2601_08273_b200.build`).  PyTorch is used for
device memory and streams only: tensors are passed as raw device pointers.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence, Tuple

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
# HIPPO_LIBRARY_PATH selects a libhippo.so built elsewhere (same ABI); default: the in-tree build.
LIB_PATH = os.environ.get("HIPPO_LIBRARY_PATH") or os.path.join(_PKG, "libhippo.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        "libhippo.so is missing (%s). Build the CUDA extension first: python -m paper_2601_08273_b200.build. "
        "There is no fallback path." % LIB_PATH)

lib = ctypes.CDLL(LIB_PATH)

HIPPO_OK = 0
HIPPO_ERR_INVALID_ARG = -1
HIPPO_ERR_UNSUPPORTED_SHAPE = -2
HIPPO_ERR_WORKSPACE_TOO_SMALL = -3
HIPPO_ERR_CUDA = -4
HIPPO_ERR_TIMEOUT = -5
HIPPO_ERR_UNIMPLEMENTED = -6
HIPPO_DTYPE_FP32 = 0
HIPPO_DTYPE_BF16 = 1
HIPPO_SCORE_ALL = 7
HIPPO_SELECT_HOLISTIC, HIPPO_SELECT_UNIFORM_PER_FRAME, HIPPO_SELECT_RANDOM, HIPPO_SELECT_FRAMES = 0, 1, 2, 3
HIPPO_ACCEPT_SAMPLE = 0
HIPPO_ACCEPT_GREEDY = 1
HIPPO_ACCEPT_ONE_LAUNCH = 16
HIPPO_ACCEPT_THREE_LAUNCHES = 32
PAGE_SIZE = 64

_vp, _i32, _u32, _sz, _f32 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_uint32, ctypes.c_size_t, ctypes.c_float


class KVCacheStruct(ctypes.Structure):
    _fields_ = [("struct_size", _u32), ("dtype", _i32), ("n_kv_heads", _i32), ("head_dim", _i32),
                ("n_pages", _i32), ("max_pages_per_seq", _i32), ("k_pages", _vp), ("v_pages", _vp),
                ("page_table", _vp)]


_KVP = ctypes.POINTER(KVCacheStruct)
_I32P = ctypes.POINTER(_i32)

lib.hippo_version.restype = _i32
lib.hippo_status_string.restype = ctypes.c_char_p
lib.hippo_status_string.argtypes = [_i32]
lib.hippo_last_error.restype = ctypes.c_char_p
lib.hippo_launch_count.restype = ctypes.c_uint64
lib.hippo_workspace_status.restype = _i32
lib.hippo_workspace_status.argtypes = [_vp, _vp]
lib.hippo_workspace_reset.restype = _i32
lib.hippo_workspace_reset.argtypes = [_vp, _sz, _vp]
lib.hippo_read_probe.restype = _i32
lib.hippo_read_probe.argtypes = [_vp, _sz, _vp, _vp]
lib.hippo_select_workspace_bytes.restype = _sz
lib.hippo_select_workspace_bytes.argtypes = [_i32, _I32P, _i32, _i32, _i32, _i32]
lib.hippo_select_tokens.restype = _i32
lib.hippo_select_tokens.argtypes = [_i32, _I32P, _i32, _i32, _i32, _i32, _i32, _i32, _vp, _vp, _I32P, _I32P, _u32, _vp, _vp,
                                    _vp, _sz, _vp]
lib.hippo_select_tokens_policy.restype = _i32
lib.hippo_select_tokens_policy.argtypes = [_i32, _I32P, _i32, _i32, _i32, _i32, _i32, _i32, _vp, _vp, _I32P, _I32P, _u32, _i32, _vp,
                                           _vp, _vp, _vp, _sz, _vp]
lib.hippo_gather_kv.restype = _i32
lib.hippo_gather_kv.argtypes = [_i32, _KVP, _sz, _KVP, _sz, _i32, _vp, _vp, _i32, _vp, _vp]
lib.hippo_attention_workspace_bytes.restype = _sz
lib.hippo_attention_workspace_bytes.argtypes = [_i32] * 5
for _name in ("hippo_verify_attention", "hippo_draft_attention"):
    getattr(lib, _name).restype = _i32
    getattr(lib, _name).argtypes = [_i32, _i32, _i32, _vp, _KVP, _vp, _I32P, _i32, _f32, _i32, _vp, _vp, _vp, _sz, _vp]
lib.hippo_verify_attention_layers_workspace_bytes.restype = _sz
lib.hippo_verify_attention_layers_workspace_bytes.argtypes = [_i32] * 6
lib.hippo_verify_attention_layers.restype = _i32
lib.hippo_verify_attention_layers.argtypes = [_i32, _i32, _i32, _i32, ctypes.POINTER(_vp), _KVP, _vp, _I32P, _i32, _f32, _i32,
                                              ctypes.POINTER(_vp), ctypes.POINTER(_vp), _vp, _sz, _vp]
lib.hippo_workspace_set_wait_limit.restype = _i32
lib.hippo_workspace_set_wait_limit.argtypes = [_vp, ctypes.c_int64, _vp]
lib.hippo_attention_mass_workspace_bytes.restype = _sz
lib.hippo_attention_mass_workspace_bytes.argtypes = [_i32, _I32P, _i32, _i32, _i32, _i32, _i32]
lib.hippo_attention_mass.restype = _i32
lib.hippo_attention_mass.argtypes = [_i32, _I32P, _i32, _i32, _vp, _KVP, _f32, _f32, _vp, _vp, _sz, _vp]
lib.hippo_accept_workspace_bytes.restype = _sz
lib.hippo_accept_workspace_bytes.argtypes = [_i32, _i32, _i32]
lib.hippo_accept.restype = _i32
lib.hippo_accept.argtypes = [_i32, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _i32, _vp, _vp, _vp, _sz, _vp]
lib.hippo_accept_noalloc.restype = _i32
lib.hippo_accept_noalloc.argtypes = [_i32, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _i32, _vp, _vp, _vp]
ACCEPT_NOALLOC_SCRATCH_BYTES = 1024 * 1024

HIPPO_VPSD_OPTIMISTIC = 0
HIPPO_VPSD_CONSERVATIVE = 1
_i64, _f64 = ctypes.c_int64, ctypes.c_double


class VpsdState(ctypes.Structure):
    _fields_ = [("struct_size", _u32), ("gamma", _i32), ("mode", _i32), ("batch", _i32), ("rounds", _i64),
                ("tokens_emitted", _i64), ("tokens_drafted", _i64), ("tokens_discarded", _i64)]


class VpsdRound(ctypes.Structure):
    _fields_ = [("mode", _i32), ("draft_before", _i32), ("verify_tokens", _i32), ("draft_during", _i32),
                ("abort_on_reject", _i32)]


class VpsdOutcome(ctypes.Structure):
    _fields_ = [("accepted", _i32), ("emitted", _i32), ("target_token", _i32), ("keep_drafted", _i32),
                ("next_mode", _i32)]


lib.hippo_vpsd_prefill_buffer.restype = _i32
lib.hippo_vpsd_prefill_buffer.argtypes = [_f64, _f64, _f64]
lib.hippo_vpsd_init.restype = _i32
lib.hippo_vpsd_init.argtypes = [ctypes.POINTER(VpsdState), _i32, _i32]
lib.hippo_vpsd_plan.restype = _i32
lib.hippo_vpsd_plan.argtypes = [ctypes.POINTER(VpsdState), ctypes.POINTER(VpsdRound)]
lib.hippo_vpsd_commit.restype = _i32
lib.hippo_vpsd_commit.argtypes = [ctypes.POINTER(VpsdState), ctypes.POINTER(VpsdRound), _i32, _i32, ctypes.POINTER(VpsdOutcome)]
lib.hippo_vpsd_round_time.restype = _f64
lib.hippo_vpsd_round_time.argtypes = [ctypes.POINTER(VpsdRound), _i32, _f64, _f64]
lib.hippo_vpsd_serial_round_time.restype = _f64
lib.hippo_vpsd_serial_round_time.argtypes = [_i32, _f64, _f64]


class HippoError(RuntimeError):
    def __init__(self, status: int):
        self.status = status
        msg = lib.hippo_last_error().decode()
        super().__init__("%s (%d): %s" % (lib.hippo_status_string(status).decode(), status, msg))


def _check(status: int) -> None:
    if status != HIPPO_OK:
        raise HippoError(status)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream) -> ctypes.c_void_p:
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return HIPPO_DTYPE_FP32
    if t.dtype == torch.bfloat16:
        return HIPPO_DTYPE_BF16
    raise TypeError("unsupported dtype %s" % t.dtype)


def _host_i32(v: Sequence[int]):
    arr = (_i32 * len(v))(*[int(x) for x in v])
    return arr


def hippo_version() -> int:
    return int(lib.hippo_version())


def hippo_launch_count() -> int:
    return int(lib.hippo_launch_count())


class KVCache:
    """Descriptor of one layer's paged cache; keeps the tensors alive.  k_pages, v_pages:
    [n_pages][n_kv_heads][64][head_dim]; page_table int32 [batch][max_pages_per_seq] or None (identity)."""

    def __init__(self, k_pages: torch.Tensor, v_pages: torch.Tensor, page_table: Optional[torch.Tensor],
                 max_pages_per_seq: Optional[int] = None):
        assert k_pages.is_contiguous() and v_pages.is_contiguous() and k_pages.shape == v_pages.shape
        assert k_pages.dim() == 4 and k_pages.shape[2] == PAGE_SIZE
        if page_table is not None:
            assert page_table.dtype == torch.int32 and page_table.is_contiguous() and page_table.dim() == 2
            max_pages_per_seq = page_table.shape[1]
        assert max_pages_per_seq is not None
        self.k_pages, self.v_pages, self.page_table = k_pages, v_pages, page_table
        self.struct = KVCacheStruct(ctypes.sizeof(KVCacheStruct), _dtype_code(k_pages), k_pages.shape[1],
                                    k_pages.shape[3], k_pages.shape[0], int(max_pages_per_seq),
                                    k_pages.data_ptr(), v_pages.data_ptr(),
                                    None if page_table is None else page_table.data_ptr())

    @property
    def n_kv_heads(self) -> int:
        return self.k_pages.shape[1]

    @property
    def head_dim(self) -> int:
        return self.k_pages.shape[3]


def new_workspace(n_bytes: int, device="cuda") -> torch.Tensor:
    """Zero-filled, 256-byte aligned byte buffer (a fresh workspace needs its header zeroed once)."""
    ws = torch.zeros(max(int(n_bytes), 256), dtype=torch.uint8, device=device)
    assert ws.data_ptr() % 256 == 0
    return ws


def hippo_workspace_status(workspace: torch.Tensor, stream=None) -> int:
    return int(lib.hippo_workspace_status(_ptr(workspace), _stream(stream)))


def hippo_workspace_reset(workspace: torch.Tensor, stream=None) -> None:
    _check(lib.hippo_workspace_reset(_ptr(workspace), workspace.numel(), _stream(stream)))


def hippo_workspace_set_wait_limit(workspace: torch.Tensor, limit_ns: int, stream=None) -> None:
    _check(lib.hippo_workspace_set_wait_limit(_ptr(workspace), int(limit_ns), _stream(stream)))


def hippo_read_probe(buffer: torch.Tensor, sink: torch.Tensor, stream=None) -> None:
    """One read-only pass over `buffer` (measurement aid); `sink`: 256 bytes of device memory."""
    assert sink.numel() * sink.element_size() >= 256
    _check(lib.hippo_read_probe(_ptr(buffer), buffer.numel() * buffer.element_size(), _ptr(sink), _stream(stream)))


# ---- selection --------------------------------------------------------------------------------------------------

def hippo_select_workspace_bytes(n_visual: Sequence[int], grid_h: int, grid_w: int, crop_h: int = 5, crop_w: int = 5) -> int:
    return int(lib.hippo_select_workspace_bytes(len(n_visual), _host_i32(n_visual), grid_h, grid_w, crop_h, crop_w))


def hippo_select_tokens(embeds: Optional[torch.Tensor], attn_mass: Optional[torch.Tensor], n_visual: Sequence[int],
                        k: Sequence[int], grid_h: int, grid_w: int, crop_h: int = 5, crop_w: int = 5,
                        score_mask: int = HIPPO_SCORE_ALL, kept_idx: Optional[torch.Tensor] = None,
                        kept_offsets: Optional[Sequence[int]] = None, fused_score: Optional[torch.Tensor] = None,
                        workspace: Optional[torch.Tensor] = None, stream=None, policy: int = HIPPO_SELECT_HOLISTIC,
                        random_keys: Optional[torch.Tensor] = None, embed_dim: Optional[int] = None,
                        device=None) -> Tuple[torch.Tensor, Optional[torch.Tensor]]:
    """embeds [sum n_visual][d]; attn_mass fp32 [sum n_visual].  Returns (kept_idx int32 [sum k], fused fp32).
    policy != HIPPO_SELECT_HOLISTIC goes through hippo_select_tokens_policy (random_keys: fp32 [sum n_visual]); the
    policies that score nothing accept embeds = attn_mass = None (then pass `device`)."""
    total = int(sum(n_visual))
    if embeds is not None:
        assert embeds.is_contiguous() and embeds.shape[0] == total
        device, embed_dim = embeds.device, embeds.shape[1]
    if attn_mass is not None:
        assert attn_mass.is_contiguous() and attn_mass.dtype == torch.float32 and attn_mass.shape[0] == total
    if random_keys is not None:
        assert random_keys.is_contiguous() and random_keys.dtype == torch.float32 and random_keys.shape[0] == total
        device = random_keys.device
    device = torch.device("cuda") if device is None else device
    if kept_idx is None:
        kept_idx = torch.empty(max(int(sum(k)), 1), dtype=torch.int32, device=device)
    if fused_score is None and policy != HIPPO_SELECT_FRAMES:
        fused_score = torch.empty(total, dtype=torch.float32, device=device)
    if workspace is None:
        workspace = new_workspace(hippo_select_workspace_bytes(n_visual, grid_h, grid_w, crop_h, crop_w), device)
    common = (len(n_visual), _host_i32(n_visual), grid_h, grid_w, crop_h, crop_w, 8 if embed_dim is None else int(embed_dim),
              HIPPO_DTYPE_BF16 if embeds is None else _dtype_code(embeds), _ptr(embeds), _ptr(attn_mass), _host_i32(k),
              None if kept_offsets is None else _host_i32(kept_offsets), score_mask)
    tail = (_ptr(kept_idx), _ptr(fused_score), _ptr(workspace), workspace.numel(), _stream(stream))
    if policy == HIPPO_SELECT_HOLISTIC and random_keys is None:
        _check(lib.hippo_select_tokens(*common, *tail))
    else:
        _check(lib.hippo_select_tokens_policy(*common, int(policy), _ptr(random_keys), *tail))
    return (kept_idx[:int(sum(k))] if kept_offsets is None else kept_idx), fused_score


# ---- gather -------------------------------------------------------------------------------------------------------

def hippo_gather_kv(n_layers: int, src: KVCache, src_layer_stride_bytes: int, dst: KVCache, dst_layer_stride_bytes: int,
                    batch: int, keep_idx: torch.Tensor, keep_offsets: torch.Tensor, total_keep: int,
                    bad_index: Optional[torch.Tensor] = None, stream=None) -> None:
    """bad_index: optional int32 device word (zeroed by the caller) that the kernel sets when it skipped an
    out-of-range entry."""
    assert keep_idx.dtype == torch.int32 and keep_offsets.dtype == torch.int32
    assert bad_index is None or bad_index.dtype == torch.int32
    _check(lib.hippo_gather_kv(n_layers, ctypes.byref(src.struct), src_layer_stride_bytes, ctypes.byref(dst.struct),
                               dst_layer_stride_bytes, batch, _ptr(keep_idx), _ptr(keep_offsets), int(total_keep),
                               _ptr(bad_index), _stream(stream)))


# ---- attention ----------------------------------------------------------------------------------------------------

def hippo_attention_workspace_bytes(batch: int, q_len: int, n_q_heads: int, n_kv_heads: int, head_dim: int) -> int:
    return int(lib.hippo_attention_workspace_bytes(batch, q_len, n_q_heads, n_kv_heads, head_dim))


def _attention(fn, q, kv, kv_len, max_kv_len, softmax_scale, num_splits, out, lse, workspace, stream, kv_len_host=None):
    assert q.is_contiguous() and q.dim() == 4 and (kv_len is None or kv_len.dtype == torch.int32)
    B, q_len, hq, d = q.shape
    assert d == kv.head_dim and _dtype_code(q) == kv.struct.dtype
    if out is None:
        out = torch.empty_like(q)
    if workspace is None:
        workspace = new_workspace(hippo_attention_workspace_bytes(B, q_len, hq, kv.n_kv_heads, d), q.device)
    _check(fn(B, q_len, hq, _ptr(q), ctypes.byref(kv.struct), _ptr(kv_len),
              None if kv_len_host is None else _host_i32(kv_len_host), int(max_kv_len), float(softmax_scale),
              int(num_splits), _ptr(out), _ptr(lse), _ptr(workspace), workspace.numel(), _stream(stream)))
    return out


def hippo_verify_attention(q: torch.Tensor, kv: KVCache, kv_len: torch.Tensor, max_kv_len: int,
                           softmax_scale: float = 0.0, num_splits: int = 0, out: Optional[torch.Tensor] = None,
                           lse: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None, stream=None,
                           kv_len_host: Optional[Sequence[int]] = None):
    return _attention(lib.hippo_verify_attention, q, kv, kv_len, max_kv_len, softmax_scale, num_splits, out, lse,
                      workspace, stream, kv_len_host)


def hippo_draft_attention(q: torch.Tensor, kv: KVCache, kv_len: torch.Tensor, max_kv_len: int,
                          softmax_scale: float = 0.0, num_splits: int = 0, out: Optional[torch.Tensor] = None,
                          lse: Optional[torch.Tensor] = None, workspace: Optional[torch.Tensor] = None, stream=None,
                          kv_len_host: Optional[Sequence[int]] = None):
    return _attention(lib.hippo_draft_attention, q, kv, kv_len, max_kv_len, softmax_scale, num_splits, out, lse,
                      workspace, stream, kv_len_host)


def hippo_verify_attention_layers_workspace_bytes(n_layers: int, batch: int, q_len: int, n_q_heads: int, n_kv_heads: int,
                                                  head_dim: int) -> int:
    return int(lib.hippo_verify_attention_layers_workspace_bytes(n_layers, batch, q_len, n_q_heads, n_kv_heads, head_dim))


def hippo_verify_attention_layers(q_layers: Sequence[torch.Tensor], kv_layers: Sequence[KVCache], kv_len: Optional[torch.Tensor],
                                  max_kv_len: int, out_layers: Sequence[torch.Tensor], softmax_scale: float = 0.0,
                                  lse_layers: Optional[Sequence[Optional[torch.Tensor]]] = None,
                                  workspace: Optional[torch.Tensor] = None, stream=None,
                                  kv_len_host: Optional[Sequence[int]] = None, max_ctas: int = 0):
    """The verification attention of several layers in one launch: out_layers[l] = attention(q_layers[l], kv_layers[l]).
    max_ctas > 0 bounds the grid, leaving the other SMs to kernels of other streams."""
    n = len(q_layers)
    assert n == len(kv_layers) == len(out_layers) and n > 0
    B, q_len, hq, d = q_layers[0].shape
    for q, o in zip(q_layers, out_layers):
        assert q.is_contiguous() and o.is_contiguous() and q.shape == (B, q_len, hq, d) and o.shape == q.shape and o.dtype == q.dtype
    assert kv_len is None or kv_len.dtype == torch.int32
    if workspace is None:
        workspace = new_workspace(hippo_verify_attention_layers_workspace_bytes(n, B, q_len, hq, kv_layers[0].n_kv_heads, d),
                                  q_layers[0].device)
    qp = (_vp * n)(*[t.data_ptr() for t in q_layers])
    op = (_vp * n)(*[t.data_ptr() for t in out_layers])
    lp = None
    if lse_layers is not None:
        lp = (_vp * n)(*[None if t is None else t.data_ptr() for t in lse_layers])
    kvs = (KVCacheStruct * n)(*[c.struct for c in kv_layers])
    _check(lib.hippo_verify_attention_layers(n, B, q_len, hq, qp, kvs, _ptr(kv_len),
                                             None if kv_len_host is None else _host_i32(kv_len_host), int(max_kv_len),
                                             float(softmax_scale), int(max_ctas), op, lp, _ptr(workspace), workspace.numel(),
                                             _stream(stream)))
    return out_layers


# ---- global semantic relevance (Eq. 2) ----------------------------------------------------------------------------

def hippo_attention_mass_workspace_bytes(n_visual: Sequence[int], l_txt: int, n_q_heads: int, n_kv_heads: int,
                                         head_dim: int, dtype: int) -> int:
    return int(lib.hippo_attention_mass_workspace_bytes(len(n_visual), _host_i32(n_visual), l_txt, n_q_heads,
                                                        n_kv_heads, head_dim, dtype))


def hippo_attention_mass(q_txt: torch.Tensor, kv: "KVCache", n_visual: Sequence[int], weight: float,
                         mass: torch.Tensor, softmax_scale: float = 0.0, workspace: Optional[torch.Tensor] = None,
                         stream=None) -> torch.Tensor:
    """One layer's share of Eq. 2, added into `mass` (fp32 [sum n_visual]).  q_txt [B][l_txt][H_q][D]."""
    B, l_txt, hq, D = q_txt.shape
    assert q_txt.is_contiguous() and mass.dtype == torch.float32 and mass.is_contiguous()
    assert len(n_visual) == B and mass.numel() >= sum(int(x) for x in n_visual)
    if workspace is None:
        workspace = new_workspace(hippo_attention_mass_workspace_bytes(n_visual, l_txt, hq, kv.struct.n_kv_heads,
                                                                        D, _dtype_code(q_txt)), q_txt.device)
    _check(lib.hippo_attention_mass(B, _host_i32(n_visual), l_txt, hq, _ptr(q_txt), ctypes.byref(kv.struct),
                                    float(softmax_scale), float(weight), _ptr(mass), _ptr(workspace),
                                    workspace.numel(), _stream(stream)))
    return mass


# ---- decoding schedule (Section 5.2), host only -------------------------------------------------------------------

def hippo_vpsd_prefill_buffer(prefill_target: float, prefill_draft: float, t_draft: float) -> int:
    return int(lib.hippo_vpsd_prefill_buffer(prefill_target, prefill_draft, t_draft))


def hippo_vpsd_init(gamma: int, buffered_tokens: int = 0) -> VpsdState:
    st = VpsdState()
    _check(lib.hippo_vpsd_init(ctypes.byref(st), gamma, buffered_tokens))
    return st


def hippo_vpsd_plan(state: VpsdState) -> VpsdRound:
    rd = VpsdRound()
    _check(lib.hippo_vpsd_plan(ctypes.byref(state), ctypes.byref(rd)))
    return rd


def hippo_vpsd_commit(state: VpsdState, rnd: VpsdRound, n_accepted: int, drafted_during: Optional[int] = None) -> VpsdOutcome:
    out = VpsdOutcome()
    d = rnd.draft_during if drafted_during is None else drafted_during
    _check(lib.hippo_vpsd_commit(ctypes.byref(state), ctypes.byref(rnd), int(n_accepted), int(d), ctypes.byref(out)))
    return out


def hippo_vpsd_round_time(rnd: VpsdRound, n_accepted: int, t_draft: float, t_target: float) -> float:
    return float(lib.hippo_vpsd_round_time(ctypes.byref(rnd), int(n_accepted), t_draft, t_target))


def hippo_vpsd_serial_round_time(gamma: int, t_draft: float, t_target: float) -> float:
    return float(lib.hippo_vpsd_serial_round_time(gamma, t_draft, t_target))


# ---- acceptance ---------------------------------------------------------------------------------------------------

def hippo_accept_workspace_bytes(batch: int, gamma: int, vocab: int) -> int:
    return int(lib.hippo_accept_workspace_bytes(batch, gamma, vocab))


def hippo_accept(target_logits: torch.Tensor, draft_logits: Optional[torch.Tensor], draft_tokens: torch.Tensor,
                 u_accept: Optional[torch.Tensor], u_resample: Optional[torch.Tensor],
                 n_accepted: Optional[torch.Tensor] = None, out_tokens: Optional[torch.Tensor] = None,
                 workspace: Optional[torch.Tensor] = None, stream=None, mode: int = HIPPO_ACCEPT_SAMPLE
                 ) -> Tuple[torch.Tensor, torch.Tensor]:
    """mode HIPPO_ACCEPT_SAMPLE: Eq. 1 with residual resampling; HIPPO_ACCEPT_GREEDY: arg-max matching (draft_logits
    and the uniforms may be None)."""
    B, g1, V = target_logits.shape
    g = g1 - 1
    for t in (target_logits, draft_logits, u_accept, u_resample):
        assert t is None or (t.dtype == torch.float32 and t.is_contiguous())
    assert draft_tokens.dtype == torch.int32 and draft_tokens.is_contiguous()
    dev = target_logits.device
    if n_accepted is None:
        n_accepted = torch.empty(B, dtype=torch.int32, device=dev)
    if out_tokens is None:
        out_tokens = torch.empty((B, g + 1), dtype=torch.int32, device=dev)
    if workspace is None:
        workspace = new_workspace(hippo_accept_workspace_bytes(B, g, V), dev)
    _check(lib.hippo_accept(B, g, V, _ptr(target_logits), _ptr(draft_logits) if g else None,
                            _ptr(draft_tokens) if g else None, _ptr(u_accept) if g else None, _ptr(u_resample), int(mode),
                            _ptr(n_accepted), _ptr(out_tokens), _ptr(workspace), workspace.numel(), _stream(stream)))
    return n_accepted, out_tokens


def hippo_accept_noalloc(target_logits: torch.Tensor, draft_logits: Optional[torch.Tensor], draft_tokens: torch.Tensor,
                         u_accept: Optional[torch.Tensor], u_resample: Optional[torch.Tensor], n_accepted: torch.Tensor,
                         out_tokens: torch.Tensor, stream=None, mode: int = HIPPO_ACCEPT_SAMPLE
                         ) -> Tuple[torch.Tensor, torch.Tensor]:
    """hippo_accept without a workspace argument, for callers that cannot allocate one (an engine that owns all
    device memory, a host that forbids cudaMalloc in its decode loop).  The scratch is a fixed array inside the
    library, shared by every call on the device; the outputs must be passed in because this wrapper allocates
    nothing either.  Problems needing more than ACCEPT_NOALLOC_SCRATCH_BYTES raise HippoError; calls that may
    overlap on the GPU must be ordered by the caller."""
    B, g1, V = target_logits.shape
    g = g1 - 1
    for t in (target_logits, draft_logits, u_accept, u_resample):
        assert t is None or (t.dtype == torch.float32 and t.is_contiguous())
    assert draft_tokens.dtype == torch.int32 and draft_tokens.is_contiguous()
    assert n_accepted.dtype == torch.int32 and n_accepted.numel() >= B
    assert out_tokens.dtype == torch.int32 and out_tokens.numel() >= B * (g + 1) and out_tokens.is_contiguous()
    _check(lib.hippo_accept_noalloc(B, g, V, _ptr(target_logits), _ptr(draft_logits) if g else None,
                                    _ptr(draft_tokens) if g else None, _ptr(u_accept) if g else None,
                                    _ptr(u_resample), int(mode), _ptr(n_accepted), _ptr(out_tokens), _stream(stream)))
    return n_accepted, out_tokens
