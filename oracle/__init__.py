"""ctypes front-end of the CPU oracle (`hippo_oracle.c`).  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this package; the
CUDA library and its Python binding never do.  The C file is compiled on first use with gcc
(`-O2 -fopenmp`, no hand vectorisation) into `oracle/_build/`.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "hippo_oracle.c")
_OUT_DIR = os.path.join(_HERE, "_build")
_LIB_PATH = os.path.join(_OUT_DIR, "liboracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle if the shared object is missing or older than its source."""
    os.makedirs(_OUT_DIR, exist_ok=True)
    stale = force or not os.path.exists(_LIB_PATH) or os.path.getmtime(_LIB_PATH) < os.path.getmtime(_SRC)
    if stale:
        tmp = _LIB_PATH + ".%d.tmp" % os.getpid()
        subprocess.check_call(["gcc", "-std=c99", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_max_threads.restype = ctypes.c_int
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32)


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int32)


def max_threads() -> int:
    return int(_load().oracle_max_threads())


def set_threads(n: int) -> None:
    _load().oracle_set_threads(ctypes.c_int(n))


def select_scores(embeds, attn_mass, grid_h: int, grid_w: int, crop_h: int = 5, crop_w: int = 5,
                  score_mask: int = 7) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Eq. 3-7.  Returns (fused, s_temp, s_spa), each float64 [n_visual]."""
    E = _f32(embeds)
    n, d = E.shape
    am = _f32(attn_mass)
    assert am.shape == (n,)
    fused, st, ss = (np.empty(n, dtype=np.float64) for _ in range(3))
    rc = _load().oracle_select_scores(n, grid_h, grid_w, crop_h, crop_w, d, _p(E), _p(am),
                                      ctypes.c_uint(score_mask), _p(st), _p(ss), _p(fused))
    if rc != 0:
        raise ValueError("oracle_select_scores rc=%d" % rc)
    return fused, st, ss


def topk(score, k: int) -> Tuple[np.ndarray, float]:
    """Indices (ascending) of the k best by (score desc, index asc), and the k-th best score."""
    s = np.ascontiguousarray(score, dtype=np.float64)
    idx = np.empty(k, dtype=np.int32)
    kth = ctypes.c_double(0.0)
    rc = _load().oracle_topk(s.shape[0], _p(s), k, _p(idx), ctypes.byref(kth))
    if rc != 0:
        raise ValueError("oracle_topk rc=%d" % rc)
    return idx, float(kth.value)


def select_tokens(embeds, attn_mass, k: int, grid_h: int, grid_w: int, crop_h: int = 5, crop_w: int = 5,
                  score_mask: int = 7):
    """Selection end to end: returns (kept_idx ascending int32[k], fused float64[n], kth_score)."""
    fused, _, _ = select_scores(embeds, attn_mass, grid_h, grid_w, crop_h, crop_w, score_mask)
    idx, kth = topk(fused, k)
    return idx, fused, kth


POLICY_HOLISTIC, POLICY_UNIFORM_PER_FRAME, POLICY_RANDOM, POLICY_FRAME = 0, 1, 2, 3


def select_policy(policy: int, score, k: int, tokens_per_frame: int):
    """The kept indices (ascending) under one of the selection rules; `score` is the fused score (policies 0, 1), the
    caller's random keys (policy 2) or ignored (policy 3).  Returns (kept int32[k], per-frame budget int32[F])."""
    s = np.ascontiguousarray(score, dtype=np.float64)
    n = s.shape[0]
    idx = np.empty(k, dtype=np.int32)
    budget = np.zeros((n + tokens_per_frame - 1) // tokens_per_frame, dtype=np.int32)
    rc = _load().oracle_select_policy(policy, n, tokens_per_frame, _p(s), k, _p(idx), _p(budget))
    if rc != 0:
        raise ValueError("oracle_select_policy rc=%d" % rc)
    return idx, budget


def gather_kv(src, keep) -> np.ndarray:
    """src [n_layers][n_src][...row...] (any dtype) -> dst [n_layers][len(keep)][...row...]."""
    s = np.ascontiguousarray(src)
    kp = _i32(keep)
    L, n_src = s.shape[0], s.shape[1]
    row_bytes = int(np.prod(s.shape[2:], dtype=np.int64)) * s.dtype.itemsize
    dst = np.empty((L, kp.shape[0]) + s.shape[2:], dtype=s.dtype)
    rc = _load().oracle_gather_kv(L, n_src, kp.shape[0], row_bytes, _p(kp), _p(s), _p(dst))
    if rc != 0:
        raise ValueError("oracle_gather_kv rc=%d" % rc)
    return dst


def attention(q, k, v, kv_len: Sequence[int], scale: Optional[float] = None, rows=None
              ) -> Tuple[np.ndarray, np.ndarray]:
    """softmax(q K^T scale) V with GQA and a bottom-right-aligned causal tail.

    q [B][q_len][H_q][D]; k, v [B][max_kv][H_kv][D].  Returns (out, lse) as float64:
    all rows ([B][q_len][H_q][D], [B][q_len][H_q]) or, when `rows` = list of (b, t, h), only those
    ([n][D], [n]).
    """
    q, k, v = _f32(q), _f32(k), _f32(v)
    B, q_len, Hq, D = q.shape
    _, max_kv, Hkv, _ = k.shape
    kl = _i32(kv_len)
    sc = ctypes.c_double(1.0 / np.sqrt(D) if scale is None else scale)
    lib = _load()
    if rows is None:
        out = np.empty((B, q_len, Hq, D), dtype=np.float64)
        lse = np.empty((B, q_len, Hq), dtype=np.float64)
        rc = lib.oracle_attention(B, q_len, Hq, Hkv, D, max_kv, _p(kl), _p(q), _p(k), _p(v), sc, _p(out), _p(lse))
    else:
        r = np.asarray(rows, dtype=np.int32).reshape(-1, 3)
        sb, st, sh = (_i32(r[:, i]) for i in range(3))
        out = np.empty((r.shape[0], D), dtype=np.float64)
        lse = np.empty((r.shape[0],), dtype=np.float64)
        rc = lib.oracle_attention_rows(r.shape[0], _p(sb), _p(st), _p(sh), q_len, Hq, Hkv, D, max_kv, _p(kl), _p(q),
                                       _p(k), _p(v), sc, _p(out), _p(lse))
    if rc != 0:
        raise ValueError("oracle_attention rc=%d" % rc)
    return out, lse


def attention_mass(q_txt, k_vid, n_visual: Sequence[int], scale: Optional[float] = None) -> np.ndarray:
    """Eq. 2: mean over layers, heads and text rows of softmax_j(scale q_i . k_j) over the visual keys.

    q_txt [n_layers][B][L_txt][H_q][D]; k_vid [n_layers][B][max_nv][H_kv][D].  Returns float64 [B][max_nv]
    (zeros at and beyond n_visual[b]).
    """
    q, k = _f32(q_txt), _f32(k_vid)
    nl, B, L_txt, Hq, D = q.shape
    _, _, max_nv, Hkv, _ = k.shape
    nv = _i32(n_visual)
    sc = ctypes.c_double(1.0 / np.sqrt(D) if scale is None else scale)
    mass = np.empty((B, max_nv), dtype=np.float64)
    rc = _load().oracle_attention_mass(nl, B, L_txt, Hq, Hkv, D, max_nv, _p(nv), _p(q), _p(k), sc, _p(mass))
    if rc != 0:
        raise ValueError("oracle_attention_mass rc=%d" % rc)
    return mass


def accept(target_logits, draft_logits, draft_tokens, u_accept, u_resample):
    """Eq. 1 + residual resample / bonus.  Returns (n_accepted [B], out_tokens [B][gamma+1],
    margin_accept [B], margin_cdf [B])."""
    tl, dl = _f32(target_logits), _f32(draft_logits)
    B, g1, V = tl.shape
    g = g1 - 1
    assert dl.shape == (B, g, V)
    x, ua, ur = _i32(draft_tokens).reshape(B, g), _f32(u_accept).reshape(B, g), _f32(u_resample).reshape(B)
    n = np.empty(B, dtype=np.int32)
    out = np.empty((B, g + 1), dtype=np.int32)
    ma, mc = np.empty(B, dtype=np.float64), np.empty(B, dtype=np.float64)
    rc = _load().oracle_accept(B, g, V, _p(tl), _p(dl), _p(x), _p(ua), _p(ur), _p(n), _p(out), _p(ma), _p(mc))
    if rc != 0:
        raise ValueError("oracle_accept rc=%d" % rc)
    return n, out, ma, mc


def accept_greedy(target_logits, draft_tokens):
    """Greedy verification: keep draft tokens while they equal the arg-max of the target row, then emit the
    target's arg-max.  Returns (n_accepted [B], out_tokens [B][gamma+1])."""
    tl = _f32(target_logits)
    B, g1, V = tl.shape
    g = g1 - 1
    x = _i32(draft_tokens).reshape(B, g)
    n = np.empty(B, dtype=np.int32)
    out = np.empty((B, g + 1), dtype=np.int32)
    rc = _load().oracle_accept_greedy(B, g, V, _p(tl), _p(x), _p(n), _p(out))
    if rc != 0:
        raise ValueError("oracle_accept_greedy rc=%d" % rc)
    return n, out
