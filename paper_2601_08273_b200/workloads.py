"""Seeded synthetic inputs shaped like HIPPO's video workloads, plus storage-layout packing.

This module is the one piece shared by the CUDA path's tests/bench and by the CPU oracle's tests:
it draws random inputs, rounds them to the storage dtype and lays them out. It contains none of the
method's arithmetic (no scores, no attention, no acceptance test) and imports neither the CUDA
binding nor the oracle. numpy only.

The five configurations follow the benchmark definition of this repository (a tiny fp32 case, a
7B-class single video, a long video, ragged batched serving on a paged cache, a 70B-class extreme
context). Their shapes mirror the paper's set-up (Appendix "Details of Experimental Setups":
196 = 14x14 tokens per frame at 64 or 128 frames, 7B draft / 72B-class target, gamma in {3,5,7},
pruning ratio 90 %, crop 5x5, batch 1) and stand in for the Video-MME / VDC / MVBench /
LongVideoBench / MLVU / LVBench videos and the trained checkpoints, none of which are available.
"""
from __future__ import annotations

import dataclasses
from dataclasses import dataclass
from typing import Dict, List, Optional, Tuple

import numpy as np

PAGE_SIZE = 64


@dataclass(frozen=True)
class HippoConfig:
    name: str
    seed: int
    batch: int
    frames: int          # maximum number of frames (grid capacity)
    grid_h: int
    grid_w: int
    n_text: int
    embed_dim: int
    dtype: str           # "fp32" | "bf16": storage type of embeddings, q, K, V
    tgt_q_heads: int
    tgt_kv_heads: int
    tgt_head_dim: int
    tgt_layers: int
    dft_q_heads: int
    dft_kv_heads: int
    dft_head_dim: int
    dft_layers: int      # the benchmark definition gives no draft depth; 28 is a labelled default
    gamma: int
    keep_pct: int        # percent of visual tokens kept (100 - pruning ratio)
    vocab: int
    logit_sigma: float
    mass_kind: str       # "softmax_boundary" (c0) | "zipf_boundary" (c1..c4)
    paged_shuffle: bool  # True: page ids are a seeded random permutation of the pool (c3)
    ragged: Optional[Tuple[int, int]] = None  # inclusive range of per-sequence visual lengths
    crop_h: int = 5
    crop_w: int = 5

    @property
    def tokens_per_frame(self) -> int:
        return self.grid_h * self.grid_w

    def replace(self, **kw) -> "HippoConfig":
        return dataclasses.replace(self, **kw)


CONFIGS: List[HippoConfig] = [
    HippoConfig("c0_tiny_fp32", 0, 1, 4, 8, 8, 32, 64, "fp32", 4, 1, 64, 1, 2, 1, 64, 1,
                4, 10, 1000, 2.0, "softmax_boundary", False),
    HippoConfig("c1_7b_video_6k", 1, 1, 32, 14, 14, 128, 3584, "bf16", 28, 4, 128, 28, 14, 2, 64, 28,
                5, 10, 152064, 3.0, "zipf_boundary", False),
    HippoConfig("c2_long_video_32k", 2, 1, 128, 16, 16, 256, 4096, "bf16", 32, 8, 128, 36, 16, 2, 64, 28,
                7, 10, 152064, 3.0, "zipf_boundary", False),
    HippoConfig("c3_batched_paged", 3, 8, 64, 14, 14, 128, 3584, "bf16", 28, 4, 128, 28, 14, 2, 64, 28,
                5, 10, 152064, 3.0, "zipf_boundary", True, ragged=(8000, 12544)),
    HippoConfig("c4_70b_64k", 4, 1, 256, 16, 16, 256, 8192, "bf16", 64, 8, 128, 80, 16, 2, 64, 28,
                5, 10, 152064, 3.0, "zipf_boundary", False),
]
C4_GAMMA_SWEEP = (3, 5, 8)
C4_KEEP_PCT_SWEEP = (50, 25, 10, 5)


def rng_for(cfg: HippoConfig, tag: int, sub: int = 0) -> np.random.Generator:
    """Independent stream per (config seed, purpose tag, sub-index)."""
    return np.random.default_rng([cfg.seed, tag, sub])


TAG_LEN, TAG_EMB, TAG_MASS, TAG_ATT_T, TAG_ATT_D, TAG_ACC, TAG_PAGES, TAG_GATHER, TAG_QTXT = range(9)

# ------------------------------------------------------------------------------------------------
# storage rounding
# ------------------------------------------------------------------------------------------------

def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit patterns (uint16), round to nearest even. Finite inputs only."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def from_bf16_bits(b: np.ndarray) -> np.ndarray:
    """bf16 bit patterns -> the exactly equal fp32 values."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def round_to_storage(x: np.ndarray, dtype: str) -> np.ndarray:
    """Return fp32 values that are exactly representable in the storage dtype."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    if dtype == "fp32":
        return x
    if dtype == "bf16":
        return from_bf16_bits(to_bf16_bits(x))
    raise ValueError(dtype)


def storage_bits(x: np.ndarray, dtype: str) -> np.ndarray:
    """The bytes handed to the GPU: fp32 array as is, or uint16 bf16 bit patterns."""
    if dtype == "fp32":
        return np.ascontiguousarray(x, dtype=np.float32)
    return to_bf16_bits(x)


def normal_f32(rng: np.random.Generator, shape, sigma: float = 1.0) -> np.ndarray:
    x = rng.standard_normal(shape, dtype=np.float32)
    if sigma != 1.0:
        x *= np.float32(sigma)
    return x

# ------------------------------------------------------------------------------------------------
# lengths and keep counts
# ------------------------------------------------------------------------------------------------

def visual_lengths(cfg: HippoConfig) -> List[int]:
    if cfg.ragged is None:
        return [cfg.frames * cfg.tokens_per_frame] * cfg.batch
    lo, hi = cfg.ragged
    r = rng_for(cfg, TAG_LEN)
    return [int(v) for v in r.integers(lo, hi + 1, size=cfg.batch)]


def keep_count(n_visual: int, keep_pct: int) -> int:
    """k = round(n_visual * keep_pct / 100) in integer arithmetic (halves round up)."""
    return (n_visual * keep_pct + 50) // 100


def is_boundary(cfg: HippoConfig, n_visual: int) -> np.ndarray:
    """True for tokens on the first/last row or column of their frame's patch grid."""
    j = np.arange(n_visual)
    cell = j % cfg.tokens_per_frame
    y, x = cell // cfg.grid_w, cell % cfg.grid_w
    return (y == 0) | (y == cfg.grid_h - 1) | (x == 0) | (x == cfg.grid_w - 1)

# ------------------------------------------------------------------------------------------------
# selection inputs
# ------------------------------------------------------------------------------------------------

def attention_mass(cfg: HippoConfig, n_visual: int, b: int = 0) -> np.ndarray:
    """Synthetic per-visual-token attention mass (fp32, sums to 1) with inflated frame borders."""
    r = rng_for(cfg, TAG_MASS, b)
    bd = is_boundary(cfg, n_visual)
    if cfg.mass_kind == "softmax_boundary":
        logit = r.standard_normal(n_visual)
        logit = logit + 3.0 * bd
        w = np.exp(logit - logit.max())
    elif cfg.mass_kind == "zipf_boundary":
        rank = r.permutation(n_visual) + 1
        w = rank.astype(np.float64) ** -1.1
        w = w * np.where(bd, 4.0, 1.0)
    else:
        raise ValueError(cfg.mass_kind)
    return (w / w.sum()).astype(np.float32)


def select_inputs(cfg: HippoConfig, b: int = 0, n_visual: Optional[int] = None) -> Dict[str, object]:
    n_v = visual_lengths(cfg)[b] if n_visual is None else n_visual
    r = rng_for(cfg, TAG_EMB, b)
    emb = round_to_storage(normal_f32(r, (n_v, cfg.embed_dim)), cfg.dtype)
    return {"n_visual": n_v, "embeds": emb, "attn_mass": attention_mass(cfg, n_v, b),
            "k": keep_count(n_v, cfg.keep_pct)}

def mass_inputs(cfg: HippoConfig, n_visual: List[int], layer: int = 0) -> Dict[str, np.ndarray]:
    """Text queries and visual keys of one target layer for the global-relevance score.

    q_txt [B][n_text][H_q][D], k_vid [B][max(n_visual)][H_kv][D].  Both are N(0,1) plus a component along one shared
    direction sized so that the resulting text-to-visual attention follows the configuration's mass profile
    (power law with inflated frame borders) up to the random part of the logits."""
    hq, hkv, d = cfg.tgt_q_heads, cfg.tgt_kv_heads, cfg.tgt_head_dim
    r = rng_for(cfg, TAG_QTXT, layer)
    B, T = len(n_visual), max(max(n_visual), 1)
    u = r.standard_normal(d)
    u = (u / np.linalg.norm(u)).astype(np.float32)
    q = normal_f32(r, (B, cfg.n_text, hq, d)) + np.float32(4.0) * u
    k = normal_f32(r, (B, T, hkv, d))
    scale = 1.0 / np.sqrt(d)
    for b, nv in enumerate(n_visual):
        if nv <= 0:
            continue
        w = attention_mass(cfg, nv, b).astype(np.float64)
        bias = np.log(w / w.max()) / (4.0 * scale)
        k[b, :nv] += (bias[:, None, None] * u[None, None, :]).astype(np.float32)
    return {"q_txt": round_to_storage(q, cfg.dtype), "k_vid": round_to_storage(k, cfg.dtype)}


# ------------------------------------------------------------------------------------------------
# attention inputs (logical layout [B][T][H_kv][D]) and the paged pool layout
# ------------------------------------------------------------------------------------------------

def attention_inputs(cfg: HippoConfig, which: str, kv_lens: List[int], q_len: int, layer: int = 0
                     ) -> Dict[str, np.ndarray]:
    """q [B][q_len][H_q][D]; k, v [B][max(kv_lens)][H_kv][D] (entries past kv_len are drawn too but unused)."""
    if which == "target":
        hq, hkv, d, tag = cfg.tgt_q_heads, cfg.tgt_kv_heads, cfg.tgt_head_dim, TAG_ATT_T
    else:
        hq, hkv, d, tag = cfg.dft_q_heads, cfg.dft_kv_heads, cfg.dft_head_dim, TAG_ATT_D
    r = rng_for(cfg, tag, layer)
    B, T = len(kv_lens), max(kv_lens)
    q = round_to_storage(normal_f32(r, (B, q_len, hq, d)), cfg.dtype)
    k = round_to_storage(normal_f32(r, (B, T, hkv, d)), cfg.dtype)
    v = round_to_storage(normal_f32(r, (B, T, hkv, d)), cfg.dtype)
    return {"q": q, "k": k, "v": v}


def pages_needed(n_tokens: int, page_size: int = PAGE_SIZE) -> int:
    return (n_tokens + page_size - 1) // page_size


def make_page_table(kv_caps: List[int], shuffle_rng: Optional[np.random.Generator],
                    page_size: int = PAGE_SIZE, spare_pages: int = 0) -> Tuple[np.ndarray, int]:
    """Page table int32 [B][max_pages] (-1 = unused) and pool size. Identity order unless shuffled."""
    per = [pages_needed(c, page_size) for c in kv_caps]
    n_pool = sum(per) + spare_pages
    ids = np.arange(n_pool, dtype=np.int32)
    if shuffle_rng is not None:
        ids = shuffle_rng.permutation(n_pool).astype(np.int32)
    table = np.full((len(kv_caps), max(per) if per else 0), -1, dtype=np.int32)
    o = 0
    for b, p in enumerate(per):
        table[b, :p] = ids[o:o + p]
        o += p
    return table, n_pool


def pack_paged(x: np.ndarray, lens: List[int], table: np.ndarray, n_pool: int,
               page_size: int = PAGE_SIZE, fill: float = 0.0) -> np.ndarray:
    """Logical [B][T][H][D] -> pool [n_pool][H][page_size][D]. Slots past a sequence's length get `fill`."""
    B, T, H, D = x.shape
    pool = np.full((n_pool, H, page_size, D), fill, dtype=x.dtype)
    for b in range(B):
        n = lens[b]
        for p in range(pages_needed(n, page_size)):
            lo, hi = p * page_size, min((p + 1) * page_size, n)
            pool[table[b, p], :, :hi - lo, :] = np.transpose(x[b, lo:hi], (1, 0, 2))
    return pool


def unpack_paged(pool: np.ndarray, lens: List[int], table: np.ndarray, page_size: int = PAGE_SIZE
                 ) -> np.ndarray:
    """Pool [n_pool][H][page_size][D] -> logical [B][max(lens)][H][D] (zeros past each length)."""
    _, H, _, D = pool.shape
    B, T = len(lens), max(lens) if lens else 0
    out = np.zeros((B, T, H, D), dtype=pool.dtype)
    for b in range(B):
        n = lens[b]
        for p in range(pages_needed(n, page_size)):
            lo, hi = p * page_size, min((p + 1) * page_size, n)
            out[b, lo:hi] = np.transpose(pool[table[b, p], :, :hi - lo, :], (1, 0, 2))
    return out

# ------------------------------------------------------------------------------------------------
# acceptance inputs
# ------------------------------------------------------------------------------------------------

def _sample_rows(logits: np.ndarray, u: np.ndarray) -> np.ndarray:
    """Harness-side draw of the draft tokens: inverse CDF of softmax(logits) per row (fp64)."""
    z = logits.astype(np.float64)
    z = np.exp(z - z.max(axis=-1, keepdims=True))
    c = np.cumsum(z, axis=-1)
    tgt = u[..., None] * c[..., -1:]
    idx = (c <= tgt).sum(axis=-1)
    return np.minimum(idx, logits.shape[-1] - 1).astype(np.int32)


def accept_inputs(cfg: HippoConfig, batch: Optional[int] = None, gamma: Optional[int] = None,
                  vocab: Optional[int] = None, corr_eps: Optional[float] = None, sub: int = 0
                  ) -> Dict[str, np.ndarray]:
    """Target logits [B][gamma+1][V], draft logits [B][gamma][V] (fp32), draft tokens, uniforms.

    corr_eps=None draws independent target and draft logits (as the benchmark definition states);
    otherwise draft = target[:gamma] + corr_eps * N(0,1), which exercises long accepted prefixes.
    """
    B = cfg.batch if batch is None else batch
    g = cfg.gamma if gamma is None else gamma
    V = cfg.vocab if vocab is None else vocab
    r = rng_for(cfg, TAG_ACC, sub)
    tl = normal_f32(r, (B, g + 1, V), cfg.logit_sigma)
    if corr_eps is None:
        dl = normal_f32(r, (B, g, V), cfg.logit_sigma)
    else:
        dl = (tl[:, :g, :] + np.float32(corr_eps) * normal_f32(r, (B, g, V))).astype(np.float32)
    u_tok = r.random((B, g))
    x = _sample_rows(dl, u_tok)
    u_acc = r.random((B, g), dtype=np.float32)
    u_res = r.random((B,), dtype=np.float32)
    return {"target_logits": tl, "draft_logits": dl, "draft_tokens": x, "u_accept": u_acc, "u_resample": u_res}
