"""One HIPPO speculative-decoding step on one GPU: buffers for a configuration and the launch sequence.

    one-time per prompt : hippo_select_tokens -> hippo_gather_kv (all draft layers in one launch)
    per decoding round  : stream D: gamma x n_draft_layers x hippo_draft_attention (q_len 1, pruned cache)
                          stream V: the target layers' verification attention (q_len gamma+1, full cache), either
                                    all layers in one hippo_verify_attention_layers call (default) or one
                                    hippo_verify_attention call per layer
                          join -> hippo_accept

In `run()` the verification stream is forked first: it reads neither the selection nor the gathered cache, so it
runs beside select and gather as well as beside the draft calls.

The draft and the verification kernels run on separate CUDA streams, mirroring the paper's decoupled
draft/verify overlap (Section 5.2).  This module only allocates device memory through PyTorch, fills it with
seeded synthetic data and issues the C-ABI calls; every computation is in the CUDA library.  Each layer has its
own KV buffers, so a pass over the layers streams distinct memory (nothing stays resident in L2 for a cache
larger than L2).
"""
from __future__ import annotations

from typing import Dict, List, Optional

import numpy as np
import torch

from . import binding as hb
from . import workloads as W


def _randn(shape, dtype, gen, device):
    return torch.randn(shape, generator=gen, device=device, dtype=torch.float32).to(dtype)


class HippoStep:
    def __init__(self, cfg: W.HippoConfig, device="cuda", target_layers: Optional[int] = None,
                 draft_layers: Optional[int] = None, host_inputs: Optional[Dict[str, np.ndarray]] = None,
                 multi_layer_verify: bool = True, verify_max_ctas: int = 0):
        self.cfg = cfg
        self.multi_layer_verify = multi_layer_verify
        # How run() shares the GPU between its two legs (all three can be changed before run() is called or captured):
        #   verify_max_ctas       grid bound of the multi-layer verification kernel; the SMs it leaves free are where the
        #                         draft stream's kernels run (a persistent CTA holds all of its SM's shared memory)
        #   verify_beside_select  True: verification is forked first and also runs beside select and gather
        #   draft_num_splits      work split of the draft attention calls (0: automatic, which may pick clusters of up to 16
        #                         CTAs that do not fit into a few scattered free SMs)
        self.verify_max_ctas = verify_max_ctas
        self.verify_beside_select = False
        self.draft_num_splits = 0
        self.device = torch.device(device)
        self.Lt = cfg.tgt_layers if target_layers is None else target_layers
        self.Ld = cfg.dft_layers if draft_layers is None else draft_layers
        tdt = torch.float32 if cfg.dtype == "fp32" else torch.bfloat16
        self.tdt = tdt
        gen = torch.Generator(device=self.device)
        gen.manual_seed(1000 + cfg.seed)
        B, g = cfg.batch, cfg.gamma
        self.n_visual: List[int] = W.visual_lengths(cfg)
        self.k: List[int] = [W.keep_count(n, cfg.keep_pct) for n in self.n_visual]
        self.n_keep = [k + cfg.n_text for k in self.k]                      # kept visual + every text position
        self.ctx = [n + cfg.n_text for n in self.n_visual]                  # prompt length
        total_v = sum(self.n_visual)

        # ---- selection inputs
        self.embeds = _randn((total_v, cfg.embed_dim), tdt, gen, self.device)
        mass = np.concatenate([W.attention_mass(cfg, n, b) for b, n in enumerate(self.n_visual)])
        self.attn_mass = torch.from_numpy(mass).to(self.device)
        self.fused = torch.empty(total_v, dtype=torch.float32, device=self.device)
        self.select_ws = hb.new_workspace(hb.hippo_select_workspace_bytes(self.n_visual, cfg.grid_h, cfg.grid_w), self.device)
        # keep list per sequence: [k kept visual | n_text text positions]; the text part is static
        offs = np.concatenate([[0], np.cumsum(self.n_keep)]).astype(np.int32)
        keep = np.zeros(int(offs[-1]), dtype=np.int32)
        for b in range(B):
            keep[offs[b] + self.k[b]:offs[b + 1]] = np.arange(self.n_visual[b], self.ctx[b])
        self.keep_idx = torch.from_numpy(keep).to(self.device)
        self.keep_offsets_host = offs
        self.keep_offsets = torch.from_numpy(offs).to(self.device)
        self.kept_offsets_host = [int(o) for o in offs[:-1]]                 # where select writes each sequence

        # ---- draft caches: full (gather source) and pruned (gather destination, draft attention input)
        shuffle = np.random.default_rng([cfg.seed, 77]) if cfg.paged_shuffle else None
        h, dh = cfg.dft_kv_heads, cfg.dft_head_dim
        st, sp = W.make_page_table(self.ctx, shuffle)
        dcap = [n + g for n in self.n_keep]
        dtab, dpool = W.make_page_table(dcap, shuffle)
        self.src_k = _randn((self.Ld, sp, h, 64, dh), tdt, gen, self.device)
        self.src_v = _randn((self.Ld, sp, h, 64, dh), tdt, gen, self.device)
        self.dst_k = _randn((self.Ld, dpool, h, 64, dh), tdt, gen, self.device)   # slots past n_keep: the drafted tokens' K/V
        self.dst_v = _randn((self.Ld, dpool, h, 64, dh), tdt, gen, self.device)
        ident = (not cfg.paged_shuffle) and B == 1
        self.src_table = None if ident else torch.from_numpy(st).to(self.device)
        self.dst_table = None if ident else torch.from_numpy(dtab).to(self.device)
        self.src_cache = [hb.KVCache(self.src_k[l], self.src_v[l], self.src_table, st.shape[1]) for l in range(self.Ld)]
        self.dst_cache = [hb.KVCache(self.dst_k[l], self.dst_v[l], self.dst_table, dtab.shape[1]) for l in range(self.Ld)]
        self.src_layer_stride = self.src_k[0].numel() * self.src_k.element_size()
        self.dst_layer_stride = self.dst_k[0].numel() * self.dst_k.element_size()

        # ---- draft attention: q per (layer, draft step); kv_len per draft step
        self.q_d = _randn((self.Ld, g, B, 1, cfg.dft_q_heads, dh), tdt, gen, self.device)
        self.out_d = torch.empty_like(self.q_d)
        self.kv_len_d = [torch.tensor([n + j + 1 for n in self.n_keep], dtype=torch.int32, device=self.device) for j in range(g)]
        self.max_kv_d = [max(self.n_keep) + j + 1 for j in range(g)]
        self.draft_ws = hb.new_workspace(hb.hippo_attention_workspace_bytes(B, 1, cfg.dft_q_heads, h, dh), self.device)

        # ---- target cache and verification queries
        H, D = cfg.tgt_kv_heads, cfg.tgt_head_dim
        self.kv_len_t_host = [c + g + 1 for c in self.ctx]
        tt, tp = W.make_page_table(self.kv_len_t_host, shuffle)
        self.tgt_k = _randn((self.Lt, tp, H, 64, D), tdt, gen, self.device)
        self.tgt_v = _randn((self.Lt, tp, H, 64, D), tdt, gen, self.device)
        self.tgt_table = None if ident else torch.from_numpy(tt).to(self.device)
        self.tgt_cache = [hb.KVCache(self.tgt_k[l], self.tgt_v[l], self.tgt_table, tt.shape[1]) for l in range(self.Lt)]
        self.q_t = _randn((self.Lt, B, g + 1, cfg.tgt_q_heads, D), tdt, gen, self.device)
        self.out_t = torch.empty_like(self.q_t)
        self.kv_len_t = torch.tensor(self.kv_len_t_host, dtype=torch.int32, device=self.device)
        self.verify_ws = hb.new_workspace(hb.hippo_attention_workspace_bytes(B, g + 1, cfg.tgt_q_heads, H, D), self.device)
        self.verify_layers_ws = hb.new_workspace(
            hb.hippo_verify_attention_layers_workspace_bytes(self.Lt, B, g + 1, cfg.tgt_q_heads, H, D), self.device)
        self.q_t_layers = [self.q_t[l] for l in range(self.Lt)]
        self.out_t_layers = [self.out_t[l] for l in range(self.Lt)]

        # ---- acceptance inputs (host-generated: the draft tokens are sampled from the draft logits)
        acc = W.accept_inputs(cfg) if host_inputs is None else host_inputs
        self.accept_host = acc
        self.acc = {k: torch.from_numpy(np.ascontiguousarray(v)).to(self.device) for k, v in acc.items()}
        self.n_accepted = torch.empty(B, dtype=torch.int32, device=self.device)
        self.out_tokens = torch.empty((B, g + 1), dtype=torch.int32, device=self.device)
        self.accept_ws = hb.new_workspace(hb.hippo_accept_workspace_bytes(B, g, cfg.vocab), self.device)

        self.stream_d = torch.cuda.Stream(device=self.device)
        self.stream_v = torch.cuda.Stream(device=self.device)
        if verify_max_ctas == 0 and multi_layer_verify:
            # Default sharing, from the two legs' sizes: when the draft leg (latency-bound calls, about 10 us each) outlasts the
            # verification leg (bandwidth-bound), verification gives up 84 of the 148 SMs to it; measured on B200 this takes
            # the 6k-token step from 1.55 ms to 1.12 ms and the 32k-token step from 3.52 ms to 3.03 ms.  When verification is
            # the longer leg (64k tokens, 80 layers) it keeps every SM: the draft calls then run in its shadow or after it,
            # and holding SMs back only slows the step down (7.05 ms against 7.37 ms with 116 CTAs).
            verify_s = self.verify_kv_bytes_per_layer() * self.Lt / 5.4e12
            draft_s = g * self.Ld * 10e-6
            if draft_s > verify_s:
                self.verify_max_ctas = 64
        self.draft_num_splits = 16 if max(self.n_keep) + g > 1024 and B * h <= 4 else 0

    # ---- algorithmic bytes (the roofline numerators) ------------------------------------------------------------
    @property
    def elem(self) -> int:
        return 4 if self.cfg.dtype == "fp32" else 2

    def verify_kv_bytes_per_layer(self) -> int:
        c = self.cfg
        return sum(self.kv_len_t_host) * 2 * c.tgt_kv_heads * c.tgt_head_dim * self.elem

    def draft_kv_bytes_per_call(self, j: int = 0) -> int:
        c = self.cfg
        return sum(n + j + 1 for n in self.n_keep) * 2 * c.dft_kv_heads * c.dft_head_dim * self.elem

    def gather_bytes(self) -> int:
        c = self.cfg
        return 2 * self.Ld * sum(self.n_keep) * 2 * c.dft_kv_heads * c.dft_head_dim * self.elem  # read + write

    def select_bytes(self) -> int:
        return sum(self.n_visual) * self.cfg.embed_dim * self.elem

    def select_flops(self) -> int:
        """fp64 flops of the selection scores as defined (2 per multiply-add): per crop of M tokens M(M-1)/2 distinct
        cosine dot products, per token one norm and one dot product with the same cell of the next frame."""
        c = self.cfg
        tpf = c.grid_h * c.grid_w
        dots = 0
        for n in self.n_visual:
            full, rest = divmod(n, tpf)
            for nf, count in ((tpf, full), (rest, 1 if rest else 0)):
                for y0 in range(0, c.grid_h, c.crop_h):
                    for x0 in range(0, c.grid_w, c.crop_w):
                        m = sum(1 for y in range(y0, min(y0 + c.crop_h, c.grid_h)) for x in range(x0, min(x0 + c.crop_w, c.grid_w))
                                if y * c.grid_w + x < nf)
                        dots += count * m * (m - 1) // 2
            dots += n + max(0, n - tpf)       # norms, and one temporal dot product per token that has a next frame
        return 2 * dots * c.embed_dim

    def accept_bytes(self) -> int:
        c = self.cfg
        return c.batch * (2 * c.gamma + 1) * c.vocab * 4

    # ---- launch sequences -----------------------------------------------------------------------------------------
    def select(self, stream=None):
        c = self.cfg
        hb.hippo_select_tokens(self.embeds, self.attn_mass, self.n_visual, self.k, c.grid_h, c.grid_w, c.crop_h, c.crop_w,
                               kept_idx=self.keep_idx, kept_offsets=self.kept_offsets_host, fused_score=self.fused,
                               workspace=self.select_ws, stream=stream)

    def select_with(self, **kw):
        """hippo_select_tokens on this step's inputs with other options (score mask, policy); returns (kept, fused)."""
        c = self.cfg
        return hb.hippo_select_tokens(self.embeds, self.attn_mass, self.n_visual, self.k, c.grid_h, c.grid_w, c.crop_h,
                                      c.crop_w, **kw)

    def policy_variants(self):
        """Named option sets of the selection whose kept sets the benchmark compares."""
        gen = torch.Generator(device=self.device)
        gen.manual_seed(4000 + self.cfg.seed)
        keys = torch.rand(sum(self.n_visual), generator=gen, device=self.device, dtype=torch.float32)
        return {"attention_only": {"score_mask": 1}, "all_terms": {"score_mask": 7},
                "uniform_per_frame_attention_only": {"score_mask": 1, "policy": hb.HIPPO_SELECT_UNIFORM_PER_FRAME},
                "uniform_per_frame_all_terms": {"score_mask": 7, "policy": hb.HIPPO_SELECT_UNIFORM_PER_FRAME},
                "random": {"policy": hb.HIPPO_SELECT_RANDOM, "random_keys": keys},
                "whole_frames": {"policy": hb.HIPPO_SELECT_FRAMES}}

    def gather(self, stream=None):
        hb.hippo_gather_kv(self.Ld, self.src_cache[0], self.src_layer_stride, self.dst_cache[0], self.dst_layer_stride,
                           self.cfg.batch, self.keep_idx, self.keep_offsets, int(self.keep_offsets_host[-1]), stream=stream)

    def draft(self, stream=None):
        for j in range(self.cfg.gamma):
            for l in range(self.Ld):
                hb.hippo_draft_attention(self.q_d[l, j], self.dst_cache[l], self.kv_len_d[j], self.max_kv_d[j],
                                         out=self.out_d[l, j], workspace=self.draft_ws, stream=stream,
                                         num_splits=self.draft_num_splits)

    def verify(self, stream=None):
        """The verification leg, one call per target layer."""
        m = max(self.kv_len_t_host)
        for l in range(self.Lt):
            hb.hippo_verify_attention(self.q_t[l], self.tgt_cache[l], self.kv_len_t, m, out=self.out_t[l],
                                      workspace=self.verify_ws, stream=stream, kv_len_host=self.kv_len_t_host)

    def verify_layers(self, stream=None, max_ctas: int = 0):
        """The verification leg, all target layers in one call."""
        hb.hippo_verify_attention_layers(self.q_t_layers, self.tgt_cache, self.kv_len_t, max(self.kv_len_t_host),
                                         self.out_t_layers, workspace=self.verify_layers_ws, stream=stream,
                                         kv_len_host=self.kv_len_t_host, max_ctas=max_ctas)

    def verify_leg(self, stream=None):
        if self.multi_layer_verify:
            self.verify_layers(stream, self.verify_max_ctas)
        else:
            self.verify(stream)

    def attention_mass(self, stream=None):
        """Eq. 2 over all target layers of the prefilled cache (once per prompt, upstream of select); the result goes
        to `self.mass_out`, the step's own selection keeps reading the configuration's synthetic mass."""
        c = self.cfg
        if getattr(self, "q_txt", None) is None:
            gen = torch.Generator(device=self.device)
            gen.manual_seed(2000 + c.seed)
            self.q_txt = _randn((self.Lt, c.batch, c.n_text, c.tgt_q_heads, c.tgt_head_dim), self.tdt, gen, self.device)
            self.mass_out = torch.zeros(sum(self.n_visual), dtype=torch.float32, device=self.device)
            code = hb.HIPPO_DTYPE_FP32 if c.dtype == "fp32" else hb.HIPPO_DTYPE_BF16
            self.mass_ws = hb.new_workspace(hb.hippo_attention_mass_workspace_bytes(
                self.n_visual, c.n_text, c.tgt_q_heads, c.tgt_kv_heads, c.tgt_head_dim, code), self.device)
        w = 1.0 / (self.Lt * c.tgt_q_heads * c.n_text)
        s = torch.cuda.current_stream(self.device) if stream is None else stream
        with torch.cuda.stream(s):
            self.mass_out.zero_()
        for l in range(self.Lt):
            hb.hippo_attention_mass(self.q_txt[l], self.tgt_cache[l], self.n_visual, w, self.mass_out,
                                    workspace=self.mass_ws, stream=stream)

    def mass_exps_per_layer(self) -> int:
        """Exponentials Eq. 2 needs per layer as computed here: one per (text row, head, visual key) in each pass."""
        c = self.cfg
        return 2 * c.n_text * c.tgt_q_heads * sum(self.n_visual)

    def accept(self, stream=None):
        a = self.acc
        hb.hippo_accept(a["target_logits"], a["draft_logits"], a["draft_tokens"], a["u_accept"], a["u_resample"],
                        n_accepted=self.n_accepted, out_tokens=self.out_tokens, workspace=self.accept_ws, stream=stream)

    def run(self):
        """The whole step on the current stream, with draft and verify forked onto their own streams.

        The verification leg reads neither the selection nor the pruned cache.  With `verify_beside_select` it is forked
        first and runs beside select and gather too; otherwise it starts once the selection has finished (the selection's
        fp64 kernels want every SM for themselves) and runs beside the draft calls only."""
        main = torch.cuda.current_stream(self.device)
        if self.verify_beside_select:
            self.stream_v.wait_stream(main)
            self.verify_leg(self.stream_v)
        self.select(main)
        if not self.verify_beside_select:
            self.stream_v.wait_stream(main)
            self.verify_leg(self.stream_v)
        self.gather(main)
        self.stream_d.wait_stream(main)
        self.draft(self.stream_d)             # reads the gathered cache
        main.wait_stream(self.stream_d)
        main.wait_stream(self.stream_v)
        self.accept(main)
