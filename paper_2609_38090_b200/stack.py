"""A stack of MoE layers decoded with beam search over a small expert cache: the fifth workload.

Every MoE layer step goes through the C ABI (mira_predict, mira_route, mira_stage_expert, mira_moe_experts).
What surrounds the layers is harness glue in plain torch ops, not part of the measured method and stated as
such: a tied embedding / output head, `x <- rmsnorm(x + MoE(x))` without learned scale between layers (keeps the
activations O(1) with random weights), and a standard beam step (log-softmax, top-W over W * V candidates).

Cache: per layer the shared experts and a fixed HOT set stay on the device; a few STAGE slots receive experts
from pinned host memory, either ahead of time (the predictor head of layer l scores the experts of layer l + 2,
Section IV-D) or on demand when the router selects an expert that is not resident. The predictor heads are the
routers of the layers they predict (a stand-in for trained heads: with random weights nothing can be learned).
"""
from __future__ import annotations

import dataclasses

import numpy as np
import torch

from . import binding, inputs
from .cache import CacheStats, LayerCache, coverage_at_k


@dataclasses.dataclass
class StackConfig:
    shape: inputs.LayerShape            # one layer; shape.T is the beam width
    n_layers: int = 24
    vocab: int = 1024
    n_hot: int = 12
    n_stage: int = 3
    k_pred: int = 16                    # ids requested from the predictor; resident ones are skipped
    seed: int = 1
    hot_init: str = "bias"              # "bias": the experts the router bias favours; "random": a seeded random set
    rebalance_every: int = 0            # tokens per layer between rebalancing passes of its HOT set (0: never)
    max_swaps: int = 2                  # HOT swaps per pass and layer
    native_cache: bool = True           # bookkeeping by the library's mira_cache_* object (else cache.LayerCache)
    native_step: bool = True            # the whole layer step inside the library (mira_stack_layer_step); else the
                                        # same steps issued from Python, call by call


class MoEStack:
    def __init__(self, cfg: StackConfig, device="cuda:0", build="device", record=None):
        """build = "device": weights drawn with torch's CUDA generator (fast, for the benchmark);
        build = "numpy": weights from the seeded numpy recipe of `inputs` (slow, for parity tests, keeps the
        fp32 weights' blobs reproducible by the oracle)."""
        sh = cfg.shape
        self.cfg, self.sh, self.dev = cfg, sh, torch.device(device)
        self.L, self.W = cfg.n_layers, sh.T
        self.n_total = sh.E + sh.n_shared
        self.m = binding.Mira(sh.C, sh.R, sh.E, n_shared=sh.n_shared, n_layers=self.L, max_tokens=self.W,
                              max_top_k=sh.k, device=self.dev)
        eb = self.m.expert_bytes
        self.host_blobs = torch.empty((self.L, self.n_total, eb), dtype=torch.uint8).pin_memory()
        self.layers = [dataclasses.replace(sh, layer=l, seed=cfg.seed) for l in range(self.L)]
        self.routers, self.biases = [], []
        g = torch.Generator(device=self.dev)
        g.manual_seed(7000 + cfg.seed)
        for l, lsh in enumerate(self.layers):
            wr, bias = inputs.router(lsh)
            self.routers.append(torch.from_numpy(wr).to(torch.bfloat16).to(self.dev))
            self.biases.append(torch.from_numpy(bias).to(self.dev))
            for e0 in range(0, self.n_total, 16):
                n = min(16, self.n_total - e0)
                if build == "device":
                    w1 = torch.randn((n, sh.R, sh.C), generator=g, device=self.dev) * 0.02
                    w2 = torch.randn((n, sh.C, sh.R), generator=g, device=self.dev) * 0.02
                    w3 = torch.randn((n, sh.R, sh.C), generator=g, device=self.dev) * 0.02
                else:
                    ws = [inputs.expert_weights(lsh, e) for e in range(e0, e0 + n)]
                    w1, w2, w3 = (torch.from_numpy(np.stack([w[i] for w in ws])).to(self.dev) for i in range(3))
                blobs = self.m.quantize_experts(w1, w2, w3)
                self.host_blobs[l, e0:e0 + n].copy_(blobs)
        torch.cuda.synchronize(self.dev)
        # HOT set: the experts the Zipf bias makes most popular
        self.caches = []                           # Python-driven mode: one bookkeeping object per layer
        self.hot_sets = []
        self.native = None                         # native mode: the library's stack runtime
        self.slot_mem = torch.empty((self.L, sh.n_shared + cfg.n_hot + cfg.n_stage, eb), dtype=torch.uint8, device=self.dev)
        for l in range(self.L):
            if cfg.hot_init == "random":
                hot = sorted(np.random.Generator(np.random.PCG64([cfg.seed, 91, l])).permutation(sh.E)[:cfg.n_hot].tolist())
            else:
                hot = sorted(np.argsort(-self.biases[l].cpu().numpy(), kind="stable")[:cfg.n_hot].tolist())
            self.hot_sets.append(hot)
            if cfg.native_step:
                continue
            c = (binding.NativeLayerCache if cfg.native_cache else LayerCache)(sh.E, sh.n_shared, hot, cfg.n_stage)
            for e, s in enumerate(c.slot_map()):
                if s >= 0:
                    self.slot_mem[l, s].copy_(self.host_blobs[l, e], non_blocking=True)
            self.caches.append(c)
        self.slots = [binding.slot_table(self.slot_mem[l]) for l in range(self.L)]
        emb = inputs.round_to_bf16(np.random.Generator(np.random.PCG64([cfg.seed, 77])).standard_normal(
            (cfg.vocab, sh.C), dtype=np.float32))
        self.emb = torch.from_numpy(emb).to(torch.bfloat16).to(self.dev)
        self.side = torch.cuda.Stream(device=self.dev)
        self.main = torch.cuda.current_stream(self.dev)
        ns = self.slot_mem.shape[1]
        self.ready = [[torch.cuda.Event() for _ in range(ns)] for _ in range(self.L)]   # slot filled
        self.freed = [[torch.cuda.Event() for _ in range(ns)] for _ in range(self.L)]   # slot's last reader done
        for l in range(self.L):
            for ev in self.freed[l] + self.ready[l]:
                ev.record(self.main)
        self.map_cache = {}                        # slot map (tuple) -> device tensor
        self.back_dev = torch.empty(self.n_total + cfg.k_pred, dtype=torch.int32, device=self.dev)
        self.back_host = torch.empty(self.n_total + cfg.k_pred, dtype=torch.int32).pin_memory()
        self.record = record                       # None or callable(step, layer, x, out) for teacher-forced parity
        self.pending_hot = [set() for _ in range(self.L)]      # HOT slots being refilled by a rebalancing swap
        self._bytes_staged = 0
        if cfg.native_step:
            self.native = binding.NativeStack(self.m, self.host_blobs, self.slot_mem, self.hot_sets, cfg.n_hot, cfg.n_stage,
                                              cfg.k_pred, self.side, rebalance_every=cfg.rebalance_every,
                                              max_swaps=cfg.max_swaps, stream=self.main)
        # Coverage@k of the predictor heads: the ids predicted for layer l + 2 wait here until that layer has routed
        self.pred_for = [None] * self.L
        self.coverage_sum = [[0.0] * cfg.k_pred for _ in range(self.L)]      # [source layer][k - 1]
        self.coverage_n = [0] * self.L
        torch.cuda.synchronize(self.dev)

    # ------------------------------------------------------------------ helpers
    def _slot_map_dev(self, values):
        """Device copy of a slot map. Maps seen before (the common case: nothing staged since) are kept."""
        key = tuple(values)
        hit = self.map_cache.get(key)
        if hit is not None:
            return hit
        if len(self.map_cache) >= 4096:
            self.map_cache.clear()
        t = torch.tensor(values, dtype=torch.int32).pin_memory().to(self.dev, non_blocking=True)
        self.map_cache[key] = t
        return t

    def _copy(self, l, e, slot):
        self.side.wait_event(self.freed[l][slot])
        self.m.stage_expert(self.host_blobs[l, e], self.slot_mem[l, slot], self.side, self.ready[l][slot])
        self._bytes_staged += self.m.expert_bytes

    def stats(self) -> CacheStats:
        if self.native is not None:
            return self.native.stats()[0]
        s = CacheStats()
        for c in self.caches:
            s.merge(c.stats)
        return s

    @property
    def bytes_staged(self) -> int:
        return self.native.stats()[1] if self.native is not None else self._bytes_staged

    def hot_swaps(self) -> int:
        return self.native.stats()[2] if self.native is not None else sum(c.swaps_done for c in self.caches)

    def slot_map(self, l: int) -> list[int]:
        return self.native.slot_map(l) if self.native is not None else self.caches[l].slot_map()

    def reset_stats(self) -> None:
        """Zeroes the cache statistics, the staged-byte count and the coverage sums (not the rebalancing windows)."""
        if self.native is not None:
            self.native.reset_stats()
            return
        for c in self.caches:
            c.reset_stats()
            c.swaps_done = 0
        self._bytes_staged = 0
        self.coverage_sum = [[0.0] * self.cfg.k_pred for _ in range(self.L)]
        self.coverage_n = [0] * self.L

    def coverage(self) -> list[list[float]]:
        """Mean Coverage@k (k = 1..k_pred) per source layer over the layer steps run so far."""
        sums, n = self.native.coverage() if self.native is not None else (self.coverage_sum, self.coverage_n)
        return [[v / max(c, 1) for v in row] for row, c in zip(sums[:max(self.L - 2, 0)], n)]

    def coverage_counts(self) -> list[int]:
        return self.native.coverage()[1] if self.native is not None else list(self.coverage_n)

    # ------------------------------------------------------------------ one layer
    def layer_step(self, l, x, step=0):
        sh, cfg, m = self.sh, self.cfg, self.m
        target = l + 2
        if self.native is not None:
            head = target < self.L and cfg.k_pred > 0
            out = self.native.layer_step(l, x, self.routers[l], self.biases[l], sh.k,
                                         self.routers[target] if head else None, self.biases[target] if head else None,
                                         stream=self.main)
            if self.record is not None:
                self.record(step, l, x, out)
            return out
        if target < self.L and cfg.k_pred > 0:          # S7: the head of layer l scores the experts of layer l + 2 (router of l + 2 as head)
            _, _, ids = m.predict(l, x, self.routers[target], self.biases[target], k_pred=cfg.k_pred, reuse=True, stream=self.main)
            self.back_dev[self.n_total:].copy_(ids)
        r = m.route(x, self.routers[l], self.biases[l], sh.k, reuse=True, stream=self.main)
        self.back_dev[:self.n_total].copy_(r["count"])
        self.back_host.copy_(self.back_dev, non_blocking=True)
        self.main.synchronize()                                      # the cache manager reads counts and predicted ids
        back = self.back_host.tolist()
        counts, pred = back[:self.n_total], back[self.n_total:]
        if self.pred_for[l] is not None:                             # made two layers back: score it on this routing
            src = l - 2
            for k in range(1, cfg.k_pred + 1):
                self.coverage_sum[src][k - 1] += coverage_at_k(self.pred_for[l], counts[:sh.E], k)
            self.coverage_n[src] += 1
            self.pred_for[l] = None
        if target < self.L and cfg.k_pred > 0:
            self.pred_for[target] = pred
            for e, slot in self.caches[target].prefetch(pred):
                self._copy(target, e, slot)
        cache = self.caches[l]
        waves = cache.plan(counts)
        out = torch.empty((self.W, sh.C), dtype=torch.bfloat16, device=self.dev)
        first_slot = sh.n_shared + cache.n_hot
        for s_ in self.pending_hot[l]:                                # swapped-in HOT experts must have landed
            self.main.wait_event(self.ready[l][s_])
        self.pending_hot[l].clear()
        for wi, wave in enumerate(waves):
            for e, slot in wave.copies:
                self._copy(l, e, slot)
            used = [wave.slot_map[e] for e in wave.experts]
            for s in used:
                if s >= first_slot:
                    self.main.wait_event(self.ready[l][s])
            m.moe_experts(x, self.slots[l], self._slot_map_dev(wave.slot_map), expert_ids=wave.experts,
                          final_wave=wi == len(waves) - 1, out=out, stream=self.main)
            for s in used:
                if s >= first_slot:
                    self.freed[l][s].record(self.main)
        cache.layer_done(n_tokens=self.W)
        if cfg.rebalance_every and cache.win_tokens >= cfg.rebalance_every:
            swaps = cache.rebalance(max_swaps=cfg.max_swaps)
            if swaps:
                done = torch.cuda.Event()
                done.record(self.main)                                    # the waves above still read the old experts
                self.side.wait_event(done)
                for _, e, slot in swaps:
                    self.m.stage_expert(self.host_blobs[l, e], self.slot_mem[l, slot], self.side, self.ready[l][slot])
                    self._bytes_staged += self.m.expert_bytes
                    self.pending_hot[l].add(slot)
        if self.record is not None:
            self.record(step, l, x, out)
        return out

    # ------------------------------------------------------------------ glue: norm, head, beam step
    def _residual_norm(self, x, out):
        """x <- rmsnorm(x + MoE(x)) without learned scale, in fp32, rounded to bf16 (glue: one small kernel of the
        library, the same arithmetic as `rms_norm(x.float() + out.float()).to(bf16)`)."""
        return binding.residual_rmsnorm(x, out, eps=1e-6, stream=self.main)

    def decode(self, n_steps: int, first_tokens=None, first_scores=None):
        """Beam search of width W for n_steps steps. Returns (tokens [n_steps, W], beam scores [W]). A search is
        continued by passing the last row of tokens and the scores of the previous call."""
        W, V = self.W, self.cfg.vocab
        tokens = torch.arange(W, device=self.dev) if first_tokens is None else first_tokens.to(self.dev)
        scores = torch.zeros(W, dtype=torch.float32, device=self.dev) if first_scores is None else first_scores.to(self.dev)
        history = []
        for step in range(n_steps):
            x = self.emb[tokens].contiguous()
            for l in range(self.L):
                out = self.layer_step(l, x, step)
                x = self._residual_norm(x, out)
            logp = torch.log_softmax(x.float() @ self.emb.float().t(), dim=-1)           # [W, V]
            cand = (scores[:, None] + logp).reshape(-1)
            scores, flat = torch.topk(cand, W)
            tokens = flat % V                                                             # beam reordering is implicit:
            history.append(tokens)                                                        # no state but the token
        return torch.stack(history), scores


__all__ = ["StackConfig", "MoEStack"]
