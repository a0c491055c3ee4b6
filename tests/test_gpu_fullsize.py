"""Full-size GPU parity in the launch configurations bench.py times: the Mixtral-8x7B-shaped layer
(decode 1 / 8 / 32 tokens and a 2048-token prefill) and the fine-grained layer (60 experts top-4 plus
4 shared; decode 64, prefill 1024). Compressed experts are compared bit for bit over all bytes; layer
outputs on every token where the oracle finishes in seconds, else on sampled tokens (a token's
output depends on that token alone, so sampled rows are exact checks, not statistics)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_38090_b200 import inputs
from gpu_util import gate_a, gate_b, gate_c, to_bf16_cuda

pytestmark = pytest.mark.gpu
TOL = 2e-3


class FullLayer:
    def __init__(self, sh, max_tokens, fmt=0):
        from paper_2609_38090_b200 import binding as b
        self.sh, self.b, self.fmt = sh, b, fmt
        self.wr, self.bias = inputs.router(sh)
        n = sh.E + sh.n_shared
        self.m = b.Mira(sh.C, sh.R, sh.E, n_shared=sh.n_shared, n_layers=32, max_tokens=max_tokens, max_top_k=sh.k, fmt=fmt)
        self.blobs_gpu = torch.empty((n, self.m.expert_bytes), dtype=torch.uint8, device="cuda")
        self.blobs = []
        for e in range(n):      # one expert at a time: the fp32 weights of all experts would not fit comfortably
            w1, w2, w3 = inputs.expert_weights(sh, e)
            self.blobs.append(oracle.quantize_expert(w1, w2, w3, fmt=self.fmt))
            d = [torch.from_numpy(w[None]).cuda() for w in (w1, w2, w3)]
            self.m.quantize_experts(*d, out=self.blobs_gpu[e:e + 1])
            torch.cuda.synchronize()
            del d, w1, w2, w3
        self.slots = b.slot_table(self.blobs_gpu)
        self.slot_map = torch.arange(n, dtype=torch.int32, device="cuda")
        self.wr_d, self.bias_d = to_bf16_cuda(self.wr), torch.from_numpy(self.bias).cuda()

    def run(self, T, step=0):
        x = inputs.hidden(self.sh, T, step=step)
        out, dbg = self.m.moe_layer(to_bf16_cuda(x), self.wr_d, self.bias_d, self.slots, self.slot_map, self.sh.k,
                                    debug=True)
        torch.cuda.synchronize()
        assert self.m.poll_status()[0] == 0
        return x, out.float().cpu().numpy(), {k: v.cpu().numpy() for k, v in dbg.items()}

    def check(self, T, sample=None, step=0):
        sh = self.sh
        x, out, dbg = self.run(T, step)
        logits = oracle.linear_scores(x, self.wr, self.bias)
        idx, w, _, margin = oracle.topk_softmax(logits, sh.k)
        safe = margin > 1e-5 * np.maximum(1.0, np.abs(logits).max(1))
        assert np.array_equal(dbg["idx"][safe], idx[safe]) and (~safe).sum() <= max(1, T // 500)
        if safe.all():
            count, offset, perm, perm_sh = oracle.group(idx, sh.E, sh.n_shared)
            assert np.array_equal(dbg["count"], count) and np.array_equal(dbg["offset"], offset)
            assert np.array_equal(dbg["perm"], np.concatenate([perm, perm_sh], axis=1))
        rows = np.arange(T) if sample is None else np.random.default_rng(5).choice(T, sample, replace=False)
        rows = np.array([t for t in rows if safe[t]])
        ref = np.stack([oracle.moe_layer(x[t:t + 1], self.wr, self.bias, self.blobs, sh.R, sh.k,
                                         n_shared=sh.n_shared, fmt=self.fmt)["out64"][0] for t in rows])
        b_, c_ = gate_b(out[rows], ref), gate_c(out[rows], ref, bf16_output=True)
        assert b_ <= TOL and c_ <= TOL, f"T={T}: gate B {b_}, gate C {c_}"
        return b_, c_


@pytest.fixture(scope="module")
def mixtral():
    return FullLayer(inputs.MIXTRAL, 2048)


@pytest.fixture(scope="module")
def fine():
    return FullLayer(inputs.FINE, 1024)


def test_mixtral_blobs_bit_exact(mixtral):
    got = mixtral.blobs_gpu.cpu().numpy()
    for e, ref in enumerate(mixtral.blobs):
        assert np.array_equal(got[e], ref), f"expert {e}"


@pytest.mark.parametrize("T", [1, 8, 32])
def test_mixtral_decode(mixtral, T):
    mixtral.check(T)


def test_mixtral_prefill_sampled(mixtral):
    mixtral.check(2048, sample=12)


def test_fine_grained_blobs_decode_and_prefill(fine):
    got = fine.blobs_gpu.cpu().numpy()
    for e, ref in enumerate(fine.blobs):
        assert np.array_equal(got[e], ref), f"expert {e}"
    fine.check(64)
    fine.check(4)                     # the per-step batch of the beam-search stack
    fine.check(1024, sample=24)


def test_mixtral_8x22b_shaped_layer_blobs_decode_and_prefill():
    """The second, larger shape (hidden 6144, ffn 16384: 302 MB per compressed expert): hidden size not a power
    of two, five down slices, blobs past 2^28 bytes. Sampled rows keep the oracle's share to seconds."""
    big = FullLayer(inputs.MIXTRAL22, 2048)
    got = big.blobs_gpu.cpu().numpy()
    for e, ref in enumerate(big.blobs):
        assert np.array_equal(got[e], ref), f"expert {e}"
    del got
    big.check(1)
    big.check(32, sample=5)
    big.check(2048, sample=4)


def test_mixtral_shape_in_the_per_matrix_scale_format():
    """The format variant at full matrix size (two experts of the Mixtral shape, every token routed to both):
    blobs bit for bit, a decode batch on the streaming kernels and a 256-token batch on the tensor-core kernels."""
    import dataclasses
    sh = dataclasses.replace(inputs.MIXTRAL, name="mixtral8x7b_2experts", E=2, k=2)
    lay = FullLayer(sh, 256, fmt=oracle.STANDARD)
    got = lay.blobs_gpu.cpu().numpy()
    for e, ref in enumerate(lay.blobs):
        assert np.array_equal(got[e], ref), f"expert {e}"
    lay.check(8)
    lay.check(256, sample=6)


def test_mixtral_prefill_with_predictor_and_a_cache_of_four_hot_and_two_stage_slots(mixtral):
    """The third workload at its full size: 2048 tokens of the Mixtral-shaped layer, the two-layers-ahead head
    (hidden 4096 -> 8 scores, top-2) scored per token, and an expert cache of 4 HOT + 2 STAGE slots for the 8
    experts: the HOT experts run as the first wave while the others are copied from pinned host memory and run
    as later waves of two. Predictor: per-token scores, pooled scores and ids against the oracle. Layer: sampled
    rows against the oracle, and the whole output bit for bit against the all-resident call."""
    sh, m, b = mixtral.sh, mixtral.m, mixtral.b
    T, n_hot, n_stage = 2048, 4, 2
    x = inputs.hidden(sh, T, step=1)
    xd = to_bf16_cuda(x)
    wp, bp = inputs.predictor(sh)
    pooled, ts, ids = m.predict(0, xd, to_bf16_cuda(wp), torch.from_numpy(bp).cuda(), k_pred=2, token_scores=True)
    ts_ref, pooled_ref, ids_ref, margin = oracle.predict(x, wp, bp, k_pred=2)
    assert np.abs(ts.cpu().numpy() - ts_ref).max() < 1e-4 and np.abs(pooled.cpu().numpy() - pooled_ref).max() < 1e-4
    assert margin > 1e-4 and np.array_equal(ids.cpu().numpy(), ids_ref)

    resident = m.moe_layer(xd, mixtral.wr_d, mixtral.bias_d, mixtral.slots, mixtral.slot_map, sh.k).clone()
    r = m.route(xd, mixtral.wr_d, mixtral.bias_d, sh.k)
    cnt = r["count"].cpu().tolist()
    hot = sorted(np.argsort(-np.array(cnt), kind="stable")[:n_hot].tolist())
    cold = [e for e in range(sh.E) if e not in hot and cnt[e] > 0]
    assert len(cold) == sh.E - n_hot                                  # 2048 tokens reach every expert: two staged waves
    host = mixtral.blobs_gpu.cpu().pin_memory()
    cache = torch.zeros((n_hot + n_stage, m.expert_bytes), dtype=torch.uint8, device="cuda")
    for i, e in enumerate(hot):
        cache[i].copy_(mixtral.blobs_gpu[e])
    cslots = b.slot_table(cache)

    def smap(pairs):
        t = torch.full((sh.E,), -1, dtype=torch.int32)
        for e, sl in pairs:
            t[e] = sl
        return t.cuda()
    side, main = torch.cuda.Stream(), torch.cuda.current_stream()
    ready = [torch.cuda.Event() for _ in range(n_stage)]
    waves = [cold[j:j + n_stage] for j in range(0, len(cold), n_stage)]
    torch.cuda.synchronize()
    for sl, e in enumerate(waves[0]):                                 # staged while the HOT wave computes
        m.stage_expert(host[e], cache[n_hot + sl], side, ready[sl])
    m.moe_experts(xd, cslots, smap([(e, i) for i, e in enumerate(hot)]), expert_ids=hot, final_wave=False)
    out = None
    for wi, wave in enumerate(waves):
        for sl in range(len(wave)):
            main.wait_event(ready[sl])
        out = m.moe_experts(xd, cslots, smap([(e, n_hot + sl) for sl, e in enumerate(wave)]), expert_ids=wave,
                            final_wave=wi == len(waves) - 1)
        if wi + 1 < len(waves):
            done = torch.cuda.Event()
            done.record(main)
            side.wait_event(done)                                     # the STAGE slots are free once this wave has run
            for sl, e in enumerate(waves[wi + 1]):
                m.stage_expert(host[e], cache[n_hot + sl], side, ready[sl])
    torch.cuda.synchronize()
    assert m.poll_status()[0] == 0
    assert torch.equal(out.view(torch.int16), resident.view(torch.int16))
    logits = oracle.linear_scores(x, mixtral.wr, mixtral.bias)
    _, _, _, mrg = oracle.topk_softmax(logits, sh.k)
    safe = mrg > 1e-5 * np.maximum(1.0, np.abs(logits).max(1))
    rows = np.array([t for t in np.random.default_rng(9).choice(T, 10, replace=False) if safe[t]])
    ref = np.stack([oracle.moe_layer(x[t:t + 1], mixtral.wr, mixtral.bias, mixtral.blobs, sh.R, sh.k)["out64"][0] for t in rows])
    got = out.float().cpu().numpy()[rows]
    assert gate_b(got, ref) <= TOL and gate_c(got, ref, bf16_output=True) <= TOL
