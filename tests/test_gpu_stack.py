"""The fifth workload at a small size: a stack of MoE layers decoded with beam search over a HOT + STAGE expert
cache with predictor-driven and on-demand staging. Beam trajectories are chaotic, so parity is teacher-forced:
the run records the input and output of sampled (step, layer) calls, and the oracle recomputes those layers
from the recorded inputs with its own compressed experts."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from paper_2609_38090_b200 import inputs
from gpu_util import gate_b, gate_c

pytestmark = pytest.mark.gpu
TOL = 2e-3


def _small():
    from paper_2609_38090_b200.stack import StackConfig
    sh = inputs.LayerShape("small_stack", C=256, R=192, E=12, k=4, T=4, n_shared=2, zipf_a=1.1, seed=1)
    return StackConfig(shape=sh, n_layers=5, vocab=96, n_hot=3, n_stage=3, k_pred=7, seed=1)


def test_stack_layers_match_the_oracle_teacher_forced_and_the_cache_is_exercised():
    from paper_2609_38090_b200.stack import MoEStack
    cfg = _small()
    rec = []
    st = MoEStack(cfg, build="numpy", record=lambda s, l, x, o: rec.append((s, l, x.clone(), o.clone())))
    tokens, scores = st.decode(4)
    torch.cuda.synchronize()
    assert st.m.poll_status()[0] == 0
    assert tokens.shape == (4, cfg.shape.T) and torch.isfinite(scores).all()
    assert len(rec) == 4 * cfg.n_layers
    stats = st.stats()
    assert stats.pairs_hot > 0 and stats.pairs_demand > 0            # both kinds of service happened
    assert stats.prefetch_issued > 0 and stats.copies >= stats.prefetch_issued
    assert st.bytes_staged == stats.copies * st.m.expert_bytes
    cov = st.coverage()                                              # Coverage@k per source layer, k = 1..k_pred
    assert len(cov) == cfg.n_layers - 2 and all(n == 4 for n in st.coverage_counts()[:cfg.n_layers - 2])
    for row in cov:
        assert all(0.0 <= a <= b <= 1.0 for a, b in zip(row, row[1:])) and row[-1] > 0.0
    sh = cfg.shape
    blob_cache = {}
    for s, l, x, out in rec[::3]:                                     # every third call
        lsh = dataclasses.replace(sh, layer=l, seed=cfg.seed)
        if l not in blob_cache:
            wr, bias = inputs.router(lsh)
            blobs = [oracle.quantize_expert(*inputs.expert_weights(lsh, e)) for e in range(sh.E + sh.n_shared)]
            blob_cache[l] = (wr, bias, blobs)
        wr, bias, blobs = blob_cache[l]
        xin = x.float().cpu().numpy()
        res = oracle.moe_layer(xin, wr, bias, blobs, sh.R, sh.k, n_shared=sh.n_shared)
        got = out.float().cpu().numpy()
        b_, c_ = gate_b(got, res["out64"]), gate_c(got, res["out64"], bf16_output=True)
        assert b_ <= TOL and c_ <= TOL, f"step {s} layer {l}: gate B {b_}, gate C {c_}"


def test_stack_with_every_expert_resident_gives_the_same_tokens():
    """The cache changes where experts live, never what the layers compute."""
    from paper_2609_38090_b200.stack import MoEStack
    cfg = _small()
    a = MoEStack(cfg, build="numpy")
    ta, sa = a.decode(3)
    big = dataclasses.replace(cfg, n_hot=cfg.shape.E, n_stage=1)
    b = MoEStack(big, build="numpy")
    tb, sb = b.decode(3)
    assert b.stats().pairs_demand == 0 and b.stats().copies == 0
    assert torch.equal(ta, tb) and torch.equal(sa, sb)


def test_rebalancing_from_a_random_hot_set_keeps_the_tokens_and_raises_the_hot_share():
    """Swapping experts into HOT slots changes residency only: same tokens as the all-resident run, fewer misses
    than without rebalancing."""
    from paper_2609_38090_b200.stack import MoEStack
    cfg = _small()
    ref = MoEStack(dataclasses.replace(cfg, n_hot=cfg.shape.E, n_stage=1), build="numpy")
    t_ref, s_ref = ref.decode(12)
    plain = MoEStack(dataclasses.replace(cfg, hot_init="random", k_pred=0), build="numpy")
    t0, s0 = plain.decode(12)
    reb = MoEStack(dataclasses.replace(cfg, hot_init="random", k_pred=0, rebalance_every=8, max_swaps=2), build="numpy")
    t1, s1 = reb.decode(12)
    torch.cuda.synchronize()
    assert reb.m.poll_status()[0] == 0
    assert torch.equal(t_ref, t0) and torch.equal(t_ref, t1) and torch.equal(s_ref, s1)
    assert reb.hot_swaps() > 0
    assert reb.stats().pairs_demand < plain.stats().pairs_demand


def test_library_runtime_and_python_issued_steps_drive_the_stack_identically():
    """The harness run three ways -- mira_stack_layer_step (the library's runtime), Python-issued calls with the
    library's cache manager, Python-issued calls with cache.LayerCache: same tokens, same statistics, same bytes
    staged, same swaps and coverage, with prefetching, demand waves and rebalancing all active."""
    from paper_2609_38090_b200.stack import MoEStack
    cfg = dataclasses.replace(_small(), hot_init="random", rebalance_every=8, max_swaps=2)
    runs = []
    for native_step, native_cache in ((True, True), (False, True), (False, False)):
        st = MoEStack(dataclasses.replace(cfg, native_step=native_step, native_cache=native_cache), build="numpy")
        tok, sc = st.decode(10)
        torch.cuda.synchronize()
        assert st.m.poll_status()[0] == 0
        runs.append((tok, sc, dataclasses.asdict(st.stats()), st.bytes_staged, st.hot_swaps(), st.coverage(),
                     [st.slot_map(l) for l in range(cfg.n_layers)]))
        st.reset_stats()
        assert st.stats().copies == 0 and st.bytes_staged == 0 and st.hot_swaps() == 0
    for other in runs[1:]:
        assert torch.equal(runs[0][0], other[0]) and torch.equal(runs[0][1], other[1])
        assert runs[0][2:] == other[2:]
    assert runs[0][4] > 0 and runs[0][2]["prefetch_issued"] > 0 and runs[0][2]["pairs_demand"] > 0


@pytest.mark.parametrize("C", [256, 2048, 16384])
def test_residual_rmsnorm_glue_matches_the_torch_formula(C):
    """The harness's glue kernel against rms_norm(x + out) in fp32 with torch ops: equal up to one bf16 rounding step
    (the reduction order differs)."""
    from paper_2609_38090_b200 import binding as b
    g = torch.Generator(device="cuda").manual_seed(C)
    x = torch.randn((5, C), generator=g, device="cuda").to(torch.bfloat16)
    y = (3.0 * torch.randn((5, C), generator=g, device="cuda")).to(torch.bfloat16)
    got = b.residual_rmsnorm(x, y, eps=1e-6).float()
    v = x.float() + y.float()
    ref = torch.nn.functional.rms_norm(v, (C,), eps=1e-6)
    assert torch.isfinite(got).all()
    assert ((got - ref).abs() <= ref.abs() * 2.0 ** -7 + 1e-30).all()          # within one bf16 ulp of the fp32 result
    assert ((got - ref.to(torch.bfloat16).float()) != 0).float().mean() < 0.01  # and almost always the same rounding


def test_full_size_stack_of_24_fine_grained_layers_teacher_forced():
    """The fifth workload at its full size: 24 layers of the fine-grained layer (hidden 2048, ffn 1408, 60 experts
    top-4 plus 4 shared), beam width 4, per layer a cache of 12 HOT + 3 STAGE slots (25 % of the routed experts),
    predictor-driven and on-demand staging from 13 GB of pinned host memory through the library's layer-step
    runtime. A few decode steps; sampled (step, layer) calls are recomputed by the oracle from the recorded
    inputs, with the experts those tokens need compressed by the oracle from the same seeded weights."""
    from paper_2609_38090_b200.stack import MoEStack, StackConfig
    sh = inputs.FINE_STACK
    cfg = StackConfig(shape=sh, n_layers=24, vocab=1024, n_hot=12, n_stage=3, k_pred=4, seed=1)
    rec = []
    st = MoEStack(cfg, build="numpy", record=lambda s, l, x, o: rec.append((s, l, x.clone(), o.clone())))
    tokens, scores = st.decode(3)
    torch.cuda.synchronize()
    assert st.m.poll_status()[0] == 0
    assert tokens.shape == (3, sh.T) and torch.isfinite(scores).all() and len(rec) == 3 * cfg.n_layers
    stats = st.stats()
    assert stats.pairs_hot > 0 and stats.pairs_demand > 0 and stats.copies > 0      # the cache was exercised
    picks = [(0, 0), (0, 11), (0, 23), (1, 5), (1, 22), (2, 1), (2, 17), (2, 23)]
    for s, l, x, out in (r for r in rec if (r[0], r[1]) in picks):
        lsh = dataclasses.replace(sh, layer=l, seed=cfg.seed)
        wr, bias = inputs.router(lsh)
        xin = x.float().cpu().numpy()
        logits = oracle.linear_scores(xin, wr, bias)
        idx, _, _, margin = oracle.topk_softmax(logits, sh.k)
        if not (margin > 1e-5 * np.maximum(1.0, np.abs(logits).max(1))).all():
            continue                                                        # a near-tie: either neighbour is a valid routing
        need = set(idx.ravel().tolist()) | set(range(sh.E, sh.E + sh.n_shared))
        blobs = [oracle.quantize_expert(*inputs.expert_weights(lsh, e)) if e in need else None
                 for e in range(sh.E + sh.n_shared)]
        res = oracle.moe_layer(xin, wr, bias, blobs, sh.R, sh.k, n_shared=sh.n_shared)
        got = out.float().cpu().numpy()
        b_, c_ = gate_b(got, res["out64"]), gate_c(got, res["out64"], bf16_output=True)
        assert b_ <= TOL and c_ <= TOL, f"step {s} layer {l}: gate B {b_}, gate C {c_}"
