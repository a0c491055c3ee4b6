"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle on the same seeded inputs.

Bars: integer / index work bit-exact (codes, scales, top-k ids, counts, offsets, positions,
predictor ids); dequantized fp32 weights identical (0 ULP); layer outputs within 2e-3 (the
spec tolerance) in the three readings written in gpu_util: pre-rounding fp32 (A), bf16
rounding-aware (B), row-wise relative L2 (C)."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from paper_2609_38090_b200 import inputs
from gpu_util import Workload, gate_a, gate_b, gate_c, to_bf16_cuda

pytestmark = pytest.mark.gpu
TOL = 2e-3

SMALL_SHARED = inputs.LayerShape("small_shared", C=128, R=192, E=12, k=4, T=37, n_shared=2, zipf_a=1.1, seed=3)


def _binding():
    from paper_2609_38090_b200 import binding
    return binding


def _mira(sh, T, k=None, **kw):
    b = _binding()
    return b.Mira(sh.C, sh.R, sh.E, n_shared=sh.n_shared, n_layers=8, max_tokens=max(T, 1),
                  max_top_k=k or sh.k, **kw)


def _setup(sh, T, k=None, **kw):
    b = _binding()
    wl = Workload(sh, T)
    d = wl.device_inputs()
    m = _mira(sh, T, k, **kw)
    blobs = m.quantize_experts(d["w1"], d["w2"], d["w3"])
    slots = b.slot_table(blobs)
    slot_map = torch.arange(sh.E + sh.n_shared, dtype=torch.int32, device="cuda")
    return wl, d, m, blobs, slots, slot_map


# ---------------------------------------------------------------- S0 / unpack
@pytest.mark.parametrize("src", ["fp32", "bf16", "heavy"])
def test_quantize_and_unpack_bit_exact(src):
    sh = inputs.TINY
    def heavy(shape, e):
        w1, w2, w3 = inputs.expert_weights(shape, e)
        g = np.random.default_rng(100 + e)
        w1 = w1 * np.exp(2 * g.standard_normal((shape.R, 1))).astype(np.float32)
        w2[g.random(w2.shape) < 0.01] *= np.float32(9.0)
        if e == 1:
            w1[5], w3[5], w2[:, 5] = 0, 0, 0        # an all-zero row-triple
        return w1, w2, w3
    wl = Workload(dataclasses.replace(sh, E=3), 4, gen=heavy if src == "heavy" else None)
    if src == "bf16":
        wl.weights = [tuple(inputs.round_to_bf16(w) for w in ws) for ws in wl.weights]
        wl.blobs = [oracle.quantize_expert(*w) for w in wl.weights]
    d = wl.device_inputs()
    m = _mira(wl.shape, 4)
    cast = (lambda t: t.to(torch.bfloat16)) if src == "bf16" else (lambda t: t)
    blobs = m.quantize_experts(cast(d["w1"]), cast(d["w2"]), cast(d["w3"]))
    torch.cuda.synchronize()
    got = blobs.cpu().numpy()
    for e, ref in enumerate(wl.blobs):
        assert got[e].size == ref.size
        assert np.array_equal(got[e], ref), f"expert {e}: {np.count_nonzero(got[e] != ref)} bytes differ"
        u = m.unpack_expert(blobs[e])
        o = oracle.unpack_expert(ref, sh.R, sh.C)
        for name in ("q1", "q2", "q3"):
            assert np.array_equal(u[name].cpu().numpy(), o[name])
        for name in ("w1", "w2", "w3"):      # 0 ULP: identical bit patterns
            assert np.array_equal(u[name].cpu().numpy().view(np.uint32), o[name].view(np.uint32))


# ---------------------------------------------------------------- S1-S3
@pytest.mark.parametrize("T", [1, 5, 16, 17, 20, 32, 33, 100])     # 16 / 17 and 32 / 33: the limits of the short grouping paths (32 and 64 pairs)
def test_route_bit_exact(T):
    sh = inputs.TINY
    wl, d, m, blobs, slots, slot_map = _setup(sh, T)
    r = m.route(d["x"], d["wr"], d["bias"], sh.k)
    torch.cuda.synchronize()
    logits = oracle.linear_scores(wl.x, wl.wr, wl.bias)
    idx, w, _, margin = oracle.topk_softmax(logits, sh.k)
    count, offset, perm, _ = oracle.group(idx, sh.E, 0)
    assert np.abs(r["logits"].cpu().numpy() - logits).max() < 1e-4
    safe = margin > 1e-5 * np.maximum(1.0, np.abs(logits).max(1))
    assert safe.all()          # the seeded workload has no near-ties, so every row is compared
    assert np.array_equal(r["idx"].cpu().numpy(), idx)
    assert np.abs(r["w"].cpu().numpy() - w).max() < 2e-6
    assert np.array_equal(r["count"].cpu().numpy(), count)
    assert np.array_equal(r["offset"].cpu().numpy(), offset)
    assert np.array_equal(r["perm"].cpu().numpy(), perm)


@pytest.mark.parametrize("T,k", [(1, 1), (1, 5), (2, 16), (3, 7), (4, 2), (4, 16)])
def test_route_single_cta_any_top_k(T, k):
    """Up to 4 tokens and 16 experts route in one CTA, which keeps the j-th selection in lane j: every k from 1 to
    the largest, selection order and weights included."""
    sh = inputs.LayerShape("route16", C=512, R=64, E=16, k=k, T=T, zipf_a=0.8, seed=31)
    wl = Workload(sh, T)
    d = wl.device_inputs()
    m = _mira(sh, T)
    r = m.route(d["x"], d["wr"], d["bias"], k)
    torch.cuda.synchronize()
    logits = oracle.linear_scores(wl.x, wl.wr, wl.bias)
    idx, w, _, margin = oracle.topk_softmax(logits, k)
    assert (margin > 1e-5 * np.maximum(1.0, np.abs(logits).max(1))).all()      # no near-ties in this seeded workload
    assert np.array_equal(r["idx"].cpu().numpy(), idx)
    assert np.abs(r["w"].cpu().numpy() - w).max() < 2e-6
    count, offset, perm, _ = oracle.group(idx, sh.E, 0)
    assert np.array_equal(r["count"].cpu().numpy(), count)
    assert np.array_equal(r["offset"].cpu().numpy(), offset)
    assert np.array_equal(r["perm"].cpu().numpy(), perm)


def test_route_ties_and_shared_positions():
    sh = SMALL_SHARED
    wl = Workload(sh, 21)
    wl.wr[3] = wl.wr[1]; wl.wr[7] = wl.wr[1]; wl.bias[3] = wl.bias[1]; wl.bias[7] = wl.bias[1]   # exact ties
    d = wl.device_inputs()
    m = _mira(sh, 21)
    r = m.route(d["x"], d["wr"], d["bias"], sh.k)
    torch.cuda.synchronize()
    got_idx = r["idx"].cpu().numpy()
    logits_gpu = r["logits"].cpu().numpy().astype(np.float64)
    assert np.array_equal(logits_gpu[:, 1], logits_gpu[:, 3]) and np.array_equal(logits_gpu[:, 1], logits_gpu[:, 7])
    # selection on the GPU's own logits must follow (value desc, index asc) exactly
    idx_ref, _, _, _ = oracle.topk_softmax(logits_gpu, sh.k)
    assert np.array_equal(got_idx, idx_ref)
    count, offset, perm, perm_sh = oracle.group(got_idx, sh.E, sh.n_shared)
    assert np.array_equal(r["count"].cpu().numpy(), count)
    assert np.array_equal(r["offset"].cpu().numpy(), offset)
    assert np.array_equal(r["perm"].cpu().numpy(), np.concatenate([perm, perm_sh], axis=1))


@pytest.mark.parametrize("shape", ["few_experts", "many_experts"])
@pytest.mark.parametrize("T", [1, 3, 9, 40, 200])
def test_route_on_signed_zeros_and_masked_experts(shape, T):
    """The selection works on integer keys derived from the logits: equal logits must tie (lower index wins; biases of
    -0.0 and +0.0 both give a logit of zero), and experts masked with a bias of -inf must never be chosen while enough
    finite logits remain. Zero tokens make every logit equal to its bias, so the logits are known exactly; every
    routing kernel (one CTA, one CTA per token, score + group kernels) is reached by the token counts."""
    sh = inputs.TINY if shape == "few_experts" else inputs.LayerShape("many", C=128, R=64, E=70, k=6, T=T, n_shared=1, seed=3)
    wl = Workload(sh, T)
    x = np.zeros((T, sh.C), dtype=np.float32)
    bias = np.zeros(sh.E, dtype=np.float32)
    bias[::2] = -0.0                                   # signed zeros: all tie, ids 0 .. k-1 in order
    m = _mira(sh, T)
    xd, wrd = to_bf16_cuda(x), to_bf16_cuda(wl.wr)
    r = m.route(xd, wrd, torch.from_numpy(bias).cuda(), sh.k)
    torch.cuda.synchronize()
    assert np.array_equal(r["idx"].cpu().numpy(), np.tile(np.arange(sh.k), (T, 1)))
    assert np.allclose(r["w"].cpu().numpy(), 1.0 / sh.k)
    g = np.random.default_rng(T)
    bias = g.standard_normal(sh.E).astype(np.float32)
    masked = g.choice(sh.E, sh.E - sh.k - 1, replace=False)        # k + 1 experts stay selectable
    bias[masked] = -np.inf
    r = m.route(xd, wrd, torch.from_numpy(bias).cuda(), sh.k)
    torch.cuda.synchronize()
    idx_ref, w_ref, _, _ = oracle.topk_softmax(np.tile(bias.astype(np.float64), (T, 1)), sh.k)
    assert np.array_equal(r["idx"].cpu().numpy(), idx_ref)
    assert np.abs(r["w"].cpu().numpy() - w_ref).max() < 1e-6
    count, offset, perm, perm_sh = oracle.group(idx_ref, sh.E, sh.n_shared)
    assert np.array_equal(r["count"].cpu().numpy(), count) and np.array_equal(r["offset"].cpu().numpy(), offset)
    assert np.array_equal(r["perm"].cpu().numpy(), np.concatenate([perm, perm_sh], axis=1))


# ---------------------------------------------------------------- S4-S6
def _check_layer(wl, out_gpu, res, fp32):
    ref = res["out64"]
    if fp32:
        a = gate_a(out_gpu, ref)
        assert a <= TOL, f"gate A {a}"
    else:
        b_, c_ = gate_b(out_gpu, ref), gate_c(out_gpu, ref, bf16_output=True)
        assert b_ <= TOL and c_ <= TOL, f"gate B {b_}, gate C {c_}"


@pytest.mark.parametrize("T", [1, 3, 16, 33, 70])
@pytest.mark.parametrize("fp32", [True, False])
def test_tiny_layer(T, fp32):
    sh = inputs.TINY
    wl, d, m, blobs, slots, slot_map = _setup(sh, T, out_fp32=fp32)
    out, dbg = m.moe_layer(d["x"], d["wr"], d["bias"], slots, slot_map, sh.k, debug=True)
    torch.cuda.synchronize()
    res = oracle.moe_layer(wl.x, wl.wr, wl.bias, wl.blobs, sh.R, sh.k)
    assert np.array_equal(dbg["idx"].cpu().numpy(), res["idx"])
    _check_layer(wl, out.float().cpu().numpy(), res, fp32)
    assert m.poll_status()[0] == 0


@pytest.mark.parametrize("T", [9, 80])              # 80 tokens: the tensor-core kernels
@pytest.mark.parametrize("act_on_w1", [False, True])
def test_dense_mixture_and_activation_flag(act_on_w1, T):
    sh = inputs.TINY
    wl, d, m, blobs, slots, slot_map = _setup(sh, T, k=sh.E, out_fp32=True, act_on_w1=act_on_w1)
    out = m.moe_layer(d["x"], d["wr"], d["bias"], slots, slot_map, sh.E)
    res = oracle.moe_layer(wl.x, wl.wr, wl.bias, wl.blobs, sh.R, sh.E, act_on_w1=act_on_w1)
    assert gate_a(out.cpu().numpy(), res["out64"]) <= TOL


@pytest.mark.parametrize("T", [37, 131])            # 131 tokens: the tensor-core kernels, ragged tiles
@pytest.mark.parametrize("scale", [1.0, 1e-3, 30.0])
def test_shared_experts_ragged_and_weight_magnitudes(scale, T):
    sh = SMALL_SHARED
    wl = Workload(sh, T, weight_scale=scale)
    d = wl.device_inputs()
    b = _binding()
    for fp32 in (True, False):
        m = _mira(sh, T, out_fp32=fp32)
        blobs = m.quantize_experts(d["w1"], d["w2"], d["w3"])
        assert np.array_equal(blobs.cpu().numpy(), np.stack(wl.blobs))
        slot_map = torch.arange(sh.E + sh.n_shared, dtype=torch.int32, device="cuda")
        out = m.moe_layer(d["x"], d["wr"], d["bias"], b.slot_table(blobs), slot_map, sh.k)
        res = oracle.moe_layer(wl.x, wl.wr, wl.bias, wl.blobs, sh.R, sh.k, n_shared=sh.n_shared)
        _check_layer(wl, out.float().cpu().numpy(), res, fp32)


@pytest.mark.parametrize("T", [6, 70])
def test_large_activations_do_not_overflow_fp16(T):
    sh = inputs.TINY
    wl = Workload(sh, T)
    wl.x = inputs.round_to_bf16(wl.x * np.float32(3.0e5))
    wl.x[2] = inputs.round_to_bf16(wl.x[2] * np.float32(1e-9))
    d = wl.device_inputs()
    b = _binding()
    m = _mira(sh, T, out_fp32=True)
    blobs = m.quantize_experts(d["w1"], d["w2"], d["w3"])
    out = m.moe_layer(d["x"], d["wr"], None, b.slot_table(blobs), torch.arange(sh.E, dtype=torch.int32, device="cuda"), sh.k)
    res = oracle.moe_layer(wl.x, wl.wr, None, wl.blobs, sh.R, sh.k)
    assert np.isfinite(out.cpu().numpy()).all()
    assert gate_a(out.cpu().numpy(), res["out64"]) <= TOL


@pytest.mark.parametrize("T", [24, 96])
def test_slot_permutation_is_bit_identical_and_missing_expert_is_reported(T):
    sh = inputs.TINY
    wl, d, m, blobs, slots, slot_map = _setup(sh, T)
    base = m.moe_layer(d["x"], d["wr"], d["bias"], slots, slot_map, sh.k)
    p = torch.tensor([5, 2, 7, 0, 3, 6, 1, 4], device="cuda")              # expert e lives in slot p[e]
    moved = torch.empty_like(blobs)
    moved[p] = blobs
    b = _binding()
    out2 = m.moe_layer(d["x"], d["wr"], d["bias"], b.slot_table(moved), p.to(torch.int32), sh.k)
    assert torch.equal(base.view(torch.int16), out2.view(torch.int16))
    # drop the most used expert
    res_full = oracle.moe_layer(wl.x, wl.wr, wl.bias, wl.blobs, sh.R, sh.k)
    victim = int(np.bincount(res_full["idx"].ravel(), minlength=sh.E).argmax())
    sm = slot_map.clone(); sm[victim] = -1
    out3 = m.moe_layer(d["x"], d["wr"], d["bias"], slots, sm, sh.k)
    code, missing = m.poll_status()
    assert code == b.MIRA_ERR_EXPERT_MISS and missing == [victim]
    holes = list(wl.blobs); holes[victim] = None
    res = oracle.moe_layer(wl.x, wl.wr, wl.bias, holes, sh.R, sh.k)
    assert gate_b(out3.float().cpu().numpy(), res["out64"]) <= TOL
    assert m.poll_status()[0] == 0          # cleared by the previous poll


def test_waves_equal_single_call():
    sh = SMALL_SHARED
    wl, d, m, blobs, slots, slot_map = _setup(sh, 29)
    one = m.moe_layer(d["x"], d["wr"], d["bias"], slots, slot_map, sh.k)
    r = m.route(d["x"], d["wr"], d["bias"], sh.k)
    needed = [e for e, c in enumerate(r["count"].cpu().tolist()) if c > 0]
    first, second = needed[::2], needed[1::2]
    m.moe_experts(d["x"], slots, slot_map, expert_ids=first, final_wave=False)
    two = m.moe_experts(d["x"], slots, slot_map, expert_ids=second, final_wave=True)
    assert torch.equal(one.view(torch.int16), two.view(torch.int16))
    assert m.poll_status()[0] == 0
    # a wave that never ran is a miss
    m.route(d["x"], d["wr"], d["bias"], sh.k)
    m.moe_experts(d["x"], slots, slot_map, expert_ids=first, final_wave=True)
    code, missing = m.poll_status()
    assert code == _binding().MIRA_ERR_EXPERT_MISS and missing == sorted(second)


# ---------------------------------------------------------------- S4-S5, tensor-core (tcgen05) path for large batches
@pytest.mark.parametrize("case", ["tiny300", "shared400"])
def test_tensor_core_path_matches_oracle_and_streaming_path(case):
    sh, T = (inputs.TINY, 300) if case == "tiny300" else (dataclasses.replace(SMALL_SHARED, R=192, C=128), 400)
    b = _binding()
    wl = Workload(sh, T)
    d = wl.device_inputs()
    res = oracle.moe_layer(wl.x, wl.wr, wl.bias, wl.blobs, sh.R, sh.k, n_shared=sh.n_shared)
    outs = {}
    for fp32 in (True, False):
        m = _mira(sh, T, out_fp32=fp32)
        blobs = m.quantize_experts(d["w1"], d["w2"], d["w3"])
        slot_map = torch.arange(sh.E + sh.n_shared, dtype=torch.int32, device="cuda")
        out = m.moe_layer(d["x"], d["wr"], d["bias"], b.slot_table(blobs), slot_map, sh.k)      # T >= 256: tcgen05 kernels
        torch.cuda.synchronize()
        assert m.poll_status()[0] == 0
        _check_layer(wl, out.float().cpu().numpy(), res, fp32)
        m.force_decode_path(True)
        out2 = m.moe_layer(d["x"], d["wr"], d["bias"], b.slot_table(blobs), slot_map, sh.k)
        torch.cuda.synchronize()
        _check_layer(wl, out2.float().cpu().numpy(), res, fp32)
        outs[fp32] = (out, out2)
    # the two paths use the same exact integer products and differ only in fp32 summation order (and what that does to the fp16 intermediate)
    a, c = outs[True]
    assert gate_a(a.cpu().numpy(), c.cpu().numpy().astype(np.float64)) < 1e-3    # fp16 rounding of the intermediate may differ


# ---------------------------------------------------------------- S7 / S8 / host checks
@pytest.mark.parametrize("T", [1, 7, 130])
def test_predictor(T):
    sh = SMALL_SHARED
    wl = Workload(dataclasses.replace(sh, E=12, n_shared=0), T)
    d = wl.device_inputs()
    m = _mira(wl.shape, T)
    pooled, ts, ids = m.predict(2, d["x"], d["wp"], d["bp"], k_pred=3, token_scores=True)
    ts_ref, pooled_ref, ids_ref, margin = oracle.predict(wl.x, wl.wp, wl.bp, k_pred=3)
    assert np.abs(ts.cpu().numpy() - ts_ref).max() < 1e-4
    assert np.abs(pooled.cpu().numpy() - pooled_ref).max() < 1e-4
    assert margin > 1e-4 and np.array_equal(ids.cpu().numpy(), ids_ref)
    pooled2, _, ids2 = m.predict(0, d["x"], d["wp"], None, k_pred=1)       # scratch token scores, no bias
    _, pooled_ref2, ids_ref2, _ = oracle.predict(wl.x, wl.wp, None, k_pred=1)
    assert np.abs(pooled2.cpu().numpy() - pooled_ref2).max() < 1e-4 and ids2.item() == ids_ref2[0]
    b = _binding()
    with pytest.raises(b.MiraError) as ei:
        m.predict(6, d["x"], d["wp"], d["bp"])          # n_layers = 8: layers 6 and 7 have no head
    assert ei.value.code == b.MIRA_ERR_NO_PREDICTOR


def test_stage_expert_copies_blob_and_records_event():
    sh = inputs.TINY
    wl, d, m, blobs, slots, slot_map = _setup(sh, 8)
    host = torch.from_numpy(np.stack(wl.blobs)).pin_memory()
    cache = torch.zeros((2, m.expert_bytes), dtype=torch.uint8, device="cuda")
    side = torch.cuda.Stream()
    ev = torch.cuda.Event()
    m.stage_expert(host[3], cache[1], side, ev)
    torch.cuda.current_stream().wait_event(ev)
    assert torch.equal(cache[1].cpu(), host[3]) and not cache[0].any()



def test_staged_waves_on_the_tensor_core_path_equal_the_resident_call():
    """The third workload's flow at a small size: a cache with fewer slots than experts, the missing experts copied
    from pinned host memory into STAGE slots on a side stream and run as later waves (T >= 256: tcgen05 kernels)."""
    b = _binding()
    sh, T = SMALL_SHARED, 320
    wl, d, m, blobs, slots, slot_map = _setup(sh, T)
    n = sh.E + sh.n_shared
    ref = m.moe_layer(d["x"], d["wr"], d["bias"], slots, slot_map, sh.k)
    host = blobs.cpu().pin_memory()
    shared = list(range(sh.E, n))
    hot = [0, 2, 4, 6, 8, 10] + shared                      # resident: half of the routed experts and the shared ones
    cold = [e for e in range(sh.E) if e not in hot]
    n_stage = 2
    cache = torch.zeros((len(hot) + n_stage, m.expert_bytes), dtype=torch.uint8, device="cuda")
    for i, e in enumerate(hot):
        cache[i].copy_(blobs[e])
    cslots = b.slot_table(cache)

    def smap(pairs):
        t = torch.full((n,), -1, dtype=torch.int32)
        for e, sl in pairs:
            t[e] = sl
        return t.cuda()
    r = m.route(d["x"], d["wr"], d["bias"], sh.k)
    cnt = r["count"].cpu().tolist()
    need_cold = [e for e in cold if cnt[e] > 0]
    assert len(need_cold) >= 3                               # at least two staged waves
    side, main = torch.cuda.Stream(), torch.cuda.current_stream()
    ready = [torch.cuda.Event() for _ in range(n_stage)]
    waves = [need_cold[j:j + n_stage] for j in range(0, len(need_cold), n_stage)]
    for sl, e in enumerate(waves[0]):
        m.stage_expert(host[e], cache[len(hot) + sl], side, ready[sl])
    m.moe_experts(d["x"], cslots, smap([(e, i) for i, e in enumerate(hot)]), expert_ids=[e for e in hot if cnt[e] > 0],
                  final_wave=False)
    out = None
    for wi, wave in enumerate(waves):
        for sl in range(len(wave)):
            main.wait_event(ready[sl])
        out = m.moe_experts(d["x"], cslots, smap([(e, len(hot) + sl) for sl, e in enumerate(wave)]), expert_ids=wave,
                            final_wave=wi == len(waves) - 1)
        if wi + 1 < len(waves):
            done = torch.cuda.Event()
            done.record(main)
            side.wait_event(done)                            # the STAGE slots are free once this wave has run
            for sl, e in enumerate(waves[wi + 1]):
                m.stage_expert(host[e], cache[len(hot) + sl], side, ready[sl])
    torch.cuda.synchronize()
    assert m.poll_status()[0] == 0
    assert torch.equal(out.view(torch.int16), ref.view(torch.int16))


def test_host_side_argument_checks():
    b = _binding()
    sh = inputs.TINY
    with pytest.raises(b.MiraError) as ei:
        b.Mira(100, sh.R, sh.E)                      # C % 64 != 0
    assert ei.value.code == b.MIRA_ERR_SHAPE
    wl, d, m, blobs, slots, slot_map = _setup(sh, 4)
    with pytest.raises(b.MiraError) as ei:
        m.moe_layer(d["x"], d["wr"], d["bias"], slots, slot_map, 3)      # k > max_top_k
    assert ei.value.code == b.MIRA_ERR_WORKSPACE
    big = to_bf16_cuda(inputs.hidden(sh, 9))
    with pytest.raises(b.MiraError) as ei:
        m.moe_layer(big, d["wr"], d["bias"], slots, slot_map, sh.k)      # T > max_tokens
    assert ei.value.code == b.MIRA_ERR_WORKSPACE
    with pytest.raises(b.MiraError) as ei:
        buf = torch.zeros(4 * sh.C + 8, dtype=torch.bfloat16, device="cuda")
        m.moe_layer(buf[1:1 + 4 * sh.C].view(4, sh.C), d["wr"], d["bias"], slots, slot_map, sh.k)   # 2-byte offset
    assert ei.value.code == b.MIRA_ERR_ALIGN
    empty = torch.empty((0, sh.C), dtype=torch.bfloat16, device="cuda")
    out = m.moe_layer(empty, d["wr"], d["bias"], slots, slot_map, sh.k)  # T = 0 is a no-op
    assert out.shape == (0, sh.C)
    assert m.kernel_launches > 0


@pytest.mark.parametrize("T", [4, 5, 8, 9, 40, 300])
def test_many_experts_near_the_limits(T):
    """200 routed + 3 shared experts (the library's limit is 256 in total), top-8: routing tables, schedule and
    both expert paths at their widest."""
    sh = inputs.LayerShape("wide", C=128, R=64, E=200, k=8, T=T, n_shared=3, zipf_a=1.1, seed=11)
    wl, d, m, blobs, slots, slot_map = _setup(sh, T)
    out, dbg = m.moe_layer(d["x"], d["wr"], d["bias"], slots, slot_map, sh.k, debug=True)
    torch.cuda.synchronize()
    assert m.poll_status()[0] == 0
    res = oracle.moe_layer(wl.x, wl.wr, wl.bias, wl.blobs, sh.R, sh.k, n_shared=sh.n_shared)
    assert np.array_equal(dbg["idx"].cpu().numpy(), res["idx"])
    count, offset, perm, perm_sh = oracle.group(res["idx"], sh.E, sh.n_shared)
    assert np.array_equal(dbg["count"].cpu().numpy(), count) and np.array_equal(dbg["offset"].cpu().numpy(), offset)
    assert np.array_equal(dbg["perm"].cpu().numpy(), np.concatenate([perm, perm_sh], axis=1))
    _check_layer(wl, out.float().cpu().numpy(), res, False)


@pytest.mark.parametrize("layout", [1, 2, 3, 4, 5])
@pytest.mark.parametrize("shape", ["tiny", "small_shared", "pairs"])
def test_every_tile_layout_of_the_tensor_core_kernels(layout, shape):
    """Each tile layout forced in turn (narrow / wide / big, and the two-SM kernel in both of its forms) on batches
    with full, ragged and multi-tile experts; left to itself a step only ever takes the layout its token count
    selects. ("small_shared" has sizes the two-SM kernel does not take: there layouts 4 and 5 must fall back.)"""
    sh = {"tiny": inputs.TINY, "small_shared": SMALL_SHARED,
          "pairs": inputs.LayerShape("pairs", C=512, R=384, E=5, k=2, T=300, n_shared=1, zipf_a=1.3, seed=17)}[shape]
    for T in (70, 300, 900):
        wl, d, m, blobs, slots, slot_map = _setup(sh, T, out_fp32=True)
        m.tensor_layout(layout)
        out = m.moe_layer(d["x"], d["wr"], d["bias"], slots, slot_map, sh.k)
        torch.cuda.synchronize()
        assert m.poll_status()[0] == 0
        res = oracle.moe_layer(wl.x, wl.wr, wl.bias, wl.blobs, sh.R, sh.k, n_shared=sh.n_shared)
        assert gate_a(out.cpu().numpy(), res["out64"]) <= TOL, f"layout {layout}, T={T}"


@pytest.mark.parametrize("T", [1, 6, 70])
def test_largest_hidden_size_and_top_k(T):
    """Hidden size 16384 (the library's limit) with a small expert width, and top-16 of 16 experts (the largest k):
    the routing kernels' shared-memory plans, the quantizer's row kernels and both expert paths at their longest
    reduction."""
    sh = inputs.LayerShape("long", C=16384, R=128, E=16, k=16, T=T, seed=12)
    wl, d, m, blobs, slots, slot_map = _setup(sh, T, out_fp32=True)
    assert np.array_equal(blobs.cpu().numpy(), np.stack(wl.blobs))
    out, dbg = m.moe_layer(d["x"], d["wr"], d["bias"], slots, slot_map, sh.k, debug=True)
    torch.cuda.synchronize()
    assert m.poll_status()[0] == 0
    res = oracle.moe_layer(wl.x, wl.wr, wl.bias, wl.blobs, sh.R, sh.k)
    assert np.array_equal(np.sort(dbg["idx"].cpu().numpy(), axis=1), np.sort(res["idx"], axis=1))   # k = E: every expert
    got = out.cpu().numpy()
    # every row, elementwise and row-wise (at this hidden size the up/gate kernels convert the codes exactly: the
    # offset form's subtracted term would cost accuracy over 1024 accumulation steps)
    assert gate_a(got, res["out64"]) <= TOL and gate_c(got, res["out64"]) <= TOL


@pytest.mark.parametrize("T", [3, 40, 150])
def test_sizes_that_are_multiples_of_64_only(T):
    """Hidden size 192 and expert width 320 (multiples of 64, not of 128): the tensor-core kernels do not take this
    shape, so the weight-streaming kernels also serve the large batches; partial last stages in both reductions."""
    sh = inputs.LayerShape("odd", C=192, R=320, E=6, k=3, T=T, n_shared=1, zipf_a=1.0, seed=13)
    wl, d, m, blobs, slots, slot_map = _setup(sh, T, out_fp32=True)
    assert np.array_equal(blobs.cpu().numpy(), np.stack(wl.blobs))
    out = m.moe_layer(d["x"], d["wr"], d["bias"], slots, slot_map, sh.k)
    torch.cuda.synchronize()
    assert m.poll_status()[0] == 0
    res = oracle.moe_layer(wl.x, wl.wr, wl.bias, wl.blobs, sh.R, sh.k, n_shared=sh.n_shared)
    assert gate_a(out.cpu().numpy(), res["out64"]) <= TOL


@pytest.mark.parametrize("T", [4, 80])
def test_layer_call_can_be_captured_in_a_cuda_graph(T):
    """mira_moe_layer makes no host synchronisation, allocation or copy, so a decode loop may capture it in a CUDA
    graph: the replay (on new input values in the same buffers) is bit-identical to a direct call."""
    sh = inputs.TINY
    wl, d, m, blobs, slots, slot_map = _setup(sh, T)
    x = d["x"].clone()
    out = torch.empty((T, sh.C), dtype=torch.bfloat16, device="cuda")
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(s):
        m.moe_layer(x, d["wr"], d["bias"], slots, slot_map, sh.k, out=out, stream=s)       # first call outside the capture
        s.synchronize()
        g.capture_begin()
        m.moe_layer(x, d["wr"], d["bias"], slots, slot_map, sh.k, out=out, stream=s)
        g.capture_end()
    torch.cuda.synchronize()
    x2 = to_bf16_cuda(inputs.hidden(sh, T, step=3))
    direct = m.moe_layer(x2, d["wr"], d["bias"], slots, slot_map, sh.k).clone()
    torch.cuda.synchronize()
    x.copy_(x2)
    out.zero_()
    g.replay()
    torch.cuda.synchronize()
    assert m.poll_status()[0] == 0
    assert torch.equal(out.view(torch.int16), direct.view(torch.int16))


def test_quantizer_does_not_depend_on_the_token_capacity():
    """A context sized for a single token and top-1 still quantizes: the quantizer's scratch (one abs-max per
    expert-hidden row) must fit whatever max_tokens is."""
    sh = inputs.LayerShape("thin", C=64, R=640, E=3, k=1, T=1, n_shared=1, seed=14)
    wl, d, m, blobs, slots, slot_map = _setup(sh, 1, out_fp32=True)
    assert np.array_equal(blobs.cpu().numpy(), np.stack(wl.blobs))
    out = m.moe_layer(d["x"], d["wr"], d["bias"], slots, slot_map, sh.k)
    res = oracle.moe_layer(wl.x, wl.wr, wl.bias, wl.blobs, sh.R, sh.k, n_shared=sh.n_shared)
    assert gate_a(out.cpu().numpy(), res["out64"]) <= TOL


@pytest.mark.parametrize("mins", [(9, 9), (17, 2 ** 31 - 1), (2 ** 31 - 1, 5), (5, 17), (33, 33), (1, 1)])
@pytest.mark.parametrize("shape", ["tiny", "small_shared"])
def test_hybrid_steps_split_the_experts_between_the_kernel_families(shape, mins):
    """A step may hand the experts with few pairs to the weight-streaming kernels and the others to the tcgen05
    kernels, per projection (thresholds forced here; the skewed routing gives both kinds in every batch). Against the
    oracle, and as waves (the split is a property of the step, so waves reproduce the single call bit for bit)."""
    sh = inputs.TINY if shape == "tiny" else SMALL_SHARED
    for T in (40, 130):
        wl, d, m, blobs, slots, slot_map = _setup(sh, T, out_fp32=True)
        m.hybrid_min(*mins)
        out, dbg = m.moe_layer(d["x"], d["wr"], d["bias"], slots, slot_map, sh.k, debug=True)
        torch.cuda.synchronize()
        assert m.poll_status()[0] == 0
        cnt = dbg["count"].cpu().numpy()
        res = oracle.moe_layer(wl.x, wl.wr, wl.bias, wl.blobs, sh.R, sh.k, n_shared=sh.n_shared)
        assert gate_a(out.cpu().numpy(), res["out64"]) <= TOL, f"T={T} mins={mins} counts={cnt.tolist()}"
        needed = [e for e, c in enumerate(cnt.tolist()) if c > 0]
        m.route(d["x"], d["wr"], d["bias"], sh.k)
        m.moe_experts(d["x"], slots, slot_map, expert_ids=needed[::2], final_wave=False)
        two = m.moe_experts(d["x"], slots, slot_map, expert_ids=needed[1::2], final_wave=True)
        assert torch.equal(out, two)


@pytest.mark.parametrize("layout", [0, 1, 2, 3])
def test_reduction_slices_of_the_tensor_core_down_kernel(layout):
    """The tcgen05 down kernel may cut the expert-hidden dimension into slices (tiles of their own, partial sums added
    by S6 in slice order). Expert width 12416 = 194 K-blocks (uneven thirds and quarters) gives the workspace four
    partial-sum slices; 1..4 slices are forced in turn on full, ragged and multi-tile experts, one of them a wide-range
    expert (two fp16 windows). Against the oracle; as waves (bit-identical: the slices are a property of the step);
    and a hybrid step whose small experts take the streaming down kernel with its own four slices."""
    def gen(shape, e):
        w1, w2, w3 = inputs.expert_weights(shape, e)
        if e == 1:
            g = np.random.default_rng(100 + e)
            w1 = w1 * np.exp(2 * g.standard_normal((shape.R, 1))).astype(np.float32)
        return w1, w2, w3
    sh = inputs.LayerShape("slices", C=256, R=12416, E=3, k=2, T=330, n_shared=1, zipf_a=1.2, seed=23)
    b = _binding()
    for T in (70, 330):
        wl = Workload(sh, T, gen=gen)
        d = wl.device_inputs()
        m = _mira(sh, T, None, out_fp32=True)
        blobs = m.quantize_experts(d["w1"], d["w2"], d["w3"])
        slots = b.slot_table(blobs)
        slot_map = torch.arange(sh.E + sh.n_shared, dtype=torch.int32, device="cuda")
        res = oracle.moe_layer(wl.x, wl.wr, wl.bias, wl.blobs, sh.R, sh.k, n_shared=sh.n_shared)
        m.tensor_layout(layout)
        outs = []
        for n in (1, 2, 3, 4):
            m.down_slices(n)
            out, dbg = m.moe_layer(d["x"], d["wr"], d["bias"], slots, slot_map, sh.k, debug=True)
            torch.cuda.synchronize()
            assert m.poll_status()[0] == 0
            assert gate_a(out.cpu().numpy(), res["out64"]) <= TOL, f"layout {layout}, T={T}, {n} slices"
            outs.append(out.clone())
        assert not torch.equal(outs[0], outs[2])                  # the slices were really taken: another order of additions
        cnt = dbg["count"].cpu().tolist()
        needed = [e for e, c in enumerate(cnt) if c > 0]
        m.down_slices(3)
        m.route(d["x"], d["wr"], d["bias"], sh.k)
        m.moe_experts(d["x"], slots, slot_map, expert_ids=needed[::2], final_wave=False)
        two = m.moe_experts(d["x"], slots, slot_map, expert_ids=needed[1::2], final_wave=True)
        assert torch.equal(outs[2], two)
        m.hybrid_min(0, sorted(cnt[:sh.E])[1] + 1)               # the two least-loaded routed experts: streaming down kernel
        out = m.moe_layer(d["x"], d["wr"], d["bias"], slots, slot_map, sh.k)
        torch.cuda.synchronize()
        assert m.poll_status()[0] == 0
        assert gate_a(out.cpu().numpy(), res["out64"]) <= TOL
        m.hybrid_min(-1, -1)
        m.down_slices(0)                                          # the library's own choice for this batch
        out = m.moe_layer(d["x"], d["wr"], d["bias"], slots, slot_map, sh.k)
        assert gate_a(out.cpu().numpy(), res["out64"]) <= TOL
        if layout == 0:                                           # the two-SM kernel takes whole reductions whatever is forced
            m.tensor_layout(4)
            m.down_slices(1)
            one = m.moe_layer(d["x"], d["wr"], d["bias"], slots, slot_map, sh.k).clone()
            m.down_slices(3)
            three = m.moe_layer(d["x"], d["wr"], d["bias"], slots, slot_map, sh.k)
            assert torch.equal(one, three) and gate_a(one.cpu().numpy(), res["out64"]) <= TOL
