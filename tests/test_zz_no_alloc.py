"""mira_predict_noalloc: the predictor head for callers that cannot allocate device memory (its scratch
is a fixed array inside the library). Collected last on purpose: if it fails, a run that stops at the
first failure has already run every other test.

Checked against the CPU oracle (pooled scores within 1e-4, ids identical wherever the oracle's margin
exceeds that) and against the ordinary entry point mira_predict on the same inputs, on two calls in a
row with different inputs, so that stale contents of the shared scratch array from the first call
would show in the second. The file also works alone in a fresh process: nothing here depends on
another test having created a context first (mira_predict's context is created after the no-alloc
calls)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2609_38090_b200 import inputs

pytestmark = pytest.mark.gpu
TOL = 1e-4


def test_predict_noalloc_matches_oracle_and_predict_on_two_calls_in_a_row():
    from paper_2609_38090_b200 import binding as b
    sh = inputs.LayerShape("noalloc", C=512, R=64, E=24, k=2, T=50, seed=11)
    dev = torch.device("cuda:0")
    wp_np, bp_np = inputs.predictor(sh)
    wp = torch.from_numpy(wp_np).to(torch.bfloat16).to(dev)
    bp = torch.from_numpy(bp_np).to(dev)
    xs_np = [inputs.hidden(sh, T, step=i) for i, T in enumerate((50, 7))]
    xs = [torch.from_numpy(x).to(torch.bfloat16).to(dev) for x in xs_np]
    # outputs are caller-provided, as a caller without an allocator would do
    pooled = [torch.zeros(sh.E, dtype=torch.float32, device=dev) for _ in xs]
    ids = [torch.zeros(3, dtype=torch.int32, device=dev) for _ in xs]
    for x, p, i in zip(xs, pooled, ids):                       # two calls in a row, same stream
        b.predict_noalloc(x, wp, bp, k_pred=3, pooled=p, ids=i)
    torch.cuda.synchronize()
    m = b.Mira(sh.C, sh.R, sh.E, n_layers=8, max_tokens=64, max_top_k=2)      # the existing entry point
    for x_np, x, p, i in zip(xs_np, xs, pooled, ids):
        _, pooled_ref, ids_ref, margin = oracle.predict(x_np, wp_np, bp_np, k_pred=3)
        assert np.abs(p.cpu().numpy() - pooled_ref).max() < TOL
        assert margin > TOL and np.array_equal(i.cpu().numpy(), ids_ref)      # no near-tie in this seeded workload
        gpu_pooled, _, gpu_ids = m.predict(0, x, wp, bp, k_pred=3)
        torch.cuda.synchronize()
        assert np.abs(p.cpu().numpy() - gpu_pooled.cpu().numpy()).max() < TOL
        assert np.array_equal(i.cpu().numpy(), gpu_ids.cpu().numpy())
    # optional arguments left out: no bias, no ids wanted
    p2 = torch.zeros(sh.E, dtype=torch.float32, device=dev)
    _, none_ids = b.predict_noalloc(xs[0], wp, None, k_pred=0, pooled=p2)
    torch.cuda.synchronize()
    _, pooled_nobias, _, _ = oracle.predict(xs_np[0], wp_np, None, k_pred=1)
    assert none_ids is None and np.abs(p2.cpu().numpy() - pooled_nobias).max() < TOL


def test_predict_noalloc_refusals():
    from paper_2609_38090_b200 import binding as b
    sh = inputs.LayerShape("noalloc", C=512, R=64, E=24, k=2, T=8, seed=11)
    dev = torch.device("cuda:0")
    wp = torch.zeros((sh.E, sh.C), dtype=torch.bfloat16, device=dev)
    x = torch.zeros((8, sh.C), dtype=torch.bfloat16, device=dev)

    def refused(code, *args, **kw):
        with pytest.raises(b.MiraError) as ei:
            b.predict_noalloc(*args, **kw)
        assert ei.value.code == code
    # sizes beyond the built-in scratch are refused with a clear status, not truncated
    refused(b.MIRA_ERR_WORKSPACE, torch.zeros((65536 // sh.E + 1, sh.C), dtype=torch.bfloat16, device=dev), wp, None, k_pred=3)
    refused(b.MIRA_ERR_SHAPE, torch.zeros((8, 100), dtype=torch.bfloat16, device=dev),
            torch.zeros((sh.E, 100), dtype=torch.bfloat16, device=dev), None, k_pred=3)          # hidden size not a multiple of 8
    refused(b.MIRA_ERR_INVALID_ARG, x, wp, None, k_pred=sh.E + 1)                                 # more ids than experts
    refused(b.MIRA_ERR_INVALID_ARG, x, wp, None, k_pred=17)                                       # beyond the largest top-k
    buf = torch.zeros(8 * sh.C + 8, dtype=torch.bfloat16, device=dev)
    refused(b.MIRA_ERR_ALIGN, buf[1:1 + 8 * sh.C].view(8, sh.C), wp, None, k_pred=3)             # 2-byte offset
