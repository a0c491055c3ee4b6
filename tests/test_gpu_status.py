"""The device status word and what mira_poll_status makes of it: an expert miss, a timed-out wait, both.

Two kinds of test. The decoding is checked by writing the status word from the host side of the test (the word
is the first int32 of the caller's workspace), with no kernel involved. The time-out path of the tcgen05 kernels
is then taken for real, in its one safe form: every wait in those kernels is bounded, and the library's test
hook makes one CTA skip one activation load and give up after a few thousand polls, so the kernel returns by
itself with the status bit set, its tensor memory freed and the context usable."""
import numpy as np
import pytest
import torch

from paper_2609_38090_b200 import inputs
from gpu_util import Workload

pytestmark = pytest.mark.gpu


def _setup(T):
    from paper_2609_38090_b200 import binding as b
    sh = inputs.TINY
    wl = Workload(sh, T)
    d = wl.device_inputs()
    m = b.Mira(sh.C, sh.R, sh.E, n_layers=4, max_tokens=T, max_top_k=sh.k)
    blobs = m.quantize_experts(d["w1"], d["w2"], d["w3"])
    return b, sh, d, m, b.slot_table(blobs), torch.arange(sh.E, dtype=torch.int32, device="cuda"), blobs


def _status_words(m):
    off = (-m.workspace.data_ptr()) % 256                  # the context starts at the next 256-byte boundary
    return m.workspace[off:off + 128].view(torch.int32)    # [0] status bits, [16..23] miss mask


def test_poll_status_decodes_miss_and_timeout_bits():
    b, sh, d, m, slots, slot_map, _ = _setup(8)
    torch.cuda.synchronize()
    words = _status_words(m)
    assert m.poll_status() == (b.MIRA_OK, [])
    words[0] = 2                                            # a wait ran out
    assert m.poll_status() == (b.MIRA_ERR_TIMEOUT, [])
    assert m.poll_status() == (b.MIRA_OK, [])               # cleared by the poll
    words[0] = 1; words[16] = 0b101000                      # experts 3 and 5 were missing
    assert m.poll_status() == (b.MIRA_ERR_EXPERT_MISS, [3, 5])
    words[0] = 3; words[16] = 0b10                          # both: the time-out wins, the mask is still reported
    assert m.poll_status() == (b.MIRA_ERR_TIMEOUT, [1])
    assert m.poll_status() == (b.MIRA_OK, [])
    assert b.mira_status_string(b.MIRA_ERR_TIMEOUT).decode() != b.mira_status_string(b.MIRA_ERR_EXPERT_MISS).decode()


def test_a_wait_that_runs_out_is_reported_and_the_context_stays_usable():
    T = 96                                                  # the tcgen05 kernels
    b, sh, d, m, slots, slot_map, _ = _setup(T)
    good = m.moe_layer(d["x"], d["wr"], d["bias"], slots, slot_map, sh.k).clone()
    assert m.poll_status()[0] == b.MIRA_OK
    m.test_wait_timeout()                                   # one CTA of the next up/gate launch never gets one of its tiles
    m.moe_layer(d["x"], d["wr"], d["bias"], slots, slot_map, sh.k)
    code, missing = m.poll_status()                         # the call returned by itself: the poll synchronises
    assert code == b.MIRA_ERR_TIMEOUT and missing == []
    again = m.moe_layer(d["x"], d["wr"], d["bias"], slots, slot_map, sh.k)
    assert m.poll_status()[0] == b.MIRA_OK                  # the hook was for one launch; tensor memory was freed
    assert torch.equal(again.view(torch.int16), good.view(torch.int16))
