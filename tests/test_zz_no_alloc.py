"""disco_draft_step_static: the draft step for hosts that are not allowed to allocate device memory.

A serving process whose GPU memory belongs to another component, or a decode loop that cannot take the
device synchronisation of a cudaMalloc, cannot create a disco context (disco_create allocates).  The
static entry point keeps its scratch in a fixed array inside libdisco.so instead.  This test calls it
through the C ABI and checks it against the context-based entry point on the same inputs, twice in a
row, because the second call finds the array as the first one left it.

The file name sorts last on purpose: a run that stops at the first failure has then already run every
other test.  The test does not depend on anything those tests leave behind.
"""
import numpy as np
import pytest
import torch

from paper_2405_04304_b200 import binding, inputs
from util import PROB_TOL, make_clf, to_gpu_clf

pytestmark = pytest.mark.gpu


def _run_both(V, d, B, seed, H=32):
    W = inputs.lm_head(V, d, seed=seed, std=0.2).cuda()
    h = inputs.hidden(B, d, seed=seed + 1).cuda()
    clf = to_gpu_clf(make_clf(H, seed=seed + 2))
    pos = (torch.arange(B, dtype=torch.int32) * 5 + 2).cuda()
    nd = (torch.arange(B, dtype=torch.int32) % 3 + 1).cuda()
    active = None if B < 3 else torch.tensor([1, 0, 1, 1][:B], dtype=torch.uint8).cuda()

    def outputs():
        return (torch.full((B,), -7, dtype=torch.int32, device="cuda"),
                torch.full((B,), -7.0, dtype=torch.float32, device="cuda"),
                torch.full((B,), 77, dtype=torch.uint8, device="cuda"),
                torch.full((B, binding.NFEAT), -7.0, dtype=torch.float32, device="cuda"))

    ctx = binding.Context(V, d, 8, max_batch=B, max_rows=8, clf_hidden=H)
    ctx.set_kernel_path(1)                      # the same kernel family the static entry point uses
    t0, c0, h0, f0 = outputs()
    ctx.draft_step(W, h, pos, nd, clf, 0.5, 3, t0, c0, h0, active=active, feats=f0)
    t1, c1, h1, f1 = outputs()
    binding.draft_step_static(W, h, pos, nd, clf, 0.5, 3, t1, c1, h1, active=active, feats=f1)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    ctx.close()
    assert torch.equal(t0, t1), "tokens differ"
    assert torch.equal(h0, h1), "halt flags differ"
    np.testing.assert_allclose(c1.cpu().numpy(), c0.cpu().numpy(), rtol=0, atol=PROB_TOL)
    np.testing.assert_allclose(f1.cpu().numpy(), f0.cpu().numpy(), rtol=0, atol=PROB_TOL)
    if active is not None:                      # a skipped sequence keeps the caller's values
        assert int(t1[1]) == -7 and int(h1[1]) == 77


def test_static_entry_point_matches_context_entry_point_twice_in_a_row():
    _run_both(V=32000, d=768, B=1, seed=100)    # first call on the device also does the set-up
    _run_both(V=32000, d=768, B=1, seed=200)    # second call: the array holds the first call's partials
    _run_both(V=4099, d=264, B=4, seed=300)     # other shape, several sequences, one of them inactive
    _run_both(V=50, d=16, B=2, seed=400)


def test_static_entry_point_rejects_what_does_not_fit():
    V, d, B = 1000, 64, binding.STATIC_MAX_BATCH + 1
    W = inputs.lm_head(V, d, seed=1).cuda()
    h = inputs.hidden(B, d, seed=2).cuda()
    clf = to_gpu_clf(make_clf(8, seed=3))
    z = torch.zeros(B, dtype=torch.int32, device="cuda")
    token, conf = torch.zeros_like(z), torch.zeros(B, device="cuda")
    halt = torch.zeros(B, dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.DiscoError) as e:
        binding.draft_step_static(W, h, z, z, clf, 0.5, 3, token, conf, halt)
    assert e.value.code == binding.ERR_STATIC_LIMIT
    assert "fixed scratch" in binding.strerror(binding.ERR_STATIC_LIMIT)
