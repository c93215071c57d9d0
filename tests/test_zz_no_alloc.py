"""disco_draft_step_static: the draft step for hosts that are not allowed to allocate device memory.

A serving process whose GPU memory belongs to another component, or a decode loop that cannot take the
device synchronisation of a cudaMalloc, cannot create a disco context (disco_create allocates).  The
static entry point keeps its scratch in a fixed array inside libdisco.so instead.  This test calls it
through the C ABI and checks it against the context-based entry point and against the CPU oracle on the
same inputs, twice in a row, because the second call finds the array as the first one left it; and it checks
that a call leaves the amount of free device memory as it found it.

The file name sorts last on purpose: a run that stops at the first failure has then already run every
other test.  The test does not depend on anything those tests leave behind.
"""
import numpy as np
import pytest
import torch

from paper_2405_04304_b200 import binding, inputs
from util import PROB_TOL, check_draft, make_clf, to_gpu_clf, to_oracle_clf

pytestmark = pytest.mark.gpu


def _run_both(oracle, V, d, B, seed, H=32):
    W_cpu = inputs.lm_head(V, d, seed=seed, std=0.2)
    h_cpu = inputs.hidden(B, d, seed=seed + 1)
    params = make_clf(H, seed=seed + 2)
    W, h, clf = W_cpu.cuda(), h_cpu.cuda(), to_gpu_clf(params)
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
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    binding.draft_step_static(W, h, pos, nd, clf, 0.5, 3, t1, c1, h1, active=active, feats=f1)
    torch.cuda.synchronize()
    if _run_both.calls > 0:      # from the second call on (the first also loads kernels): nothing is allocated
        assert torch.cuda.mem_get_info()[0] == free_before, "the allocation-free call changed the free device memory"
    _run_both.calls += 1
    assert ctx.device_status() == 0
    ctx.close()
    assert torch.equal(t0, t1), "tokens differ"
    assert torch.equal(h0, h1), "halt flags differ"
    np.testing.assert_allclose(c1.cpu().numpy(), c0.cpu().numpy(), rtol=0, atol=PROB_TOL)
    np.testing.assert_allclose(f1.cpu().numpy(), f0.cpu().numpy(), rtol=0, atol=PROB_TOL)
    if active is not None:                      # a skipped sequence keeps the caller's values
        assert int(t1[1]) == -7 and int(h1[1]) == 77
    # and against the CPU oracle, under the tolerances of the other parity tests
    act = None if active is None else active.cpu().numpy()
    ref = oracle.draft_step(inputs.bf16_bits(W_cpu), inputs.bf16_bits(h_cpu), pos.cpu().numpy(), nd.cpu().numpy(),
                            to_oracle_clf(oracle, params), 0.5, 3, active=act, nthreads=8)
    got = dict(token=t1.cpu().numpy(), conf=c1.cpu().numpy(), halt=h1.cpu().numpy(), feats=f1.cpu().numpy(), probs=None)
    check_draft(got, ref, 0.5, active=act)


_run_both.calls = 0


def test_static_entry_point_matches_context_entry_point_twice_in_a_row(oracle):
    _run_both(oracle, V=32000, d=768, B=1, seed=100)    # first call on the device also does the set-up
    _run_both(oracle, V=32000, d=768, B=1, seed=200)    # second call: the array holds the first call's partials
    _run_both(oracle, V=4099, d=264, B=4, seed=300)     # other shape, several sequences, one of them inactive
    _run_both(oracle, V=50, d=16, B=2, seed=400)


def test_static_entry_point_at_its_largest_grid(oracle):
    """DISCO_STATIC_MAX_GRID slabs of 2048 vocabulary rows: the most the fixed array has records for.  One row
    more needs another slab and is refused."""
    V, d = 2048 * 1024 - 5, 8
    _run_both(oracle, V=V, d=d, B=2, seed=500)
    V = 2048 * 1024 + 1
    W = torch.zeros((V, d), dtype=torch.bfloat16, device="cuda")
    h = inputs.hidden(1, d, seed=2).cuda()
    clf = to_gpu_clf(make_clf(8, seed=3))
    one = torch.ones(1, dtype=torch.int32, device="cuda")
    token, conf = torch.zeros_like(one), torch.zeros(1, device="cuda")
    halt = torch.zeros(1, dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.DiscoError) as e:
        binding.draft_step_static(W, h, one, one, clf, 0.5, 3, token, conf, halt)
    assert e.value.code == binding.ERR_STATIC_LIMIT


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
