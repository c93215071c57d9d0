"""Parity of the CUDA library (through its C ABI) with the CPU oracle, element by element on the same
seeded inputs.  Needs a B200: run with -m gpu."""
import numpy as np
import pytest
import torch

from paper_2405_04304_b200 import binding, inputs
import util
from util import (check_draft, check_verify, gpu_draft_step, gpu_verify, make_clf, near_tie_ids, to_gpu_clf,
                  to_oracle_clf, top2_ids)

pytestmark = pytest.mark.gpu


def _bits(t):
    return inputs.bf16_bits(t)


def _ctx(V, dD, dT, max_batch=8, max_rows=64, H=64):
    return binding.Context(V, dD, dT, max_batch=max_batch, max_rows=max_rows, clf_hidden=H)


# ---------------------------------------------------------------------------------- draft step
@pytest.mark.parametrize("V,d,B", [(1, 8, 1), (5, 8, 2), (9, 16, 1), (10, 16, 3), (11, 24, 1), (64, 64, 5),
                                   (217, 72, 2), (1000, 128, 4), (4099, 264, 7), (33, 8, 8)])
def test_draft_step_small_shapes(oracle, V, d, B):
    W = inputs.lm_head(V, d, seed=V + d, std=0.3)
    h = inputs.hidden(B, d, seed=V * 7 + B)
    params = make_clf(16, seed=V)
    pos = np.arange(1, B + 1, dtype=np.int32) * 3
    nd = (np.arange(B, dtype=np.int32) % 4) + 1
    ctx = _ctx(V, d, 8, max_batch=8, H=16)
    got = gpu_draft_step(ctx, W.cuda(), h, pos, nd, to_gpu_clf(params), 0.5, 3, want_probs=True)
    ref = oracle.draft_step(_bits(W), _bits(h), pos, nd, to_oracle_clf(oracle, params), 0.5, 3, want_probs=True)
    check_draft(got, ref, 0.5)
    assert ctx.device_status() == 0
    ctx.close()


@pytest.mark.parametrize("B", [1, 2, 3])
@pytest.mark.parametrize("path", [0, 1, 2, 3])
def test_every_small_vocabulary(oracle, path, B):
    """V = 1 .. 64 without a gap (fewer than ten logits, one CTA with rows and 147 without, ragged last tile), the
    narrowest hidden state, one to three sequences, both tails, on each kernel family."""
    d, SL = 8, 3
    params = make_clf(8, seed=5)
    clf_g, clf_o = to_gpu_clf(params), to_oracle_clf(oracle, params)
    pos, nd = np.array([4, 9, 2][:B], np.int32), np.array([1, 2, 3][:B], np.int32)
    for V in range(1, 65):
        W = inputs.lm_head(V, d, seed=1000 + V, std=0.3)
        h = inputs.hidden(B, d, seed=2000 + V)
        ctx = _ctx(V, d, d, max_batch=8, max_rows=64, H=8)
        ctx.set_kernel_path(path)
        got = gpu_draft_step(ctx, W.cuda(), h, pos, nd, clf_g, 0.5, 3, want_probs=True)
        ref = oracle.draft_step(_bits(W), _bits(h), pos, nd, clf_o, 0.5, 3, want_probs=True)
        check_draft(got, ref, 0.5)
        R = B * (SL + 1)
        H = inputs.hidden(R, d, seed=3000 + V)
        off = np.arange(B + 1, dtype=np.int32) * (SL + 1)
        free = oracle.verify_ragged(_bits(W), _bits(H), np.zeros(R - B, np.int32), off)
        clean = np.concatenate([free.target_ids[off[b]:off[b + 1] - 1] for b in range(B)]).astype(np.int32)
        draft = inputs.corrupt_ids(torch.from_numpy(clean), 0.3, V, seed=V).numpy()
        refv = oracle.verify_ragged(_bits(W), _bits(H), draft, off)
        gotv = gpu_verify(ctx, W.cuda(), H, draft, row_off=off)
        check_verify(gotv, refv, off, draft, near_tie_ids(oracle, _bits(W), _bits(H), refv.gap))
        assert ctx.device_status() == 0, f"V = {V}"
        ctx.close()


def test_draft_step_tiny_workload_shapes(oracle):
    wl = inputs.WORKLOADS["tiny"]
    W = inputs.lm_head(wl.V, wl.d_D, seed=inputs.sub_seed(wl.seed, 1))
    params = make_clf(wl.H, seed=inputs.sub_seed(wl.seed, 2))
    ctx = _ctx(wl.V, wl.d_D, wl.d_T, H=wl.H)
    Wg, clf_g, clf_o = W.cuda(), to_gpu_clf(params), to_oracle_clf(oracle, params)
    exempt = 0
    for step in range(6):
        h = inputs.hidden(1, wl.d_D, seed=inputs.sub_seed(wl.seed, 3, step))
        pos, nd = np.array([step + 1], np.int32), np.array([step % wl.sl_max + 1], np.int32)
        got = gpu_draft_step(ctx, Wg, h, pos, nd, clf_g, wl.tau, wl.sl_max, want_probs=(step == 0))
        ref = oracle.draft_step(_bits(W), _bits(h), pos, nd, clf_o, wl.tau, wl.sl_max, want_probs=(step == 0),
                                nthreads=8)
        exempt += check_draft(got, ref, wl.tau)
    assert exempt <= 1
    assert ctx.device_status() == 0
    ctx.close()


@pytest.mark.parametrize("name", ["vicuna_b1", "starcoder_b1"])
def test_draft_step_full_size_heads(oracle, name):
    wl = inputs.WORKLOADS[name]
    W = inputs.lm_head(wl.V, wl.d_D, seed=inputs.sub_seed(wl.seed, 1))
    params = make_clf(wl.H, seed=inputs.sub_seed(wl.seed, 2))
    ctx = _ctx(wl.V, wl.d_D, wl.d_T, H=wl.H)
    for B in (1, 3):
        h = inputs.hidden(B, wl.d_D, seed=inputs.sub_seed(wl.seed, 3, B))
        pos, nd = np.arange(10, 10 + B, dtype=np.int32), np.ones(B, np.int32)
        got = gpu_draft_step(ctx, W.cuda(), h, pos, nd, to_gpu_clf(params), wl.tau, wl.sl_max)
        ref = oracle.draft_step(_bits(W), _bits(h), pos, nd, to_oracle_clf(oracle, params), wl.tau, wl.sl_max,
                                nthreads=8)
        check_draft(got, ref, wl.tau)
    assert ctx.device_status() == 0
    ctx.close()


def test_draft_step_closed_forms(oracle):
    V, d = 3000, 64
    W = inputs.lm_head(V, d, seed=5, std=0.1)
    params = make_clf(8, seed=6)
    ctx = _ctx(V, d, 8, H=8)
    # zero hidden state: uniform distribution, entropy ln V, token 0 (lowest index among equals)
    h = torch.zeros(1, d, dtype=torch.bfloat16)
    got = gpu_draft_step(ctx, W.cuda(), h, [4], [1], to_gpu_clf(params), 0.5, 5, want_probs=True)
    assert got["token"][0] == 0
    np.testing.assert_allclose(got["probs"][0], 1.0 / V, rtol=1e-5)
    np.testing.assert_allclose(got["feats"][0, :10], 1.0 / V, rtol=1e-5)
    assert abs(got["feats"][0, 10] - np.log(V)) < 1e-4
    # planted peak: hidden state aligned with one row
    h = (W[1234].float() * 300.0).to(torch.bfloat16).view(1, d)
    got = gpu_draft_step(ctx, W.cuda(), h, [4], [1], to_gpu_clf(params), 0.5, 5)
    ref = oracle.draft_step(_bits(W), _bits(h), [4], [1], to_oracle_clf(oracle, params), 0.5, 5)
    assert got["token"][0] == 1234 == ref.token[0]
    check_draft(got, ref, 0.5)
    assert got["feats"][0, 0] > 0.99
    ctx.close()


def test_threshold_rule_and_cap(oracle):
    V, d, B = 500, 32, 4
    W = inputs.lm_head(V, d, seed=8, std=0.2)
    h = inputs.hidden(B, d, seed=9)
    params = make_clf(8, seed=10)
    flat = make_clf(8, seed=10, zero_head=True)
    ctx = _ctx(V, d, 8, H=8)
    Wg = W.cuda()
    pos = np.arange(1, B + 1, dtype=np.int32)
    for nd, expect in ((1, 0), (4, 0), (5, 1), (7, 1)):      # tau <= 0: static SL = SL_max
        got = gpu_draft_step(ctx, Wg, h, pos, np.full(B, nd, np.int32), to_gpu_clf(params), 0.0, 5)
        assert list(got["halt"]) == [expect] * B
    got = gpu_draft_step(ctx, Wg, h, pos, np.ones(B, np.int32), to_gpu_clf(params), 1.5, 5)
    assert list(got["halt"]) == [1] * B                      # tau > 1: SL = 1
    got = gpu_draft_step(ctx, Wg, h, pos, np.ones(B, np.int32), to_gpu_clf(flat), 0.5, 5)
    assert list(got["conf"]) == [0.5] * B and list(got["halt"]) == [0] * B   # C == tau continues
    got = gpu_draft_step(ctx, Wg, h, pos, np.ones(B, np.int32), to_gpu_clf(flat), 0.5000001, 5)
    assert list(got["halt"]) == [1] * B
    halts = [gpu_draft_step(ctx, Wg, h, pos, np.ones(B, np.int32), to_gpu_clf(params), tau, 9)["halt"]
             for tau in (0.3, 0.5, 0.7)]
    assert np.all(halts[0] <= halts[1]) and np.all(halts[1] <= halts[2])
    ctx.close()


def test_inactive_sequences_are_not_written(oracle):
    V, d, B = 700, 40, 5
    W = inputs.lm_head(V, d, seed=11, std=0.2)
    h = inputs.hidden(B, d, seed=12)
    params = make_clf(8, seed=13)
    active = np.array([1, 0, 1, 0, 1], np.uint8)
    pos, nd = np.arange(B, dtype=np.int32) + 2, np.ones(B, np.int32)
    ctx = _ctx(V, d, 8, H=8)
    ref = oracle.draft_step(_bits(W), _bits(h), pos, nd, to_oracle_clf(oracle, params), 0.5, 5, active=active)
    for host in (False, True):
        got = gpu_draft_step(ctx, W.cuda(), h, pos, nd, to_gpu_clf(params), 0.5, 5, active=active, host=host)
        check_draft(got, ref, 0.5, active=active)
    ctx.close()


def test_draft_step_is_deterministic_and_host_variant_matches():
    V, d, B = 32000, 768, 2
    W = inputs.lm_head(V, d, seed=14).cuda()
    h = inputs.hidden(B, d, seed=15)
    clf = to_gpu_clf(make_clf(64, seed=16))
    ctx = _ctx(V, d, 8)
    a = gpu_draft_step(ctx, W, h, [1, 2], [1, 1], clf, 0.5, 5)
    b = gpu_draft_step(ctx, W, h, [1, 2], [1, 1], clf, 0.5, 5)
    c = gpu_draft_step(ctx, W, h, [1, 2], [1, 1], clf, 0.5, 5, host=True)
    for k in ("token", "conf", "halt", "feats"):
        np.testing.assert_array_equal(a[k], b[k])
        np.testing.assert_array_equal(a[k], c[k])
    ctx.close()


# ---------------------------------------------------------------------------------- verification
@pytest.mark.parametrize("V,d,sls", [(1, 8, [0]), (7, 8, [2]), (64, 16, [5]), (64, 16, [3, 0, 5, 1]),
                                     (1000, 136, [10]), (4099, 72, [1, 2, 3, 4, 5, 6]), (300, 64, [40, 33, 0])])
def test_verify_small_shapes(oracle, V, d, sls):
    sl = torch.tensor(sls, dtype=torch.int32)
    off = inputs.row_offsets(sl).numpy()
    R, B = int(off[-1]), len(sls)
    W = inputs.lm_head(V, d, seed=V + d, std=0.3)
    H = inputs.hidden(R, d, seed=V + R)
    free = oracle.verify_ragged(_bits(W), _bits(H), np.zeros(R - B, np.int32), off)   # target ids only
    clean = np.concatenate([free.target_ids[off[b]:off[b + 1] - 1] for b in range(B)]).astype(np.int32)
    draft = inputs.corrupt_ids(torch.from_numpy(clean), 0.25, V, seed=R).numpy()
    ref = oracle.verify_ragged(_bits(W), _bits(H), draft, off)
    ctx = binding.Context(V, 8, d, max_batch=8, max_rows=128)
    got = gpu_verify(ctx, W.cuda(), H, draft, row_off=off)
    check_verify(got, ref, off, draft, near_tie_ids(oracle, _bits(W), _bits(H), ref.gap))
    got_h = gpu_verify(ctx, W.cuda(), H, draft, row_off=off, host=True)
    for k in ("n_accept", "bonus", "target_ids"):
        np.testing.assert_array_equal(got[k], got_h[k])
    if len(set(sls)) == 1:                                    # uniform entry point == ragged entry point
        got_u = gpu_verify(ctx, W.cuda(), H, draft, B=B, SL=sls[0])
        for k in ("n_accept", "bonus", "target_ids"):
            np.testing.assert_array_equal(got[k], got_u[k])
    assert ctx.device_status() == 0
    ctx.close()


def test_verify_fig1_and_special_cases(oracle):
    V, d, SL = 2000, 64, 5
    W = inputs.lm_head(V, d, seed=21, std=0.3)
    H = inputs.hidden(SL + 1, d, seed=22)
    a = oracle.verify(_bits(W), _bits(H), np.zeros(SL, np.int32), 1, SL).target_ids
    ctx = binding.Context(V, 8, d, max_batch=2, max_rows=16)
    Wg = W.cuda()
    got = gpu_verify(ctx, Wg, H, a[:SL], B=1, SL=SL)               # draft == target: all accepted
    assert got["n_accept"][0] == SL and got["bonus"][0] == a[SL]
    fig1 = a[:SL].copy()
    fig1[3] = (fig1[3] + 1) % V                                     # Fig. 1: t4 and t5 rejected
    fig1[4] = (fig1[4] + 1) % V
    got = gpu_verify(ctx, Wg, H, fig1, B=1, SL=SL)
    assert got["n_accept"][0] == 3 and got["bonus"][0] == a[3]
    hole = a[:SL].copy()
    hole[0] = (hole[0] + 1) % V                                     # first wrong: later matches do not count
    got = gpu_verify(ctx, Wg, H, hole, B=1, SL=SL)
    assert got["n_accept"][0] == 0 and got["bonus"][0] == a[0]
    got = gpu_verify(ctx, Wg, H[:1], np.zeros(0, np.int32), B=1, SL=0)   # SL = 0: plain target step
    assert got["n_accept"][0] == 0 and got["bonus"][0] == a[0]
    ctx.close()


@pytest.mark.parametrize("name,SL", [("tiny", 5), ("vicuna_b1", 10), ("starcoder_b1", 10)])
def test_verify_full_size_heads(oracle, name, SL):
    wl = inputs.WORKLOADS[name]
    W = inputs.lm_head(wl.V, wl.d_T, seed=inputs.sub_seed(wl.seed, 4))
    H = inputs.hidden(SL + 1, wl.d_T, seed=inputs.sub_seed(wl.seed, 5))
    free = oracle.verify(_bits(W), _bits(H), np.zeros(SL, np.int32), 1, SL, nthreads=8)
    draft = inputs.corrupt_ids(torch.from_numpy(free.target_ids[:SL].copy()), wl.p_corrupt, wl.V,
                               seed=inputs.sub_seed(wl.seed, 6)).numpy()
    ref_n, ref_bonus = oracle.accept_prefix(draft, free.target_ids)
    ctx = binding.Context(wl.V, wl.d_D, wl.d_T, max_batch=1, max_rows=SL + 1)
    got = gpu_verify(ctx, W.cuda(), H, draft, B=1, SL=SL)
    ref = oracle.VerifyResult(np.array([ref_n], np.int32), np.array([ref_bonus], np.int32), free.target_ids,
                              free.gap)
    check_verify(got, ref, [0, SL + 1], draft, near_tie_ids(oracle, _bits(W), _bits(H), ref.gap))
    assert ctx.device_status() == 0
    ctx.close()


@pytest.mark.parametrize("d_T", [5120, 6144])
@pytest.mark.parametrize("path", [0, 1])
def test_plain_target_step_at_full_width(oracle, d_T, path):
    """SL = 0 (one row per sequence: n = 0, bonus = the target's token) at the two target widths of the paper's
    model pairs.  A single row goes to the CUDA-core streaming kernel; path 1 forces that kernel for the
    three-sequence case too.  The 6144-wide rows make its ring shallower than its warp count."""
    V = 3001
    W = inputs.lm_head(V, d_T, seed=d_T + 1, std=0.05)
    ctx = binding.Context(V, 768, d_T, max_batch=4, max_rows=16)
    ctx.set_kernel_path(path)
    for B in (1, 3):
        H = inputs.hidden(B, d_T, seed=d_T + 7 * B)
        off = np.arange(B + 1, dtype=np.int32)
        ref = oracle.verify_ragged(_bits(W), _bits(H), np.zeros(0, np.int32), off, nthreads=8)
        got = gpu_verify(ctx, W.cuda(), H, np.zeros(0, np.int32), row_off=off)
        check_verify(got, ref, off, np.zeros(0, np.int32), near_tie_ids(oracle, _bits(W), _bits(H), ref.gap))
        assert np.all(got["n_accept"] == 0)
    assert ctx.device_status() == 0
    ctx.close()


@pytest.mark.parametrize("B,sls", [(1, [10]), (2, [3, 4])])
def test_streaming_kernel_at_the_widest_hidden_size(oracle, B, sls):
    """Path 1 (CUDA-core streaming kernel) with 6144-wide hidden rows, draft step and verification: rows of
    12 KB leave the ring fewer slots than the kernel has consumer warps, so some warps own no slot."""
    V, d = 2500, 6144
    W = inputs.lm_head(V, d, seed=61, std=0.05)
    params = make_clf(16, seed=62)
    ctx = binding.Context(V, d, d, max_batch=4, max_rows=32, clf_hidden=16)
    ctx.set_kernel_path(1)
    h = inputs.hidden(B, d, seed=63 + B)
    pos, nd = np.arange(1, B + 1, dtype=np.int32), np.ones(B, np.int32)
    got = gpu_draft_step(ctx, W.cuda(), h, pos, nd, to_gpu_clf(params), 0.5, 4, want_probs=True)
    ref = oracle.draft_step(_bits(W), _bits(h), pos, nd, to_oracle_clf(oracle, params), 0.5, 4, want_probs=True,
                            nthreads=8)
    check_draft(got, ref, 0.5)
    off = inputs.row_offsets(torch.tensor(sls, dtype=torch.int32)).numpy()
    R = int(off[-1])
    H = inputs.hidden(R, d, seed=70 + B)
    free = oracle.verify_ragged(_bits(W), _bits(H), np.zeros(R - B, np.int32), off, nthreads=8)
    clean = np.concatenate([free.target_ids[off[b]:off[b + 1] - 1] for b in range(B)]).astype(np.int32)
    draft = inputs.corrupt_ids(torch.from_numpy(clean), 0.2, V, seed=R).numpy()
    ref = oracle.verify_ragged(_bits(W), _bits(H), draft, off, nthreads=8)
    got = gpu_verify(ctx, W.cuda(), H, draft, row_off=off)
    check_verify(got, ref, off, draft, near_tie_ids(oracle, _bits(W), _bits(H), ref.gap))
    assert ctx.device_status() == 0
    ctx.close()


# ---------------------------------------------------------------------------------- error handling
def test_errors_are_codes_not_faults():
    V, d = 100, 16
    ctx = binding.Context(V, d, d, max_batch=3, max_rows=8, clf_hidden=8)
    W = inputs.lm_head(V, d, seed=1).cuda()
    clf = to_gpu_clf(make_clf(8, seed=2))
    h3 = inputs.hidden(4, d, seed=3)
    with pytest.raises(binding.DiscoError) as e:
        gpu_draft_step(ctx, W, h3, [1, 2, 3, 4], [1, 1, 1, 1], clf, 0.5, 5)
    assert e.value.code == binding.ERR_WORKSPACE
    big = to_gpu_clf(make_clf(16, seed=2))
    with pytest.raises(binding.DiscoError) as e:
        gpu_draft_step(ctx, W, h3[:1], [1], [1], big, 0.5, 5)
    assert e.value.code == binding.ERR_WORKSPACE
    with pytest.raises(binding.DiscoError) as e:
        gpu_verify(ctx, W, inputs.hidden(9, d, seed=4), np.zeros(8, np.int32), B=1, SL=8)
    assert e.value.code == binding.ERR_WORKSPACE
    with pytest.raises(binding.DiscoError) as e:                     # misaligned LM head
        gpu_draft_step(ctx, W.view(-1)[4:4 + 50 * d].view(50, d), h3[:1], [1], [1], clf, 0.5, 5)
    assert e.value.code == binding.ERR_INVALID_ARG
    # inconsistent row offsets are caught by the kernel: status word + -1 outputs, no fault
    H = inputs.hidden(6, d, seed=5)
    got = gpu_verify(ctx, W, H, np.zeros(4, np.int32), row_off=[0, 4, 7])
    assert got["n_accept"][1] == -1 and got["bonus"][1] == -1
    assert ctx.device_status() == binding.ERR_INVALID_ARG
    assert ctx.device_status() == 0
    # offsets that rise locally but would put a sequence's draft ids outside the id array
    H7 = inputs.hidden(7, d, seed=6)
    got = gpu_verify(ctx, W, H7, np.zeros(4, np.int32), row_off=[0, 5, 1, 7])
    assert got["n_accept"][1] == -1 and got["n_accept"][2] == -1
    assert ctx.device_status() == binding.ERR_INVALID_ARG
    got = gpu_verify(ctx, W, H7, np.zeros(4, np.int32), row_off=[0, 6, 7, 7])
    assert got["n_accept"][0] == -1 and got["n_accept"][2] == -1
    assert ctx.device_status() == binding.ERR_INVALID_ARG
    # the context still works afterwards
    got = gpu_verify(ctx, W, H, np.zeros(4, np.int32), row_off=[0, 4, 6])
    assert np.all(got["n_accept"] >= 0)
    ctx.close()


# ---------------------------------------------------------------------------------- both kernel families
@pytest.mark.parametrize("path", [1, 2, 3])
@pytest.mark.parametrize("V,d,B", [(50, 16, 1), (1000, 72, 3), (4099, 264, 7), (32000, 768, 1), (20011, 320, 16),
                                   (5000, 768, 64), (3000, 128, 130)])
def test_draft_step_on_each_kernel_path(oracle, path, V, d, B):
    if path == 1 and B > 16:
        pytest.skip("the CUDA-core kernel is only meant for a handful of rows")
    if path == 3 and B > 16:
        pytest.skip("the vocabulary-on-lanes kernel takes at most 16 sequences")
    W = inputs.lm_head(V, d, seed=3 * V + d, std=0.2)
    h = inputs.hidden(B, d, seed=V + 11 * B)
    params = make_clf(32, seed=B)
    pos = (np.arange(B, dtype=np.int32) * 7) % 50 + 1
    nd = (np.arange(B, dtype=np.int32) % 5) + 1
    active = None if B < 5 else (np.arange(B) % 3 != 1).astype(np.uint8)
    ctx = _ctx(V, d, 8, max_batch=B, H=32)
    ctx.set_kernel_path(path)
    got = gpu_draft_step(ctx, W.cuda(), h, pos, nd, to_gpu_clf(params), 0.5, 4, active=active,
                         want_probs=(B <= 7))
    ref = oracle.draft_step(_bits(W), _bits(h), pos, nd, to_oracle_clf(oracle, params), 0.5, 4, active=active,
                            want_probs=(B <= 7), nthreads=8)
    check_draft(got, ref, 0.5, active=active)
    assert ctx.device_status() == 0
    ctx.close()


@pytest.mark.parametrize("path", [1, 2])
@pytest.mark.parametrize("V,d,sls", [(7, 8, [0]), (64, 16, [5]), (1000, 136, [10]), (4099, 72, [1, 2, 3, 4, 5, 6]),
                                     (2000, 5120, [10]), (3000, 128, [16] * 9 + [3, 0, 7]), (600, 64, [9] * 40)])
def test_verify_on_each_kernel_path(oracle, path, V, d, sls):
    sl = torch.tensor(sls, dtype=torch.int32)
    off = inputs.row_offsets(sl).numpy()
    R, B = int(off[-1]), len(sls)
    if path == 1 and R > 64:
        pytest.skip("the CUDA-core kernel is only meant for a handful of rows")
    W = inputs.lm_head(V, d, seed=V + 2 * d, std=0.3)
    H = inputs.hidden(R, d, seed=V + 3 * R)
    free = oracle.verify_ragged(_bits(W), _bits(H), np.zeros(R - B, np.int32), off, nthreads=8)
    clean = np.concatenate([free.target_ids[off[b]:off[b + 1] - 1] for b in range(B)]).astype(np.int32)
    draft = inputs.corrupt_ids(torch.from_numpy(clean), 0.2, V, seed=R).numpy()
    n_b = [oracle.accept_prefix(draft[off[b] - b: off[b + 1] - b - 1], free.target_ids[off[b]:off[b + 1]])
           for b in range(B)]
    ref = oracle.VerifyResult(np.array([x[0] for x in n_b], np.int32), np.array([x[1] for x in n_b], np.int32),
                              free.target_ids, free.gap)
    ctx = binding.Context(V, 8, d, max_batch=B, max_rows=R)
    ctx.set_kernel_path(path)
    got = gpu_verify(ctx, W.cuda(), H, draft, row_off=off)
    check_verify(got, ref, off, draft, near_tie_ids(oracle, _bits(W), _bits(H), free.gap))
    got2 = gpu_verify(ctx, W.cuda(), H, draft, row_off=off)          # scratch is clean for the next call
    for k in ("n_accept", "bonus", "target_ids"):
        np.testing.assert_array_equal(got[k], got2[k])
    assert ctx.device_status() == 0
    ctx.close()


# ---------------------------------------------------------------------------------- full-size batched workloads
def _prefix_rule(draft, target_rows):
    n = 0
    while n < len(draft) and draft[n] == target_rows[n]:
        n += 1
    return n, target_rows[n]


def _stratified_rows(R, per_tile, rng):
    """A sample of hidden rows that hits every 128-row tile of the tensor-core kernel: the first and the last
    row of each tile plus per_tile - 2 random ones."""
    rows = []
    for t0 in range(0, R, 128):
        t1 = min(R, t0 + 128)
        pick = {t0, t1 - 1}
        extra = rng.choice(np.arange(t0, t1), size=min(max(per_tile - 2, 0), t1 - t0), replace=False)
        pick.update(int(x) for x in extra)
        rows.extend(sorted(pick))
    return np.array(sorted(set(rows)), dtype=np.int64)


@pytest.mark.parametrize("name,per_tile", [("vicuna_b64", 24), ("starcoder_b256", 4)])
def test_batched_verification_at_full_size(oracle, name, per_tile):
    """The launch configuration bench.py times (ragged rows over the whole LM head).  The oracle projects a
    stratified sample of rows one by one (every 128-row tile of hidden rows, both of its ends); two of the
    sampled rows are made to win in the first and in the last vocabulary tile; every sequence is checked
    against the prefix rule applied to the ids the library itself reported."""
    wl = inputs.WORKLOADS[name]
    B, S = wl.B, wl.sl_max
    if wl.sl_mode == "uniform":
        sl = inputs.uniform_sl(B, 1, S, inputs.sub_seed(wl.seed, 8))
    else:
        sl = torch.full((B,), S, dtype=torch.int32)
    off = inputs.row_offsets(sl).numpy()
    R = int(off[-1])
    W = inputs.lm_head(wl.V, wl.d_T, seed=inputs.sub_seed(wl.seed, 2))
    H = inputs.hidden(R, wl.d_T, seed=inputs.sub_seed(wl.seed, 5))
    rng = np.random.default_rng(wl.seed)
    draft = rng.integers(0, wl.V, size=R - B).astype(np.int32)
    rows = _stratified_rows(R, per_tile, rng)
    # two sampled rows point along the first and the last row of the LM head: their arg-max lies in the first
    # and in the last vocabulary tile
    H[int(rows[1])] = (W[0].float() * 200.0).to(torch.bfloat16)
    H[int(rows[-2])] = (W[wl.V - 1].float() * 200.0).to(torch.bfloat16)
    z = oracle.project(_bits(W), _bits(H[torch.from_numpy(rows)]), nthreads=16)
    want = [oracle.argmax(z[i]) for i in range(len(rows))]
    assert want[1][0] == 0 and want[-2][0] == wl.V - 1
    # make some sampled rows "accepted": the draft id at that position equals the oracle's target id
    row_seq = np.searchsorted(off, rows, side="right") - 1
    for (r, b), (tok, gap) in zip(zip(rows, row_seq), want):
        j = r - off[b]
        if j < sl[b]:
            draft[off[b] - b + j] = tok
    ctx = binding.Context(wl.V, wl.d_D, wl.d_T, max_batch=B, max_rows=R)
    Wg = W.cuda()
    got = gpu_verify(ctx, Wg, H, draft, row_off=off)
    assert ctx.device_status() == 0
    tid = got["target_ids"]
    exempt = 0
    for i, (r, (tok, gap)) in enumerate(zip(rows, want)):
        if gap < 1e-3:          # a near tie may return the best id or the runner-up, nothing else
            exempt += 1
            util.COUNTS["verify_rows_near_tie"] += 1
            assert tid[r] in np.argsort(-z[i], kind="stable")[:2], f"row {r}: id {tid[r]} is neither of the tied top-2"
            continue
        assert tid[r] == tok, f"row {r}: target id {tid[r]} != oracle {tok}"
    assert exempt <= max(3, len(rows) // 25)     # expected about 0.5 % of the rows (gap of the largest of V Gaussians)
    assert np.all((tid >= 0) & (tid < wl.V))
    for b in range(B):
        n, bonus = _prefix_rule(draft[off[b] - b: off[b + 1] - b - 1], tid[off[b]:off[b + 1]])
        assert got["n_accept"][b] == n and got["bonus"][b] == bonus
    got2 = gpu_verify(ctx, Wg, H, draft, row_off=off)            # deterministic, scratch left clean
    for k in ("n_accept", "bonus", "target_ids"):
        np.testing.assert_array_equal(got[k], got2[k])
    ctx.close()


@pytest.mark.parametrize("name", ["vicuna_b64", "starcoder_b256"])
def test_batched_draft_step_at_full_size(oracle, name):
    wl = inputs.WORKLOADS[name]
    B = wl.B
    W = inputs.lm_head(wl.V, wl.d_D, seed=inputs.sub_seed(wl.seed, 1))
    h = inputs.hidden(B, wl.d_D, seed=inputs.sub_seed(wl.seed, 4))
    params = make_clf(wl.H, seed=inputs.sub_seed(wl.seed, 3))
    pos = (np.arange(B, dtype=np.int32) * 13) % 97 + 1
    nd = (np.arange(B, dtype=np.int32) % wl.sl_max) + 1
    active = (np.arange(B) % 5 != 2).astype(np.uint8)
    ctx = _ctx(wl.V, wl.d_D, wl.d_T, max_batch=B, H=wl.H)
    got = gpu_draft_step(ctx, W.cuda(), h, pos, nd, to_gpu_clf(params), wl.tau, wl.sl_max, active=active)
    ref = oracle.draft_step(_bits(W), _bits(h), pos, nd, to_oracle_clf(oracle, params), wl.tau, wl.sl_max,
                            active=active, nthreads=16)
    exempt = check_draft(got, ref, wl.tau, active=active)
    assert exempt <= max(2, B // 50)
    assert ctx.device_status() == 0
    ctx.close()


# ---------------------------------------------------------------------------------- perplexity stopping rule
@pytest.mark.parametrize("path", [0, 1, 2, 3])
@pytest.mark.parametrize("V,d,B", [(700, 40, 1), (4099, 264, 5), (32000, 768, 1), (5000, 128, 40)])
def test_draft_step_with_perplexity_rule(oracle, path, V, d, B):
    if (path == 1 or path == 3) and B > 16:
        pytest.skip("kernel family not meant for this many sequences")
    W = inputs.lm_head(V, d, seed=V + d, std=0.3)
    ctx = _ctx(V, d, 8, max_batch=B)
    ctx.set_kernel_path(path)
    Wg = W.cuda()
    active = None if B < 3 else (np.arange(B) % 4 != 1).astype(np.uint8)
    nll_ref = np.zeros(B)
    nll_gpu = torch.zeros(B, dtype=torch.float32, device="cuda")
    bound = float(np.exp(0.6 * np.log(V)))
    for n in (1, 2, 3):                                        # three consecutive draft steps of one iteration
        h = inputs.hidden(B, d, seed=V + 17 * n)
        nd = np.full(B, n, np.int32)
        tok_r, ppl_r, halt_r, gap_r, nll_ref = oracle.draft_step_ppl(_bits(W), _bits(h), nd, nll_ref, bound, 3,
                                                                       active=active, nthreads=8)
        token = torch.full((B,), -7, dtype=torch.int32, device="cuda")
        ppl = torch.full((B,), -7.0, dtype=torch.float32, device="cuda")
        halt = torch.full((B,), 77, dtype=torch.uint8, device="cuda")
        ctx.draft_step_ppl(Wg, h.cuda(), torch.from_numpy(nd).cuda(), nll_gpu, bound, 3, token, ppl, halt,
                           active=None if active is None else torch.from_numpy(active).cuda())
        torch.cuda.synchronize()
        token, ppl, halt = token.cpu().numpy(), ppl.cpu().numpy(), halt.cpu().numpy()
        for b in range(B):
            if active is not None and not active[b]:
                assert token[b] == -7 and halt[b] == 77 and ppl[b] == -7.0
                continue
            if gap_r[b] >= 1e-3:
                assert token[b] == tok_r[b]
            assert abs(ppl[b] - ppl_r[b]) <= 2e-3 * ppl_r[b]   # relative: a perplexity is not bounded by 1
            if abs(ppl_r[b] - bound) > 2e-3 * bound:
                assert halt[b] == halt_r[b]
        np.testing.assert_allclose(nll_gpu.cpu().numpy(), nll_ref, rtol=1e-4, atol=1e-4)
    assert ctx.device_status() == 0
    ctx.close()


# ---------------------------------------------------------------------------------- sampling at temperature 1
CDF_TOL = 2e-5      # slack on a running sum of fp32 probabilities against the fp64 ones
RATIO_TOL = 1e-4    # an acceptance test whose two sides are closer than this (relative) may go either way


def _valid_draw(weights, u, tok, tol=CDF_TOL):
    """Is tok an inverse-CDF draw from the (fp64) weights for u, up to tol of the total on the running sums?"""
    cdf = np.cumsum(np.asarray(weights, dtype=np.float64))
    target = float(u) * cdf[-1]
    slack = tol * cdf[-1]
    if tok < 0 or tok >= len(cdf) or weights[tok] <= 0:
        return False
    return cdf[tok] > target - slack and (tok == 0 or cdf[tok - 1] <= target + slack)


@pytest.mark.parametrize("path", [0, 1, 2, 3])
@pytest.mark.parametrize("V,d,B", [(11, 8, 2), (1000, 72, 5), (4099, 264, 7), (32000, 768, 1), (5000, 128, 40)])
def test_draft_step_sample(oracle, path, V, d, B):
    if path == 3 and B > 16:
        pytest.skip("the kernel with the vocabulary on the TMEM lanes takes up to 16 sequences")
    W = inputs.lm_head(V, d, seed=V + 2 * d, std=0.25)
    h = inputs.hidden(B, d, seed=V * 5 + B)
    params = make_clf(32, seed=V + 3)
    pos = np.arange(1, B + 1, dtype=np.int32) * 2
    nd = (np.arange(B, dtype=np.int32) % 5) + 1
    g = torch.Generator().manual_seed(V + B)
    u = torch.rand(B, generator=g, dtype=torch.float32)
    u[0] = 0.0
    if B > 1:
        u[1] = float(np.nextafter(np.float32(1.0), np.float32(0.0)))
    active = np.ones(B, dtype=np.uint8)
    if B > 2:
        active[2] = 0
    ctx = _ctx(V, d, 8, max_batch=max(8, B), H=32)
    ctx.set_kernel_path(path)
    token = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    p_tok = torch.full((B,), -7.0, dtype=torch.float32, device="cuda")
    conf = torch.full((B,), -7.0, dtype=torch.float32, device="cuda")
    halt = torch.full((B,), 77, dtype=torch.uint8, device="cuda")
    feats = torch.full((B, binding.NFEAT), -7.0, dtype=torch.float32, device="cuda")
    probs = torch.full((B, V), -7.0, dtype=torch.float32, device="cuda")
    ctx.draft_step_sample(W.cuda(), h.cuda(), torch.from_numpy(pos).cuda(), torch.from_numpy(nd).cuda(),
                          to_gpu_clf(params), 0.5, 4, u.cuda(), token, conf, halt, probs, p_token=p_tok,
                          active=torch.from_numpy(active).cuda(), feats=feats)
    torch.cuda.synchronize()
    ref = oracle.draft_step_sample(_bits(W), _bits(h), pos, nd, to_oracle_clf(oracle, params), 0.5, 4,
                                   u.numpy().astype(np.float64), active=active)
    got = dict(token=token.cpu().numpy(), conf=conf.cpu().numpy(), halt=halt.cpu().numpy(),
               feats=feats.cpu().numpy(), probs=probs.cpu().numpy())
    pt = p_tok.cpu().numpy()
    for b in range(B):
        if not active[b]:
            assert got["token"][b] == -7 and pt[b] == -7.0 and got["halt"][b] == 77
            assert np.all(got["probs"][b] == -7.0), "the probs row of a masked sequence was written"
            continue
        np.testing.assert_allclose(got["probs"][b], ref.probs[b], rtol=0, atol=2e-3)
        np.testing.assert_allclose(got["feats"][b], ref.feats[b], rtol=0, atol=2e-3)
        assert abs(float(got["conf"][b]) - ref.conf[b]) <= 2e-3
        if abs(ref.conf[b] - 0.5) >= 1e-4:
            assert got["halt"][b] == ref.halt[b]
        tok = int(got["token"][b])
        assert tok == ref.token[b] or _valid_draw(ref.probs[b], float(u[b]), tok), f"seq {b}: token {tok}"
        assert abs(pt[b] - ref.probs[b, tok]) <= 2e-3
    assert int(got["token"][0]) == int(ref.token[0])            # u = 0: the first token with mass
    assert ctx.device_status() == 0
    ctx.close()


def _verify_sample_case(oracle, V, d, sls, seed, path=0, uniform=False, noise=0.6):
    B = len(sls)
    row_off = np.concatenate([[0], np.cumsum([s + 1 for s in sls])]).astype(np.int32)
    R = int(row_off[-1])
    W = inputs.lm_head(V, d, seed=seed, std=0.25)
    H = inputs.hidden(R, d, seed=seed + 1)
    rng = np.random.default_rng(seed)
    steps = max(max(sls), 1)
    # draft distributions near the target's (so that a good share of the tokens is accepted): soft-max of
    # the oracle's target logits plus noise, in binary32; tokens drawn from them
    z = oracle.project(_bits(W), _bits(H), nthreads=8)
    dp = np.zeros((steps, B, V), dtype=np.float32)
    ids = np.zeros(R - B, dtype=np.int32)
    for b in range(B):
        for i in range(sls[b]):
            zz = z[row_off[b] + i] + noise * rng.normal(size=V)
            e = np.exp(zz - zz.max())
            dp[i, b] = (e / e.sum()).astype(np.float32)
            ids[row_off[b] - b + i] = rng.choice(V, p=dp[i, b].astype(np.float64) / dp[i, b].astype(np.float64).sum())
    ua = rng.random(R - B).astype(np.float32)
    us = rng.random(B).astype(np.float32)
    ctx = _ctx(V, 8, d, max_batch=max(8, B), max_rows=max(64, R))
    ctx.set_kernel_path(path)
    n_acc = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    nxt = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    yT = torch.full((R, V), -7.0, dtype=torch.float32, device="cuda")
    tids = torch.full((R,), -7, dtype=torch.int32, device="cuda")
    ctx.verify_sample_ragged(W.cuda(), H.cuda(), torch.from_numpy(ids).cuda() if R > B else None,
                             torch.from_numpy(dp).cuda() if R > B else None,
                             None if uniform else torch.from_numpy(row_off).cuda(), B, R,
                             torch.from_numpy(ua).cuda() if R > B else None, torch.from_numpy(us).cuda(),
                             n_acc, nxt, yT, target_ids=tids)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    ctx.close()
    ref = oracle.verify_sample(_bits(W), _bits(H), ids, dp, row_off, ua.astype(np.float64), us.astype(np.float64),
                               nthreads=8)
    n_g, x_g, y_g = n_acc.cpu().numpy(), nxt.cpu().numpy(), yT.cpu().numpy()
    np.testing.assert_allclose(y_g, ref.y_T, rtol=0, atol=2e-3)
    np.testing.assert_allclose(y_g.astype(np.float64).sum(axis=1), 1.0, atol=1e-4)
    order = np.argsort(-z, axis=1, kind="stable")[:, :2]
    tg = tids.cpu().numpy()
    for r in range(R):
        tied = V > 1 and z[r, order[r, 0]] - z[r, order[r, -1]] < 1e-3
        assert tg[r] == order[r, 0] or (tied and tg[r] == order[r, -1]), f"row {r}: arg-max id {tg[r]}"

    accepted_total = 0
    for b in range(B):
        r0, sl = int(row_off[b]), sls[b]
        n_o = int(ref.n_accept[b])
        # acceptance tests that are decided by less than RATIO_TOL may go either way
        close = []
        for i in range(sl):
            t = ids[r0 - b + i]
            pT, pD = ref.y_T[r0 + i, t], float(dp[i, b, t])
            close.append(abs(float(ua[r0 - b + i]) * pD - pT) <= RATIO_TOL * max(pT, 1e-30))
        n = int(n_g[b])
        assert 0 <= n <= sl
        if n != n_o:
            assert close[min(n, n_o)], f"seq {b}: n_accept {n} != {n_o}"
        if n < sl:
            w = np.maximum(0.0, ref.y_T[r0 + n] - dp[n, b].astype(np.float64))
            if not w.sum() > 0:
                w = ref.y_T[r0 + n]
        else:
            w = ref.y_T[r0 + sl]
        tok = int(x_g[b])
        assert (n == n_o and tok == ref.next_token[b]) or _valid_draw(w, float(us[b]), tok), f"seq {b}: next {tok}"
        accepted_total += n
    return accepted_total, R - B


@pytest.mark.parametrize("path", [0, 1])
@pytest.mark.parametrize("V,d,sls", [(7, 8, [0]), (64, 16, [5]), (1000, 136, [3, 0, 5, 1]),
                                     (4099, 72, [1, 2, 3, 4, 5, 6]), (5000, 64, [7] * 20)])
def test_verify_sample_small_shapes(oracle, path, V, d, sls):
    _verify_sample_case(oracle, V, d, sls, seed=V + len(sls), path=path)


def test_verify_sample_uniform_look_ahead_and_acceptance_range(oracle):
    acc, tot = _verify_sample_case(oracle, 2000, 64, [4] * 12, seed=77, uniform=True, noise=0.3)
    assert 0.3 * tot < acc <= tot                # close distributions: most tokens pass
    acc2, tot2 = _verify_sample_case(oracle, 2000, 64, [4] * 12, seed=78, uniform=True, noise=6.0)
    assert acc2 < 0.6 * tot2                     # distant distributions: early rejections


@pytest.mark.parametrize("name,SL", [("vicuna_b1", 10), ("starcoder_b1", 10)])
def test_verify_sample_full_size_heads(oracle, name, SL):
    wl = inputs.WORKLOADS[name]
    _verify_sample_case(oracle, wl.V, wl.d_T, [SL], seed=wl.seed + 40)


# ---------------------------------------------------------------------------------- bulk feature extraction (App. D)
def _extract_case(oracle, V, dD, dT, N, seed, path=0):
    WD = inputs.lm_head(V, dD, seed=seed, std=0.25)
    WT = inputs.lm_head(V, dT, seed=seed + 1, std=0.25)
    HD = inputs.hidden(N, dD, seed=seed + 2)
    HT = inputs.hidden(N, dT, seed=seed + 3)
    # a share of the positions agrees by construction: both hidden states point along their head's row of one token
    g = torch.Generator().manual_seed(seed)
    toks = torch.randint(0, V, (N,), generator=g)
    for n in range(0, N, 3):
        HD[n] = (8.0 / 0.25 ** 2 / dD) * WD[toks[n]].float()
        HT[n] = (8.0 / 0.25 ** 2 / dT) * WT[toks[n]].float()
    HD, HT = HD.to(torch.bfloat16), HT.to(torch.bfloat16)
    pos = np.arange(N, dtype=np.int32) * 2 + 1
    ctx = _ctx(V, dD, dT, max_batch=8, max_rows=max(64, N))
    ctx.set_kernel_path(path)
    dev = "cuda"
    fD = torch.full((N, binding.NFEAT), -7.0, device=dev); fT = torch.full((N, binding.NFEAT), -7.0, device=dev)
    tv = torch.full((N,), -7.0, device=dev); label = torch.full((N,), 77, dtype=torch.uint8, device=dev)
    tD = torch.full((N,), -7, dtype=torch.int32, device=dev); tT = torch.full((N,), -7, dtype=torch.int32, device=dev)
    yD = torch.full((N, V), -7.0, device=dev); yT = torch.full((N, V), -7.0, device=dev)
    ctx.extract_features(WD.cuda(), HD.cuda(), WT.cuda(), HT.cuda(), torch.from_numpy(pos).cuda(), fD, fT, tv, label,
                         tD, tT, yD, yT)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    ctx.close()
    ref = oracle.extract_features(_bits(WD), _bits(HD), _bits(WT), _bits(HT), pos, nthreads=8)
    np.testing.assert_allclose(fD.cpu().numpy(), ref.feats_D, rtol=0, atol=2e-3)
    np.testing.assert_allclose(fT.cpu().numpy(), ref.feats_T, rtol=0, atol=2e-3)
    np.testing.assert_allclose(tv.cpu().numpy(), ref.tv, rtol=0, atol=2e-3)
    np.testing.assert_allclose(yD.cpu().numpy().astype(np.float64).sum(axis=1), 1.0, atol=1e-4)
    tDg, tTg, lab = tD.cpu().numpy(), tT.cpu().numpy(), label.cpu().numpy()
    tiedD, tiedT = ref.gap_D < 1e-3, ref.gap_T < 1e-3
    assert np.all((tDg == ref.token_D) | tiedD) and np.all((tTg == ref.token_T) | tiedT)
    for got_ids, Wm, Hm, tied in ((tDg, WD, HD, tiedD), (tTg, WT, HT, tiedT)):   # a near tie: best or runner-up only
        for n, pair in top2_ids(oracle, _bits(Wm), _bits(Hm), np.nonzero(tied)[0]).items():
            assert got_ids[n] in pair
    np.testing.assert_array_equal(lab, (tDg == tTg).astype(np.uint8))          # the rule, on the ids it reported
    ok = ~(tiedD | tiedT)
    np.testing.assert_array_equal(lab[ok], ref.label[ok])
    assert ref.label[::3].all() and lab[::3].all()                              # the constructed agreements
    return ref


@pytest.mark.parametrize("path", [0, 1])
@pytest.mark.parametrize("V,dD,dT,N", [(50, 16, 24, 1), (1000, 64, 136, 5), (4099, 72, 264, 19), (5000, 128, 64, 150)])
def test_extract_features_small_shapes(oracle, path, V, dD, dT, N):
    _extract_case(oracle, V, dD, dT, N, seed=V + N, path=path)


def test_extract_features_full_size_heads(oracle):
    wl = inputs.WORKLOADS["vicuna_b1"]
    ref = _extract_case(oracle, wl.V, wl.d_D, wl.d_T, 12, seed=wl.seed + 60)
    assert 0.0 < ref.tv.min() and ref.tv.max() <= 1.0


def test_verify_sample_edge_cases(oracle):
    """Identical distributions accept everything; draws at u = 0 and next to 1; a draft id outside the
    vocabulary is reported through the status word and ends that sequence's acceptance, nothing else."""
    V, d, B, SL = 3000, 64, 3, 4
    R = B * (SL + 1)
    W = inputs.lm_head(V, d, seed=5, std=0.25)
    H = inputs.hidden(R, d, seed=6)
    z = oracle.project(_bits(W), _bits(H), nthreads=8)
    e = np.exp(z - z.max(axis=1, keepdims=True))
    yT = e / e.sum(axis=1, keepdims=True)                                   # oracle's target rows
    dp = np.zeros((SL, B, V), dtype=np.float32)
    for b in range(B):
        dp[:, b] = yT[b * (SL + 1): b * (SL + 1) + SL].astype(np.float32)   # draft distributions = target's
    rng = np.random.default_rng(3)
    ids = np.array([rng.choice(V, p=yT[b * (SL + 1) + i]) for b in range(B) for i in range(SL)], dtype=np.int32)
    ua = rng.uniform(0.0, 0.99, size=B * SL).astype(np.float32)
    us = np.array([0.0, float(np.nextafter(np.float32(1.0), np.float32(0.0))), 0.5], dtype=np.float32)

    def run(ids_):
        ctx = _ctx(V, 8, d, max_batch=8, max_rows=64)
        n_acc = torch.full((B,), -7, dtype=torch.int32, device="cuda")
        nxt = torch.full((B,), -7, dtype=torch.int32, device="cuda")
        y = torch.zeros((R, V), dtype=torch.float32, device="cuda")
        ctx.verify_sample_ragged(W.cuda(), H.cuda(), torch.from_numpy(ids_).cuda(), torch.from_numpy(dp).cuda(), None, B, R,
                                 torch.from_numpy(ua).cuda(), torch.from_numpy(us).cuda(), n_acc, nxt, y)
        torch.cuda.synchronize()
        st = ctx.device_status()
        ctx.close()
        return n_acc.cpu().numpy(), nxt.cpu().numpy(), st

    n, x, st = run(ids)
    assert st == 0
    np.testing.assert_array_equal(n, SL)                                     # ratio ~ 1 > u: everything passes
    last = yT[np.arange(B) * (SL + 1) + SL]
    for b in range(B):
        assert _valid_draw(last[b], float(us[b]), int(x[b]))
    assert x[0] == int(np.argmax(last[0] > 0))                               # u = 0: first entry with mass
    assert last[1][x[1] + 1:].sum() < 1e-4                                   # u next to 1: only crumbs lie beyond

    bad = ids.copy()
    bad[SL + 2] = V                                                          # sequence 1, position 2
    n, x, st = run(bad)
    assert st == binding.ERR_INVALID_ARG
    assert n[0] == SL and n[2] == SL and n[1] == 2


def test_verify_sample_context_is_reusable_after_malformed_offsets(oracle):
    """The per-sequence tickets of the sampling kernel live in the context.  A call with overlapping row offsets
    (reported as an invalid argument) may leave them half counted; the next call must not inherit that: the same
    well-formed call before and after gives the same answer, and the answer matches the oracle."""
    V, d, sls = 1500, 72, [3, 0, 5, 2]
    B, R = len(sls), sum(sls) + len(sls)
    row_off = np.concatenate([[0], np.cumsum(np.array(sls) + 1)]).astype(np.int32)
    W = inputs.lm_head(V, d, seed=31, std=0.25)
    H = inputs.hidden(R, d, seed=32)
    rng = np.random.default_rng(33)
    z = oracle.project(_bits(W), _bits(H), nthreads=8)
    S = R - B          # as many steps as any look-ahead that fits the rows: whatever offsets arrive, reads stay inside
    dp = np.full((S, B, V), 1.0 / V, dtype=np.float32)
    ids = np.zeros(R - B, dtype=np.int32)
    for b in range(B):
        for i in range(sls[b]):
            zz = z[row_off[b] + i] + rng.normal(0.0, 1.0, V)
            e = np.exp(zz - zz.max())
            dp[i, b] = (e / e.sum()).astype(np.float32)
            ids[row_off[b] - b + i] = rng.choice(V, p=dp[i, b].astype(np.float64) / dp[i, b].astype(np.float64).sum())
    ua = rng.uniform(0.0, 1.0, R - B).astype(np.float32)
    us = rng.uniform(0.0, 1.0, B).astype(np.float32)
    ctx = _ctx(V, 8, d, max_batch=8, max_rows=64)
    Wc, Hc = W.cuda(), H.cuda()
    dev = lambda a: torch.from_numpy(a).cuda()

    def run(off):
        n_acc = torch.full((B,), -7, dtype=torch.int32, device="cuda")
        nxt = torch.full((B,), -7, dtype=torch.int32, device="cuda")
        y = torch.zeros((R, V), dtype=torch.float32, device="cuda")
        ctx.verify_sample_ragged(Wc, Hc, dev(ids), dev(dp), dev(off), B, R, dev(ua), dev(us), n_acc, nxt, y)
        torch.cuda.synchronize()
        return n_acc.cpu().numpy(), nxt.cpu().numpy(), y.cpu().numpy(), ctx.device_status()

    n1, x1, y1, st1 = run(row_off)
    assert st1 == 0
    bad = row_off.copy()
    bad[2] = bad[1] - 1          # sequence 1 ends before it starts; sequence 2 overlaps sequence 0
    _, _, _, st_bad = run(bad)
    assert st_bad == binding.ERR_INVALID_ARG
    n2, x2, y2, st2 = run(row_off)
    assert st2 == 0
    np.testing.assert_array_equal(n1, n2)
    np.testing.assert_array_equal(x1, x2)
    np.testing.assert_array_equal(y1, y2)
    ctx.close()
    ref = oracle.verify_sample(_bits(W), _bits(H), ids, dp, row_off, ua.astype(np.float64), us.astype(np.float64), nthreads=8)
    np.testing.assert_allclose(y1, ref.y_T, rtol=0, atol=2e-3)
    for b in range(B):
        if int(n1[b]) == int(ref.n_accept[b]):
            n = int(n1[b])
            r0 = int(row_off[b])
            w = np.maximum(0.0, ref.y_T[r0 + n] - dp[n, b].astype(np.float64)) if n < sls[b] else ref.y_T[r0 + sls[b]]
            assert x1[b] == ref.next_token[b] or _valid_draw(w, float(us[b]), int(x1[b]))
    assert (n1 == ref.n_accept).sum() >= B - 1      # an acceptance decided in the last bits may go either way


def test_look_ahead_is_monotone_in_the_threshold_at_full_size():
    """Batched Starcoder shapes, no oracle needed: on the same stream of hidden states the look-ahead that the
    stopping rule produces cannot grow with the threshold, the cap ends every sequence, and tau <= 0 never
    halts before the cap (the static policy)."""
    wl = inputs.WORKLOADS["starcoder_b256"]
    B, S = wl.B, wl.sl_max
    W = inputs.lm_head(wl.V, wl.d_D, seed=wl.seed, device="cuda")
    params = make_clf(wl.H, seed=wl.seed + 3)
    clf = to_gpu_clf(params)
    hs = [inputs.hidden(B, wl.d_D, seed=wl.seed * 100 + j, device="cuda") for j in range(S)]
    ctx = binding.Context(wl.V, wl.d_D, wl.d_T, max_batch=B, max_rows=B * (S + 1), clf_hidden=wl.H)
    pos = torch.arange(B, dtype=torch.int32, device="cuda")
    token = torch.zeros(B, dtype=torch.int32, device="cuda")
    conf = torch.zeros(B, dtype=torch.float32, device="cuda")
    halt = torch.zeros(B, dtype=torch.uint8, device="cuda")
    sl, confs = {}, {}
    for tau in (0.0, 0.3, 0.5, 0.7):
        active = torch.ones(B, dtype=torch.uint8, device="cuda")
        n = torch.zeros(B, dtype=torch.int64, device="cuda")
        cs = []
        for j in range(S):
            nd = torch.full((B,), j + 1, dtype=torch.int32, device="cuda")
            ctx.draft_step(W, hs[j], pos + j, nd, clf, tau, S, token, conf, halt, active=active)
            torch.cuda.synchronize()
            n += active.to(torch.int64)
            cs.append(torch.where(active.bool(), conf, torch.full_like(conf, float("nan"))).cpu().numpy())
            active = active & (1 - halt) if j + 1 < S else torch.zeros_like(active)
            if not bool(active.any()):
                break
        sl[tau] = n.cpu().numpy()
        confs[tau] = np.stack(cs)
    assert ctx.device_status() == 0
    ctx.close()
    assert np.all(sl[0.0] == S)                                       # tau = 0: only the cap halts
    assert np.all((sl[0.3] >= sl[0.5]) & (sl[0.5] >= sl[0.7]))
    assert np.all((sl[0.7] >= 1) & (sl[0.3] <= S))
    # the confidences do not depend on the threshold: wherever two runs both computed one, they agree bit for bit
    a, b = confs[0.0][: confs[0.7].shape[0]], confs[0.7]
    both = ~np.isnan(a) & ~np.isnan(b)
    assert both.any() and np.array_equal(a[both], b[both])
    # and each look-ahead is the first step whose confidence falls below the threshold
    c0 = confs[0.0]
    for tau in (0.3, 0.5, 0.7):
        below = c0 < np.float32(tau)
        first = np.where(below.any(axis=0), below.argmax(axis=0) + 1, S)
        np.testing.assert_array_equal(sl[tau], np.minimum(first, S))


# ---------------------------------------------------------------------------------- bounded waits
def test_a_wait_that_runs_out_is_reported_and_nothing_hangs():
    """The finishing warps of the batched draft step wait (bounded) for the per-CTA records of their sequence.
    With the test hook set those records never come: the wait must give up within the (shortened) budget, the
    kernel must return by itself, the status word must say DISCO_ERR_TIMEOUT, and after the context has been
    thrown away a fresh one must work as before."""
    V, d, B = 5000, 128, 12
    W = inputs.lm_head(V, d, seed=31, std=0.2).cuda()
    h = inputs.hidden(B, d, seed=32)
    clf = to_gpu_clf(make_clf(16, seed=33))
    pos, nd = np.arange(1, B + 1, dtype=np.int32), np.ones(B, np.int32)
    good_ctx = _ctx(V, d, 8, max_batch=B, H=16)
    good = gpu_draft_step(good_ctx, W, h, pos, nd, clf, 0.5, 4)
    assert good_ctx.device_status() == 0
    ctx = _ctx(V, d, 8, max_batch=B, H=16)
    ctx.test_hooks(wait_budget_clocks=2_000_000, withhold_records=True)      # about a millisecond
    try:
        gpu_draft_step(ctx, W, h, pos, nd, clf, 0.5, 4)                       # returns: the kernel ended by itself
        assert ctx.device_status() == binding.ERR_TIMEOUT
        assert ctx.device_status() == 0                                       # the word is cleared by the query
    finally:
        ctx.test_hooks(0, False)                                              # default budget again
        ctx.close()
    again = gpu_draft_step(good_ctx, W, h, pos, nd, clf, 0.5, 4)              # other contexts are not affected
    fresh = _ctx(V, d, 8, max_batch=B, H=16)
    new = gpu_draft_step(fresh, W, h, pos, nd, clf, 0.5, 4)
    for k in ("token", "conf", "halt", "feats"):
        np.testing.assert_array_equal(good[k], again[k])
        np.testing.assert_array_equal(good[k], new[k])
    assert fresh.device_status() == 0 and good_ctx.device_status() == 0
    fresh.close()
    good_ctx.close()
