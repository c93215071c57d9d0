"""Parity of the device-resident iteration (disco_draft_loop, disco_verify_sl, disco_iteration) with the CPU
oracle's plain loop, on the same seeded inputs.  Needs a B200: run with -m gpu."""
import numpy as np
import pytest
import torch

from paper_2405_04304_b200 import binding, inputs
import util
from util import GAP_EXEMPT, HALT_MARGIN, PROB_TOL, make_clf, to_gpu_clf, to_oracle_clf, top2_ids

pytestmark = pytest.mark.gpu


def _bits(t):
    return inputs.bf16_bits(t.reshape(-1, t.shape[-1])).reshape(t.shape)


def position_clf(cut: float, H: int = 4):
    """C = sigmoid(6 - 30 relu(pos - cut)): continue up to position cut, halt from cut + 1 on."""
    W1 = torch.zeros(H, 12)
    b1 = torch.zeros(H)
    w2 = torch.zeros(H)
    W1[0, 11], b1[0], w2[0] = 1.0, -cut, -30.0
    return W1, b1, w2, torch.tensor([6.0])


def make_inputs(V, dD, dT, B, S, seed, std=0.3):
    W_D = inputs.lm_head(V, dD, seed=seed, std=std)
    W_T = inputs.lm_head(V, dT, seed=seed + 1, std=std)
    h_D = inputs.hidden(S * B, dD, seed=seed + 2).view(S, B, dD)
    H_T = inputs.hidden(B * (S + 1), dT, seed=seed + 3).view(B, S + 1, dT)
    return W_D, W_T, h_D, H_T


def gpu_iteration(ctx, W_D, W_T, h_D, H_T, pos0, clf, tau, S, sl_forced=None, draft_ids=None, copies=1,
                  split=False, graph=False):
    """Run disco_iteration (or its two halves, split=True) and return numpy outputs; unwritten entries keep
    their sentinels (-7 / 77)."""
    B = h_D.shape[1]
    dev = "cuda"
    Wd = W_D.cuda()
    stride = 0
    if copies > 1:                                  # the same head once per step: every step reads its own copy
        assert copies >= S
        Wd = torch.stack([W_D] * copies).cuda()
        stride = W_D.numel() * 2
    Wt, hd, Ht = W_T.cuda(), h_D.cuda().contiguous(), H_T.cuda().contiguous()
    out = dict(token=torch.full((S, B), -7, dtype=torch.int32, device=dev),
               conf=torch.full((S, B), -7.0, dtype=torch.float32, device=dev),
               halt=torch.full((S, B), 77, dtype=torch.uint8, device=dev),
               feats=torch.full((S, B, binding.NFEAT), -7.0, dtype=torch.float32, device=dev),
               sl=torch.full((B,), -7, dtype=torch.int32, device=dev),
               n_accept=torch.full((B,), -7, dtype=torch.int32, device=dev),
               bonus=torch.full((B,), -7, dtype=torch.int32, device=dev),
               target_ids=torch.full((B, S + 1), -7, dtype=torch.int32, device=dev),
               row_off=torch.full((B + 1,), -7, dtype=torch.int32, device=dev),
               pos_next=torch.full((B,), -7, dtype=torch.int32, device=dev))
    p0 = torch.as_tensor(pos0, dtype=torch.int32).cuda()
    forced = None if sl_forced is None else torch.as_tensor(sl_forced, dtype=torch.int32).cuda()
    ids = None if draft_ids is None else torch.as_tensor(draft_ids, dtype=torch.int32).cuda().contiguous()

    def call(stream=None):
        if split:
            ctx.draft_loop(Wd, hd, p0, clf, tau, S, out["token"], out["conf"], out["halt"], out["sl"],
                           sl_forced=forced, feats=out["feats"], w_step_stride=stride, stream=stream)
            if ids is None:
                ctx.verify_sl(Wt, Ht, out["token"], 1, B, out["sl"], B, S, out["n_accept"], out["bonus"],
                              target_ids=out["target_ids"], row_off=out["row_off"], pos0=p0,
                              pos_next=out["pos_next"], stream=stream)
            else:
                ctx.verify_sl(Wt, Ht, ids, S, 1, out["sl"], B, S, out["n_accept"], out["bonus"],
                              target_ids=out["target_ids"], row_off=out["row_off"], pos0=p0,
                              pos_next=out["pos_next"], stream=stream)
        else:
            ctx.iteration(Wd, hd, Wt, Ht, p0, clf, tau, S, out["token"], out["conf"], out["halt"], out["sl"],
                          out["n_accept"], out["bonus"], sl_forced=forced, draft_ids=ids, feats=out["feats"],
                          target_ids=out["target_ids"], row_off=out["row_off"], pos_next=out["pos_next"],
                          w_step_stride=stride, stream=stream)

    if graph:
        st = torch.cuda.Stream()
        with torch.cuda.stream(st):
            call(st)                                 # eager once (kernel set-up happens outside the capture)
            st.synchronize()
            for v in out.values():
                v.fill_(-7 if v.dtype != torch.uint8 else 77)
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=st):
                call(st)
            g.replay()
            g.replay()                               # scratch must be left clean for the next replay
            st.synchronize()
    else:
        call()
    torch.cuda.synchronize()
    res = {k: v.cpu().numpy() for k, v in out.items()}
    res["pos0"] = np.asarray(pos0, dtype=np.int32)
    return res


def check_iteration(oracle, got, ref, W_T, H_T, tau, S, draft_ids=None):
    """Element by element against the oracle's IterationResult.  Returns the number of sequences exempted
    because of a near-tie arg-max."""
    B = ref.sl.shape[0]
    exempt = 0
    # near-tie rows of the verification: the two ids such a row may return
    tie_rows = [(b, j) for b in range(B) for j in range(ref.sl[b] + 1) if ref.gap_T[b, j] < GAP_EXEMPT]
    pairs = {}
    if tie_rows:
        flat = [b * (S + 1) + j for b, j in tie_rows]
        t2 = top2_ids(oracle, _bits(W_T), _bits(H_T).reshape(B * (S + 1), -1), flat)
        pairs = {bj: t2[f] for bj, f in zip(tie_rows, flat)}
    for b in range(B):
        n = int(ref.sl[b])
        # no halt decision of this sequence was within the margin of tau: the look-ahead must be the oracle's
        close = [i for i in range(n) if abs(ref.conf[i, b] - tau) < HALT_MARGIN]
        util.COUNTS["halt_checked"] += n
        util.COUNTS["halt_exempt"] += len(close)
        assert not close, "a halt decision within the margin: pick another seed for this case"
        assert got["sl"][b] == n, f"seq {b}: look-ahead {got['sl'][b]} != {n}"
        tok_tie = False
        for i in range(n):
            if ref.gap_D[i, b] < GAP_EXEMPT:
                util.COUNTS["argmax_near_tie"] += 1
                tok_tie = True
            else:
                assert got["token"][i, b] == ref.token[i, b], f"seq {b} step {i}: token"
            assert abs(float(got["conf"][i, b]) - ref.conf[i, b]) <= PROB_TOL
            util.COUNTS["max_conf_err"] = max(util.COUNTS["max_conf_err"], abs(float(got["conf"][i, b]) - ref.conf[i, b]))
            assert got["halt"][i, b] == ref.halt[i, b], f"seq {b} step {i}: halt"
            np.testing.assert_allclose(got["feats"][i, b], ref.feats[i, b], rtol=0, atol=PROB_TOL)
        # steps the sequence did not take were not written
        assert np.all(got["token"][n:, b] == -7) and np.all(got["halt"][n:, b] == 77)
        assert np.all(got["conf"][n:, b] == -7.0) and np.all(got["feats"][n:, b] == -7.0)
        # verification
        tid = got["target_ids"][b]
        assert np.all(tid[n + 1:] == -7), "target ids beyond the look-ahead were written"
        tied = False
        for j in range(n + 1):
            if (b, j) in pairs:
                tied = True
                util.COUNTS["verify_rows_near_tie"] += 1
                assert int(tid[j]) in pairs[(b, j)]
            else:
                assert tid[j] == ref.target_ids[b, j], f"seq {b} row {j}: target id"
        offered = got["token"][:n, b] if draft_ids is None else np.asarray(draft_ids)[b, :n]
        k = 0
        while k < n and offered[k] == tid[k]:
            k += 1
        assert got["n_accept"][b] == k and got["bonus"][b] == tid[k], "not the prefix rule on the reported ids"
        if tied or (draft_ids is None and tok_tie):
            exempt += 1
        else:
            assert got["n_accept"][b] == ref.n_accept[b] and got["bonus"][b] == ref.bonus[b]
    np.testing.assert_array_equal(got["row_off"], np.concatenate([[0], np.cumsum(ref.sl + 1)]))
    if "pos0" in got:                                     # the next iteration's position base
        np.testing.assert_array_equal(got["pos_next"], got["pos0"] + got["n_accept"] + 1)
    return exempt


@pytest.mark.parametrize("split,graph", [(False, False), (True, False), (False, True)])
@pytest.mark.parametrize("V,dD,dT,B,S", [(50, 16, 24, 1, 4), (1000, 72, 136, 3, 6), (4099, 264, 72, 7, 5),
                                         (3000, 128, 64, 20, 9), (2000, 64, 72, 12, 11), (1500, 64, 136, 40, 16)])
def test_iteration_small_shapes(oracle, V, dD, dT, B, S, split, graph):
    W_D, W_T, h_D, H_T = make_inputs(V, dD, dT, B, S, seed=V + B)
    pos0 = (np.arange(B, dtype=np.int32) * 3) % 11
    params = position_clf(cut=8.0)                         # look-aheads 1 .. S, some sequences capped
    ctx = binding.Context(V, dD, dT, max_batch=B, max_rows=B * (S + 1), clf_hidden=8)
    clf_o = to_oracle_clf(oracle, params)
    # offered ids: the oracle's own target tokens, corrupted
    free = oracle.verify_padded(_bits(W_T), _bits(H_T), [S] * B, np.zeros((B, S), np.int32), S, 1, nthreads=8)[2]
    ids = inputs.corrupt_ids(torch.from_numpy(free[:, :S].copy()), 0.25, V, seed=B).numpy()
    for draft_ids in (ids, None):
        got = gpu_iteration(ctx, W_D, W_T, h_D, H_T, pos0, to_gpu_clf(params), 0.5, S, draft_ids=draft_ids,
                            split=split, graph=graph)
        ref = oracle.iteration(_bits(W_D), _bits(h_D), _bits(W_T), _bits(H_T), pos0, clf_o, 0.5, S,
                               draft_ids=draft_ids, nthreads=8)
        check_iteration(oracle, got, ref, W_T, H_T, 0.5, S, draft_ids)
        assert len(set(ref.sl.tolist())) > 1 or B == 1      # the look-aheads really differ
    assert ctx.device_status() == 0
    ctx.close()


@pytest.mark.parametrize("B", [1, 2, 4, 5])
def test_iteration_every_small_vocabulary(oracle, B):
    """V = 1 .. 48 without a gap through the whole iteration: the persistent draft-phase kernel for up to four
    sequences (147 CTAs without a vocabulary row, fewer than ten logits), the chained per-step launches for five."""
    dD, dT, S = 16, 24, 4
    params = position_clf(cut=6.0)
    clf_g, clf_o = to_gpu_clf(params), to_oracle_clf(oracle, params)
    pos0 = (np.arange(B, dtype=np.int32) * 2 + 3) % 8
    for V in range(1, 49):
        W_D, W_T, h_D, H_T = make_inputs(V, dD, dT, B, S, seed=500 + V)
        ctx = binding.Context(V, dD, dT, max_batch=B, max_rows=B * (S + 1), clf_hidden=8)
        got = gpu_iteration(ctx, W_D, W_T, h_D, H_T, pos0, clf_g, 0.5, S)
        ref = oracle.iteration(_bits(W_D), _bits(h_D), _bits(W_T), _bits(H_T), pos0, clf_o, 0.5, S, nthreads=4)
        check_iteration(oracle, got, ref, W_T, H_T, 0.5, S)
        assert ctx.device_status() == 0, f"V = {V}"
        ctx.close()


@pytest.mark.parametrize("path", [1, 2, 3])
@pytest.mark.parametrize("B", [2, 12])
def test_iteration_on_each_kernel_path(oracle, path, B):
    V, dD, dT, S = 2000, 64, 136, 6
    W_D, W_T, h_D, H_T = make_inputs(V, dD, dT, B, S, seed=40 + B)
    pos0 = np.arange(B, dtype=np.int32) % 7
    params = position_clf(cut=5.0)
    ctx = binding.Context(V, dD, dT, max_batch=B, max_rows=B * (S + 1), clf_hidden=8)
    ctx.set_kernel_path(path)
    got = gpu_iteration(ctx, W_D, W_T, h_D, H_T, pos0, to_gpu_clf(params), 0.5, S, copies=S)
    ref = oracle.iteration(_bits(W_D), _bits(h_D), _bits(W_T), _bits(H_T), pos0, to_oracle_clf(oracle, params), 0.5,
                           S, nthreads=8)
    check_iteration(oracle, got, ref, W_T, H_T, 0.5, S)
    assert ctx.device_status() == 0
    ctx.close()


def test_iteration_degenerate_policies(oracle):
    """tau <= 0: the static policy, every sequence drafts SL_max tokens; tau > 1: one token; a forced
    look-ahead overrules the classifier; a random-initialised classifier at its own threshold."""
    V, dD, dT, B, S = 1500, 40, 48, 6, 5
    W_D, W_T, h_D, H_T = make_inputs(V, dD, dT, B, S, seed=77)
    pos0 = np.arange(B, dtype=np.int32) * 2
    params = make_clf(16, seed=5)
    ctx = binding.Context(V, dD, dT, max_batch=B, max_rows=B * (S + 1), clf_hidden=16)
    clf_g, clf_o = to_gpu_clf(params), to_oracle_clf(oracle, params)
    args = (_bits(W_D), _bits(h_D), _bits(W_T), _bits(H_T), pos0, clf_o)
    got = gpu_iteration(ctx, W_D, W_T, h_D, H_T, pos0, clf_g, 0.0, S)
    assert list(got["sl"]) == [S] * B and np.all(got["halt"][: S - 1] == 0) and np.all(got["halt"][S - 1] == 1)
    check_iteration(oracle, got, oracle.iteration(*args, 0.0, S, nthreads=8), W_T, H_T, 0.0, S)
    got = gpu_iteration(ctx, W_D, W_T, h_D, H_T, pos0, clf_g, 1.5, S)
    assert list(got["sl"]) == [1] * B
    check_iteration(oracle, got, oracle.iteration(*args, 1.5, S, nthreads=8), W_T, H_T, 1.5, S)
    forced = np.array([3, 1, 9, 5, 2, 4], np.int32)
    got = gpu_iteration(ctx, W_D, W_T, h_D, H_T, pos0, clf_g, 1.5, S, sl_forced=forced)
    assert list(got["sl"]) == list(np.minimum(forced, S))
    check_iteration(oracle, got, oracle.iteration(*args, 1.5, S, sl_forced=forced, nthreads=8), W_T, H_T, 1.5, S)
    assert ctx.device_status() == 0
    ctx.close()


def test_iteration_host_entry_point_matches_the_device_one(oracle):
    """disco_iteration_host: the same iteration with every per-iteration array in host memory; the position
    base is advanced in place, as a host loop would carry it from one iteration to the next."""
    V, dD, dT, B, S = 3000, 72, 136, 5, 6
    W_D, W_T, h_D, H_T = make_inputs(V, dD, dT, B, S, seed=91)
    pos0 = np.array([0, 2, 4, 6, 8], np.int32)
    params = position_clf(cut=6.0)
    rng = np.random.default_rng(9)
    ids = rng.integers(0, V, size=(B, S)).astype(np.int32)
    ctx = binding.Context(V, dD, dT, max_batch=B, max_rows=B * (S + 1), clf_hidden=8)
    clf = to_gpu_clf(params)
    dev = gpu_iteration(ctx, W_D, W_T, h_D, H_T, pos0, clf, 0.5, S, draft_ids=ids)
    pin = lambda t: t.contiguous().pin_memory()
    token, conf = pin(torch.full((S, B), -7, dtype=torch.int32)), pin(torch.full((S, B), -7.0))
    halt = pin(torch.full((S, B), 77, dtype=torch.uint8))
    sl, n_acc, bonus = (pin(torch.full((B,), -7, dtype=torch.int32)) for _ in range(3))
    pos = pin(torch.from_numpy(pos0.copy()))
    ctx.iteration_host(W_D.cuda(), pin(h_D), W_T.cuda(), pin(H_T), pos, clf, 0.5, S, token, conf, halt, sl, n_acc,
                       bonus, draft_ids=pin(torch.from_numpy(ids)), pos_next=pos)
    for k, t in (("token", token), ("conf", conf), ("halt", halt), ("sl", sl), ("n_accept", n_acc), ("bonus", bonus)):
        np.testing.assert_array_equal(t.numpy(), dev[k])
    np.testing.assert_array_equal(pos.numpy(), pos0 + dev["n_accept"] + 1)
    assert ctx.device_status() == 0
    ctx.close()


def test_verify_sl_rejects_a_look_ahead_outside_its_range():
    V, d, B, S = 300, 32, 3, 4
    ctx = binding.Context(V, 8, d, max_batch=B, max_rows=B * (S + 1))
    W = inputs.lm_head(V, d, seed=1).cuda()
    H = inputs.hidden(B * (S + 1), d, seed=2).cuda()
    ids = torch.zeros(B * S, dtype=torch.int32, device="cuda")
    n = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    bonus = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    sl = torch.tensor([2, S + 1, -1], dtype=torch.int32, device="cuda")
    ctx.verify_sl(W, H, ids, S, 1, sl, B, S, n, bonus)
    torch.cuda.synchronize()
    assert n[0] >= 0 and n[1] == -1 and n[2] == -1 and bonus[1] == -1
    assert ctx.device_status() == binding.ERR_INVALID_ARG
    with pytest.raises(binding.DiscoError) as e:          # more rows than the context was created for
        ctx.verify_sl(W, H, ids, S, 1, sl, B + 1, S, n, bonus)
    assert e.value.code == binding.ERR_WORKSPACE
    ctx.close()


@pytest.mark.parametrize("name", ["vicuna_b1", "starcoder_b1"])
def test_iteration_full_size_single_sequence(oracle, name):
    """The configuration bench.py times: full-size heads, one sequence, ids offered = the target's own tokens
    corrupted at the workload's rate; a look-ahead in the middle of the range."""
    wl = inputs.WORKLOADS[name]
    S = wl.sl_max
    W_D = inputs.lm_head(wl.V, wl.d_D, seed=inputs.sub_seed(wl.seed, 1))
    W_T = inputs.lm_head(wl.V, wl.d_T, seed=inputs.sub_seed(wl.seed, 2))
    h_D = inputs.hidden(S, wl.d_D, seed=inputs.sub_seed(wl.seed, 4)).view(S, 1, wl.d_D)
    H_T = inputs.hidden(S + 1, wl.d_T, seed=inputs.sub_seed(wl.seed, 5)).view(1, S + 1, wl.d_T)
    params = position_clf(cut=13.0)
    pos0 = np.array([9], np.int32)                          # look-ahead 5
    free = oracle.verify_padded(_bits(W_T), _bits(H_T), [S], np.zeros((1, S), np.int32), S, 1, nthreads=16)[2]
    ids = inputs.corrupt_ids(torch.from_numpy(free[:, :S].copy()), wl.p_corrupt, wl.V, seed=wl.seed).numpy()
    ctx = binding.Context(wl.V, wl.d_D, wl.d_T, max_batch=1, max_rows=S + 1, clf_hidden=8)
    got = gpu_iteration(ctx, W_D, W_T, h_D, H_T, pos0, to_gpu_clf(params), 0.5, S, draft_ids=ids, copies=S)
    ref = oracle.iteration(_bits(W_D), _bits(h_D), _bits(W_T), _bits(H_T), pos0, to_oracle_clf(oracle, params), 0.5,
                           S, draft_ids=ids, nthreads=16)
    assert ref.sl[0] == 5
    check_iteration(oracle, got, ref, W_T, H_T, 0.5, S, ids)
    assert ctx.device_status() == 0
    ctx.close()


def test_iteration_full_size_ragged_batch(oracle):
    """Batched Vicuna shapes, 64 sequences with forced look-aheads drawn from 1..10 (the workload's recipe).
    The sequences are independent, so the oracle runs a sample of them, each as a batch of one."""
    wl = inputs.WORKLOADS["vicuna_b64"]
    B, S = wl.B, wl.sl_max
    W_D = inputs.lm_head(wl.V, wl.d_D, seed=inputs.sub_seed(wl.seed, 1))
    W_T = inputs.lm_head(wl.V, wl.d_T, seed=inputs.sub_seed(wl.seed, 2))
    h_D = inputs.hidden(S * B, wl.d_D, seed=inputs.sub_seed(wl.seed, 4)).view(S, B, wl.d_D)
    H_T = inputs.hidden(B * (S + 1), wl.d_T, seed=inputs.sub_seed(wl.seed, 5)).view(B, S + 1, wl.d_T)
    forced = inputs.uniform_sl(B, 1, S, inputs.sub_seed(wl.seed, 8)).numpy()
    params = make_clf(wl.H, seed=inputs.sub_seed(wl.seed, 3))
    pos0 = (np.arange(B, dtype=np.int32) * 5) % 23
    rng = np.random.default_rng(wl.seed)
    ids = rng.integers(0, wl.V, size=(B, S)).astype(np.int32)
    sample = [0, 1, 17, 31, 32, 62, 63]
    clf_o = to_oracle_clf(oracle, params)
    # plant the oracle's target tokens in the sampled sequences' first positions so that some are accepted
    for b in sample:
        free = oracle.verify_padded(_bits(W_T), _bits(H_T[b:b + 1]), [int(forced[b])], np.zeros((1, S), np.int32),
                                    S, 1, nthreads=16)[2][0]
        ids[b, : max(1, int(forced[b]) - 1)] = free[: max(1, int(forced[b]) - 1)]
    ctx = binding.Context(wl.V, wl.d_D, wl.d_T, max_batch=B, max_rows=B * (S + 1), clf_hidden=wl.H)
    got = gpu_iteration(ctx, W_D, W_T, h_D, H_T, pos0, to_gpu_clf(params), wl.tau, S, sl_forced=forced, draft_ids=ids)
    assert ctx.device_status() == 0
    ctx.close()
    np.testing.assert_array_equal(got["sl"], forced)
    np.testing.assert_array_equal(got["row_off"], np.concatenate([[0], np.cumsum(forced + 1)]))
    for b in range(B):                                     # every sequence: the prefix rule on the reported ids
        n, tid = int(forced[b]), got["target_ids"][b]
        k = 0
        while k < n and ids[b, k] == tid[k]:
            k += 1
        assert got["n_accept"][b] == k and got["bonus"][b] == tid[k]
        assert np.all(tid[n + 1:] == -7) and np.all(got["token"][n:, b] == -7)
    for b in sample:
        ref = oracle.iteration(_bits(W_D), _bits(h_D[:, b:b + 1]), _bits(W_T), _bits(H_T[b:b + 1]), pos0[b:b + 1],
                               clf_o, wl.tau, S, sl_forced=forced[b:b + 1], draft_ids=ids[b:b + 1], nthreads=16)
        one = {k: (v[:, b:b + 1] if k in ("token", "conf", "halt", "feats") else v[b:b + 1]) for k, v in got.items()
               if k != "row_off"}
        one["row_off"] = np.array([0, forced[b] + 1])
        check_iteration(oracle, one, ref, W_T, H_T[b:b + 1], wl.tau, S, ids[b:b + 1])
