"""Pins of the CPU oracle: each oracle function is fixed to something other than itself
(closed forms, textbook special cases, brute force with independent code, values the paper prints).
"""
import math
import os
import struct

import numpy as np
import pytest
import torch

from paper_2405_04304_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bits_of(t: torch.Tensor) -> np.ndarray:
    return inputs.bf16_bits(t.to(torch.bfloat16))


def py_bf16(bits: int) -> float:
    """Decode one bf16 pattern with the struct module (independent of the oracle's decoder)."""
    return struct.unpack("<f", struct.pack("<I", int(bits) << 16))[0]


# ------------------------------------------------------------------ projection
def test_project_brute_force_python_loops(oracle):
    rng = np.random.default_rng(5)
    V, d, R = 37, 19, 3   # all different: a transposed operand or swapped extent cannot pass
    W = bits_of(torch.from_numpy(rng.normal(size=(V, d)).astype(np.float32)))
    H = bits_of(torch.from_numpy(rng.normal(size=(R, d)).astype(np.float32)))
    z = oracle.project(W, H)
    assert z.shape == (R, V)
    for r in range(R):
        for v in range(V):
            ref = math.fsum(py_bf16(W[v, j]) * py_bf16(H[r, j]) for j in range(d))
            assert abs(z[r, v] - ref) < 1e-12


def test_project_unit_vector_selects_column(oracle):
    V, d = 33, 24
    Wt = torch.randn(V, d, generator=torch.Generator().manual_seed(1)).to(torch.bfloat16)
    for j in (0, 7, d - 1):
        h = torch.zeros(1, d)
        h[0, j] = 1.0
        z = oracle.project(bits_of(Wt), bits_of(h))
        np.testing.assert_array_equal(z[0], Wt[:, j].double().numpy())


def test_project_one_hot_rows_copy_hidden(oracle):
    d = 16
    Wt = torch.eye(d)                       # V = d, row v is e_v
    h = torch.randn(2, d, generator=torch.Generator().manual_seed(2)).to(torch.bfloat16)
    z = oracle.project(bits_of(Wt), bits_of(h))
    np.testing.assert_array_equal(z, h.double().numpy())


def test_project_matches_numpy_matmul_and_threads(oracle):
    g = torch.Generator().manual_seed(3)
    Wt = (torch.randn(200, 72, generator=g) * 0.02).to(torch.bfloat16)
    Ht = torch.randn(5, 72, generator=g).to(torch.bfloat16)
    z1 = oracle.project(bits_of(Wt), bits_of(Ht), nthreads=1)
    z4 = oracle.project(bits_of(Wt), bits_of(Ht), nthreads=4)
    np.testing.assert_array_equal(z1, z4)          # threads split rows, never a sum
    ref = Ht.double().numpy() @ Wt.double().numpy().T
    np.testing.assert_allclose(z1, ref, rtol=0, atol=1e-13)


# ------------------------------------------------------------------ argmax
def test_argmax_lowest_index_on_ties_and_gap(oracle):
    assert oracle.argmax(np.array([1.0, 3.0, 3.0, 2.0])) == (1, 0.0)
    best, gap = oracle.argmax(np.array([0.5, -1.0, 4.0, 3.25]))
    assert best == 2 and gap == 0.75
    best, gap = oracle.argmax(np.array([7.0]))
    assert best == 0 and math.isinf(gap)
    assert oracle.argmax(np.zeros(9))[0] == 0


# ------------------------------------------------------------------ soft-max
def test_softmax_sums_to_one_and_matches_scipy(oracle):
    from scipy.special import softmax as sp_softmax
    rng = np.random.default_rng(0)
    for V in (1, 2, 10, 1000):
        z = rng.normal(scale=3.0, size=V)
        y = oracle.softmax(z)
        assert abs(y.sum() - 1.0) < 1e-12
        np.testing.assert_allclose(y, sp_softmax(z), rtol=1e-12, atol=0)


def test_softmax_shift_invariance_and_large_logits(oracle):
    z = np.array([1000.0, 999.0, 998.0])
    y = oracle.softmax(z)
    e = np.exp([0.0, -1.0, -2.0])
    np.testing.assert_allclose(y, e / e.sum(), rtol=1e-14)
    np.testing.assert_allclose(oracle.softmax(z - 1000.0), y, rtol=1e-14)


def test_zero_hidden_state_gives_uniform(oracle):
    V, d = 50, 8
    W = bits_of(torch.randn(V, d, generator=torch.Generator().manual_seed(4)))
    z = oracle.project(W, bits_of(torch.zeros(1, d)))[0]
    y = oracle.softmax(z)
    np.testing.assert_allclose(y, np.full(V, 1.0 / V), rtol=1e-15)
    assert abs(oracle.entropy(y) - math.log(V)) < 1e-12
    assert oracle.argmax(z)[0] == 0


# ------------------------------------------------------------------ top-k
def test_topk_equals_full_sort(oracle):
    rng = np.random.default_rng(1)
    y = rng.dirichlet(np.ones(64))
    vals, ids = oracle.topk(y, 10)
    order = sorted(range(64), key=lambda v: (-y[v], v))[:10]
    assert list(ids) == order
    np.testing.assert_array_equal(vals, y[order])
    assert all(vals[i] >= vals[i + 1] for i in range(9))
    assert vals.sum() <= 1.0 + 1e-15


def test_topk_ties_keep_lowest_index_and_padding(oracle):
    y = np.array([0.1, 0.3, 0.3, 0.1, 0.2])
    vals, ids = oracle.topk(y, 10)
    assert list(ids[:5]) == [1, 2, 4, 0, 3]
    assert list(ids[5:]) == [-1] * 5
    np.testing.assert_array_equal(vals, [0.3, 0.3, 0.2, 0.1, 0.1, 0, 0, 0, 0, 0])


def test_top0_is_one_over_Z(oracle):
    rng = np.random.default_rng(2)
    z = rng.normal(size=300)
    y = oracle.softmax(z)
    vals, ids = oracle.topk(y, 10)
    assert ids[0] == oracle.argmax(z)[0]
    assert abs(vals[0] - 1.0 / np.exp(z - z.max()).sum()) < 1e-15


# ------------------------------------------------------------------ entropy
def test_entropy_two_level_closed_form(oracle):
    V = 1000
    for L in (0.0, 1.0, 5.0, 12.0):
        z = np.zeros(V)
        z[123] = L
        y = oracle.softmax(z)
        p = math.exp(L) / (math.exp(L) + V - 1)
        ref = -p * math.log(p) - (1 - p) * math.log((1 - p) / (V - 1))
        assert abs(oracle.entropy(y) - ref) < 1e-12


def test_entropy_bounds_zero_terms_and_scipy(oracle):
    from scipy.stats import entropy as sp_entropy
    assert oracle.entropy(np.array([1.0, 0.0, 0.0])) == 0.0
    rng = np.random.default_rng(3)
    y = rng.dirichlet(np.ones(200) * 0.3)
    e = oracle.entropy(y)
    assert 0.0 <= e <= math.log(200)
    assert abs(e - sp_entropy(y)) < 1e-12          # natural logarithm


def test_planted_peak_drives_top0_to_one(oracle):
    V, d = 64, 32
    g = torch.Generator().manual_seed(6)
    Wt = (torch.randn(V, d, generator=g) * 0.1).to(torch.bfloat16)
    h = (Wt[17].float() * 400.0).to(torch.bfloat16).view(1, d)
    z = oracle.project(bits_of(Wt), bits_of(h))[0]
    y = oracle.softmax(z)
    x = oracle.features(y, pos=3)
    assert oracle.argmax(z)[0] == 17
    assert x[0] > 0.999 and x[10] < 0.02


# ------------------------------------------------------------------ features
def test_feature_layout(oracle):
    rng = np.random.default_rng(4)
    y = rng.dirichlet(np.ones(40))
    x = oracle.features(y, pos=77)
    assert x.shape == (12,)
    np.testing.assert_array_equal(x[:10], np.sort(y)[::-1][:10])
    assert abs(x[10] + float((y * np.log(y)).sum())) < 1e-13
    assert x[11] == 77.0


# ------------------------------------------------------------------ classifier
def _clf(oracle, W1, b1, w2, b2):
    return oracle.Classifier(np.array(W1, np.float32), np.array(b1, np.float32),
                             np.array(w2, np.float32), np.array([b2], np.float32))


def test_classifier_zero_head_gives_half(oracle):
    rng = np.random.default_rng(5)
    clf = _clf(oracle, rng.normal(size=(8, 12)), rng.normal(size=8), np.zeros(8), 0.0)
    assert oracle.classifier(rng.normal(size=12), clf) == 0.5


def test_classifier_hand_computed(oracle):
    # two hidden units on three features: a = relu([x0 - x2 + 0.5, -x1 + 0.25]) ; s = 2 a0 - 3 a1 + 0.125
    clf = _clf(oracle, [[1, 0, -1], [0, -1, 0]], [0.5, 0.25], [2, -3], 0.125)
    x = np.array([0.75, 0.5, 0.25])              # a = [1.0, relu(-0.25) = 0]
    assert abs(oracle.classifier(x, clf) - 1 / (1 + math.exp(-2.125))) < 1e-15
    x = np.array([0.0, -0.75, 1.0])              # a = [relu(-0.5) = 0, 1.0] ; s = -2.875
    assert abs(oracle.classifier(x, clf) - 1 / (1 + math.exp(2.875))) < 1e-15


def test_classifier_relu_is_not_identity(oracle):
    clf = _clf(oracle, [[1.0]], [0.0], [1.0], 0.0)
    assert oracle.classifier(np.array([-5.0]), clf) == 0.5            # clipped to 0
    assert abs(oracle.classifier(np.array([2.0]), clf) - 1 / (1 + math.exp(-2.0))) < 1e-15


# ------------------------------------------------------------------ whole draft step
def _small_problem(seed, V=50, d=16, B=3, H=8):
    g = torch.Generator().manual_seed(seed)
    W = (torch.randn(V, d, generator=g) * 0.5).to(torch.bfloat16)
    h = torch.randn(B, d, generator=g).to(torch.bfloat16)
    W1, b1, w2, b2 = inputs.classifier_params(H, seed + 100)
    return W, h, (W1.numpy(), b1.numpy(), w2.numpy(), b2.numpy())


def test_draft_step_against_independent_numpy_pipeline(oracle):
    from scipy.special import softmax as sp_softmax
    W, h, (W1, b1, w2, b2) = _small_problem(11)
    clf = oracle.Classifier(W1, b1, w2, b2)
    pos = np.array([1, 5, 9], np.int32)
    nd = np.array([1, 2, 3], np.int32)
    res = oracle.draft_step(bits_of(W), bits_of(h), pos, nd, clf, tau=0.5, sl_max=4, want_probs=True)
    z = h.double().numpy() @ W.double().numpy().T
    y = sp_softmax(z, axis=1)
    for b in range(3):
        assert res.token[b] == int(np.argmax(z[b]))
        np.testing.assert_allclose(res.probs[b], y[b], rtol=1e-12)
        x = np.concatenate([np.sort(y[b])[::-1][:10], [-(y[b] * np.log(y[b])).sum()], [float(pos[b])]])
        np.testing.assert_allclose(res.feats[b], x, rtol=1e-12)
        a = np.maximum(W1.astype(np.float64) @ x + b1, 0.0)
        C = 1.0 / (1.0 + math.exp(-(float(w2.astype(np.float64) @ a) + float(b2[0]))))
        assert abs(res.conf[b] - C) < 1e-14
        assert res.halt[b] == int(np.float32(C) < np.float32(0.5) or nd[b] >= 4)


def test_threshold_rule_static_sl_special_cases(oracle):
    W, h, (W1, b1, w2, b2) = _small_problem(12)
    clf = oracle.Classifier(W1, b1, w2, b2)
    pos = np.arange(1, 4, dtype=np.int32)
    # tau <= 0 never halts before the cap: static SL = SL_max (Sec. 3)
    for nd, expect in ((1, 0), (4, 0), (5, 1), (6, 1)):
        r = oracle.draft_step(bits_of(W), bits_of(h), pos, np.full(3, nd, np.int32), clf, 0.0, 5)
        assert list(r.halt) == [expect] * 3
    # tau > 1 halts after the first token
    r = oracle.draft_step(bits_of(W), bits_of(h), pos, np.ones(3, np.int32), clf, 1.5, 5)
    assert list(r.halt) == [1, 1, 1]
    # C == tau continues: zero output layer gives C = 0.5 exactly
    flat = oracle.Classifier(W1, b1, np.zeros_like(w2), np.zeros(1, np.float32))
    r = oracle.draft_step(bits_of(W), bits_of(h), pos, np.ones(3, np.int32), flat, 0.5, 5)
    assert list(r.conf) == [0.5] * 3 and list(r.halt) == [0, 0, 0]
    r = oracle.draft_step(bits_of(W), bits_of(h), pos, np.ones(3, np.int32), flat, 0.5000001, 5)
    assert list(r.halt) == [1, 1, 1]


def test_halt_is_monotone_in_tau(oracle):
    W, h, (W1, b1, w2, b2) = _small_problem(13, B=3)
    clf = oracle.Classifier(W1, b1, w2, b2)
    pos = np.array([2, 3, 4], np.int32)
    nd = np.ones(3, np.int32)
    halts = [oracle.draft_step(bits_of(W), bits_of(h), pos, nd, clf, tau, 9).halt for tau in (0.3, 0.5, 0.7)]
    assert np.all(halts[0] <= halts[1]) and np.all(halts[1] <= halts[2])


def test_inactive_sequences_untouched(oracle):
    W, h, (W1, b1, w2, b2) = _small_problem(14)
    clf = oracle.Classifier(W1, b1, w2, b2)
    pos = np.ones(3, np.int32)
    r = oracle.draft_step(bits_of(W), bits_of(h), pos, pos, clf, 0.5, 5, active=np.array([1, 0, 1], np.uint8))
    assert r.token[1] == -1 and r.halt[1] == 255 and np.isnan(r.conf[1])
    assert r.token[0] >= 0 and r.token[2] >= 0


# ------------------------------------------------------------------ verification
def _golden_pairs(name):
    rows = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append(line.split())
    return rows


def test_fig1_worked_example(oracle):
    g = dict((k, int(v)) for k, v in _golden_pairs("fig1_iteration.txt"))
    SL = g["SL"]
    target = np.array([11, 12, 13, 14, 15, 16], np.int32)        # SL + 1 target tokens
    draft = target[:SL].copy()
    draft[g["accepted"]] = 99                                     # t4 wrong
    draft[g["accepted"] + 1] = 98                                 # t5 wrong
    n, bonus = oracle.accept_prefix(draft, target)
    assert n == g["accepted"] and n + 1 == g["emitted"]
    assert bonus == target[n]


def test_prefix_rule_special_cases(oracle):
    target = np.array([5, 6, 7, 8, 9, 10], np.int32)
    assert oracle.accept_prefix(target[:5], target) == (5, 10)             # all accepted -> row SL
    bad_first = np.array([0, 6, 7, 8, 9], np.int32)
    assert oracle.accept_prefix(bad_first, target) == (0, 5)               # later matches do not count
    hole = np.array([5, 6, 7, 0, 9], np.int32)
    assert oracle.accept_prefix(hole, target) == (3, 8)
    assert oracle.accept_prefix(np.zeros(0, np.int32), target[:1]) == (0, 5)   # SL = 0: plain target step


def test_verify_draft_equal_to_argmax_accepts_all(oracle):
    g = torch.Generator().manual_seed(21)
    V, d, SL = 64, 24, 4
    W = (torch.randn(V, d, generator=g)).to(torch.bfloat16)
    H = torch.randn(SL + 1, d, generator=g).to(torch.bfloat16)
    z = H.double().numpy() @ W.double().numpy().T
    a = np.argmax(z, axis=1).astype(np.int32)
    r = oracle.verify(bits_of(W), bits_of(H), a[:SL], B=1, SL=SL)
    assert r.n_accept[0] == SL and r.bonus[0] == a[SL]
    np.testing.assert_array_equal(r.target_ids, a)
    srt = np.sort(z, axis=1)
    np.testing.assert_allclose(r.gap, srt[:, -1] - srt[:, -2], atol=1e-12)
    wrong = a[:SL].copy()
    wrong[0] = (wrong[0] + 1) % V
    r = oracle.verify(bits_of(W), bits_of(H), wrong, B=1, SL=SL)
    assert r.n_accept[0] == 0 and r.bonus[0] == a[0]


def test_ragged_equals_loop_of_single_calls_and_row_permutation(oracle):
    g = torch.Generator().manual_seed(22)
    V, d = 48, 16
    W = torch.randn(V, d, generator=g).to(torch.bfloat16)
    sl = torch.tensor([3, 0, 5, 1], dtype=torch.int32)
    off = inputs.row_offsets(sl).numpy()
    R = int(off[-1])
    H = torch.randn(R, d, generator=g).to(torch.bfloat16)
    a = np.argmax(H.double().numpy() @ W.double().numpy().T, axis=1).astype(np.int32)
    draft = np.concatenate([a[off[b]:off[b + 1] - 1] for b in range(4)]).astype(np.int32)
    draft[1] = (draft[1] + 7) % V                       # sequence 0: second token wrong
    rag = oracle.verify_ragged(bits_of(W), bits_of(H), draft, off)
    assert np.all(rag.n_accept >= 0) and np.all(rag.n_accept <= sl.numpy())
    assert list(rag.n_accept) == [1, 0, 5, 1]
    for b in range(4):
        one = oracle.verify(bits_of(W), bits_of(H[off[b]:off[b + 1]]), draft[off[b] - b: off[b + 1] - b - 1],
                            B=1, SL=int(sl[b]))
        assert one.n_accept[0] == rag.n_accept[b] and one.bonus[0] == rag.bonus[b]
    perm = torch.randperm(V, generator=g)
    inv = torch.empty_like(perm)
    inv[perm] = torch.arange(V)
    ragp = oracle.verify_ragged(bits_of(W[perm]), bits_of(H), inv.numpy()[draft].astype(np.int32), off)
    np.testing.assert_array_equal(ragp.n_accept, rag.n_accept)
    np.testing.assert_array_equal(perm.numpy()[ragp.bonus], rag.bonus)
    np.testing.assert_array_equal(perm.numpy()[ragp.target_ids], rag.target_ids)


def test_eq1_numerator_golden_and_sample_mean(oracle):
    for alpha, gamma, expected in _golden_pairs("eq1_expected_tokens.txt"):
        alpha, gamma, expected = float(alpha), int(gamma), float(expected)
        closed = (1 - alpha ** (gamma + 1)) / (1 - alpha)
        assert abs(closed - expected) < 1e-5
    # i.i.d. corruption with probability p per position: acceptance rate 1 - p (1 - 1/V)
    V, SL, p, N = 32000, 5, 0.2, 20000
    rng = np.random.default_rng(7)
    target = rng.integers(0, V, size=(N, SL + 1)).astype(np.int32)
    flat = inputs.corrupt_ids(torch.from_numpy(target[:, :SL].copy()), p, V, seed=9).numpy()
    emitted = np.array([oracle.accept_prefix(flat[i], target[i])[0] + 1 for i in range(N)])
    alpha = 1 - p * (1 - 1 / V)
    mean = (1 - alpha ** (SL + 1)) / (1 - alpha)
    sigma = emitted.std() / math.sqrt(N)
    assert abs(emitted.mean() - mean) < 3 * sigma + 1e-9
    assert abs(mean - 3.68928) < 1e-3              # Eq. 1 numerator at alpha = 0.8, gamma = 5


# ------------------------------------------------------------------ perplexity stopping rule (App. F)
def test_ppl_rule_uniform_distribution_has_perplexity_V(oracle):
    V, d = 50, 8
    W = bits_of(torch.randn(V, d, generator=torch.Generator().manual_seed(31)))
    h0 = bits_of(torch.zeros(1, d))
    nll = np.zeros(1)
    for n in (1, 2, 3):                       # every token of a uniform model costs ln V: perplexity V at any length
        tok, ppl, halt, gap, nll = oracle.draft_step_ppl(W, h0, [n], nll, ppl_max=V + 1.0, sl_max=10)
        assert tok[0] == 0 and abs(ppl[0] - V) < 1e-9 and halt[0] == 0
        assert abs(nll[0] - n * math.log(V)) < 1e-12
    tok, ppl, halt, gap, _ = oracle.draft_step_ppl(W, h0, [1], np.zeros(1), ppl_max=V - 1.0, sl_max=10)
    assert halt[0] == 1                       # perplexity above the bound: stop drafting
    tok, ppl, halt, gap, _ = oracle.draft_step_ppl(W, h0, [10], np.zeros(1), ppl_max=1e9, sl_max=10)
    assert halt[0] == 1                       # the cap still applies


def test_ppl_rule_is_geometric_mean_of_inverse_token_probabilities(oracle):
    from scipy.special import softmax as sp_softmax
    g = torch.Generator().manual_seed(32)
    V, d = 40, 12
    Wt = torch.randn(V, d, generator=g).to(torch.bfloat16)
    hs = torch.randn(3, d, generator=g).to(torch.bfloat16)
    nll = np.zeros(1)
    inv = []
    for n in range(1, 4):
        h = hs[n - 1:n]
        tok, ppl, halt, gap, nll = oracle.draft_step_ppl(bits_of(Wt), bits_of(h), [n], nll, 1e9, 10)
        y = sp_softmax(h.double().numpy() @ Wt.double().numpy().T, axis=1)[0]
        assert tok[0] == int(np.argmax(y))
        inv.append(1.0 / y.max())
        assert abs(ppl[0] - float(np.prod(inv)) ** (1.0 / n)) < 1e-9 * ppl[0]
    # a confident (peaked) step pulls the perplexity towards 1
    peaked = (Wt[5].float() * 50).to(torch.bfloat16).view(1, d)
    _, ppl1, _, _, _ = oracle.draft_step_ppl(bits_of(Wt), bits_of(peaked), [1], np.zeros(1), 1e9, 10)
    assert 1.0 <= ppl1[0] < 1.001


def test_ppl_rule_halts_monotonically_in_the_bound_and_skips_inactive(oracle):
    W, h, _ = _small_problem(33, B=3)
    nd = np.array([1, 2, 3], np.int32)
    halts = [oracle.draft_step_ppl(bits_of(W), bits_of(h), nd, np.zeros(3), bound, 9)[2] for bound in (40.0, 20.0, 5.0)]
    assert np.all(halts[0] <= halts[1]) and np.all(halts[1] <= halts[2])
    tok, ppl, halt, gap, nll = oracle.draft_step_ppl(bits_of(W), bits_of(h), nd, np.full(3, 0.25), 20.0, 9,
                                                     active=np.array([1, 0, 1], np.uint8))
    assert tok[1] == -1 and halt[1] == 255 and nll[1] == 0.25 and nll[0] > 0.25


# ------------------------------------------------------------------ sampling at temperature 1 (Table 6)
def test_sample_cdf_closed_forms(oracle):
    # uniform weights: token = floor(u * V), whatever the common scale of the weights
    V = 8
    for scale in (1.0, 0.125, 3.0):
        for u in (0.0, 0.1, 0.124, 0.126, 0.5, 0.874, 0.876, 0.9999):
            tok, total = oracle.sample_cdf(np.full(V, scale), u)
            assert tok == int(math.floor(u * V)) and abs(total - V * scale) < 1e-12
    # boundary convention: the running sum has to EXCEED u * total
    assert oracle.sample_cdf([0.5, 0.25, 0.25], 0.5)[0] == 1
    assert oracle.sample_cdf([0.5, 0.25, 0.25], 0.4999)[0] == 0
    assert oracle.sample_cdf([0.5, 0.25, 0.25], 0.75)[0] == 2
    # entries of weight zero are never drawn, not even at u = 0 or next to 1
    assert oracle.sample_cdf([0.0, 1.0, 0.0], 0.0)[0] == 1
    assert oracle.sample_cdf([0.0, 0.3, 0.0, 0.7, 0.0], 1.0 - 1e-17)[0] == 3
    assert oracle.sample_cdf([0.0, 0.0], 0.3)[0] == -1


def test_speculative_sampling_reproduces_the_target_distribution(oracle):
    """Brute force over a grid of the three uniforms (draft draw, acceptance, final draw): the token
    that position 0 ends up with is distributed as the target, which is the property the scheme is
    built for.  A wrong ratio, a missing clamp or a swapped residual shifts the histogram by far more
    than the grid's resolution."""
    yD = np.array([0.70, 0.10, 0.15, 0.05])
    yT = np.array([0.10, 0.20, 0.30, 0.40])
    N = 40
    grid = (np.arange(N) + 0.5) / N
    hist = np.zeros(4)
    accepted = 0
    for ud in grid:
        t, _ = oracle.sample_cdf(yD, ud)
        for ua in grid:
            for us in grid:
                n, nxt = oracle.speculative_sample(np.stack([yT, yT]), yD[None, :], [t], [ua], us)
                hist[t if n == 1 else nxt] += 1
                accepted += n
    hist /= N ** 3
    assert np.max(np.abs(hist - yT)) < 2.5 / N
    # acceptance rate = sum_v min(yD_v, yT_v) = 1 - total variation distance: computed here from the
    # histogram of accepted events only, not from the formula the oracle uses
    assert abs(accepted / N ** 3 - (1.0 - 0.5 * np.abs(yD - yT).sum())) < 2.5 / N


def test_speculative_identical_distributions_accept_everything(oracle):
    rng = np.random.default_rng(3)
    V, SL = 11, 4
    y = rng.dirichlet(np.ones(V), size=SL + 1)
    toks = rng.integers(0, V, size=SL)
    for trial in range(20):
        ua = rng.random(SL)
        us = float(rng.random())
        n, nxt = oracle.speculative_sample(y, y[:SL], toks, ua, us)
        assert n == SL
        assert nxt == oracle.sample_cdf(y[SL], us)[0]          # the extra token comes from the last target row


def test_speculative_residual_closed_form(oracle):
    # draft certain of token 0, target splits between 0 and 1: accepted with probability 1/2, and a
    # rejection can only ever be repaired with token 1
    yD = np.array([[1.0, 0.0, 0.0]])
    yT = np.array([[0.5, 0.5, 0.0], [0.2, 0.3, 0.5]])
    for us in (0.0, 0.3, 0.99):
        assert oracle.speculative_sample(yT, yD, [0], [0.6], us) == (0, 1)
        assert oracle.speculative_sample(yT, yD, [0], [0.5], us) == (0, 1)      # u * p_D < p_T is strict
    assert oracle.speculative_sample(yT, yD, [0], [0.4], 0.1) == (1, 0)         # accepted: next from row 1
    assert oracle.speculative_sample(yT, yD, [0], [0.4], 0.45) == (1, 1)
    assert oracle.speculative_sample(yT, yD, [0], [0.4], 0.55) == (1, 2)
    # a token the target gives no mass is rejected even at u = 0
    assert oracle.speculative_sample(yT, np.array([[0.0, 0.0, 1.0]]), [2], [0.0], 0.7)[0] == 0
    # SL = 0: nothing to accept, one draw from the single target row
    assert oracle.speculative_sample(yT[:1], np.zeros((0, 3)), [], [], 0.7) == (0, 1)


def test_verify_sample_with_sharp_distributions_is_greedy_verification(oracle):
    """As the distributions approach one-hot vectors the sampling scheme becomes the token-equality rule
    of Sec. 3: same n_accept and the same next token as the greedy oracle, for any uniforms."""
    rng = np.random.default_rng(9)
    V, d, B = 60, 48, 3
    sls = [3, 0, 4]
    row_off = np.concatenate([[0], np.cumsum([s + 1 for s in sls])]).astype(np.int32)
    R = int(row_off[-1])
    Wf = rng.normal(size=(V, d)).astype(np.float32)
    W = bits_of(torch.from_numpy(Wf))
    # each hidden row points along the LM-head row of one token: that token's logit towers over the rest
    H = bits_of(torch.from_numpy(20.0 * Wf[rng.integers(0, V, size=R)]))
    z = oracle.project(W, H)
    top = z.argmax(axis=1)
    srt = np.sort(z, axis=1)
    assert np.all(srt[:, -1] - srt[:, -2] > 40.0)             # softmax is one-hot to 1e-17
    ids = []
    for b in range(B):
        want = top[row_off[b]: row_off[b + 1] - 1].copy()
        if len(want) > 1:
            want[len(want) // 2] = (want[len(want) // 2] + 1) % V   # one mismatch in the middle
        ids.extend(want.tolist())
    ids = np.array(ids, dtype=np.int32)
    dp = np.zeros((max(sls), B, V), dtype=np.float32)
    for b in range(B):
        for i in range(sls[b]):
            dp[i, b, ids[row_off[b] - b + i]] = 1.0
    greedy = oracle.verify_ragged(W, H, ids, row_off)
    for trial in range(5):
        ua = rng.uniform(1e-6, 1 - 1e-6, size=R - B)
        us = rng.uniform(1e-6, 1 - 1e-6, size=B)
        res = oracle.verify_sample(W, H, ids, dp, row_off, ua, us)
        np.testing.assert_array_equal(res.n_accept, greedy.n_accept)
        np.testing.assert_array_equal(res.next_token, greedy.bonus)
    np.testing.assert_allclose(res.y_T.sum(axis=1), 1.0, atol=1e-12)


def test_verify_sample_is_the_per_sequence_rule_on_softmax_rows(oracle):
    """The batched call = softmax of the projected rows, step-major draft distributions gathered per
    sequence, and the one-sequence rule; checked with rows built here from project() and numpy."""
    rng = np.random.default_rng(21)
    V, d, B = 23, 8, 3
    sls = [2, 3, 1]
    row_off = np.concatenate([[0], np.cumsum([s + 1 for s in sls])]).astype(np.int32)
    R = int(row_off[-1])
    W = bits_of(torch.from_numpy(rng.normal(size=(V, d)).astype(np.float32)))
    H = bits_of(torch.from_numpy(rng.normal(size=(R, d)).astype(np.float32)))
    z = oracle.project(W, H)
    e = np.exp(z - z.max(axis=1, keepdims=True))
    yT = e / e.sum(axis=1, keepdims=True)
    dp = rng.dirichlet(np.ones(V), size=(max(sls), B)).astype(np.float32)
    ids = rng.integers(0, V, size=R - B).astype(np.int32)
    ua, us = rng.random(R - B), rng.random(B)
    res = oracle.verify_sample(W, H, ids, dp, row_off, ua, us)
    np.testing.assert_allclose(res.y_T, yT, atol=1e-14)
    for b in range(B):
        r0, sl = int(row_off[b]), sls[b]
        n, nxt = oracle.speculative_sample(yT[r0: r0 + sl + 1], dp[:sl, b].astype(np.float64),
                                           ids[r0 - b: r0 - b + sl], ua[r0 - b: r0 - b + sl], us[b])
        assert (res.n_accept[b], res.next_token[b]) == (n, nxt)


def test_draft_step_sample_differs_from_greedy_step_only_in_the_token(oracle):
    rng = np.random.default_rng(4)
    V, d, B, Hc = 97, 24, 4, 8
    W = bits_of(torch.from_numpy(rng.normal(size=(V, d)).astype(np.float32)))
    h = bits_of(torch.from_numpy(rng.normal(size=(B, d)).astype(np.float32)))
    clf = oracle.Classifier(rng.normal(size=(Hc, 12)).astype(np.float32), rng.normal(size=Hc).astype(np.float32),
                            rng.normal(size=Hc).astype(np.float32), np.array([0.1], dtype=np.float32))
    pos, nd = np.arange(B) + 5, np.array([1, 2, 3, 9])
    u = np.array([0.0, 0.3, 0.77, 0.999])
    act = np.array([1, 1, 0, 1], dtype=np.uint8)
    g = oracle.draft_step(W, h, pos, nd, clf, 0.5, 9, active=act, want_probs=True)
    s = oracle.draft_step_sample(W, h, pos, nd, clf, 0.5, 9, u, active=act)
    for b in range(B):
        if not act[b]:
            assert s.token[b] == -1 and np.isnan(s.p_token[b])
            continue
        np.testing.assert_array_equal(s.probs[b], g.probs[b])
        np.testing.assert_array_equal(s.feats[b], g.feats[b])
        assert s.conf[b] == g.conf[b] and s.halt[b] == g.halt[b]
        assert s.token[b] == oracle.sample_cdf(g.probs[b], u[b])[0]
        assert s.p_token[b] == g.probs[b, s.token[b]]
        cdf = np.cumsum(g.probs[b])
        assert cdf[s.token[b]] > u[b] * cdf[-1] - 1e-15 and (s.token[b] == 0 or cdf[s.token[b] - 1] <= u[b] * cdf[-1] + 1e-15)
    assert s.token[0] == int(np.argmax(g.probs[0] > 0))           # u = 0 draws the first token with mass


# ------------------------------------------------------------------ bulk feature extraction (App. D)
def test_total_variation_closed_forms_and_event_characterisation(oracle):
    assert oracle.total_variation([0.5, 0.5], [0.9, 0.1]) == pytest.approx(0.4, abs=1e-15)
    assert oracle.total_variation([0.2, 0.3, 0.5], [0.2, 0.3, 0.5]) == 0.0
    assert oracle.total_variation([1.0, 0.0, 0.0], [0.0, 0.0, 1.0]) == 1.0          # disjoint supports
    rng = np.random.default_rng(8)
    p, q = rng.dirichlet(np.ones(7)), rng.dirichlet(np.ones(7))
    tv = oracle.total_variation(p, q)
    assert tv == pytest.approx(oracle.total_variation(q, p), abs=1e-15)             # symmetric
    # TV is the largest difference in probability that the two distributions give to any event:
    # brute force over all 2^7 subsets of the vocabulary
    best = 0.0
    for mask in range(1 << 7):
        sel = [(mask >> v) & 1 == 1 for v in range(7)]
        best = max(best, abs(p[sel].sum() - q[sel].sum()))
    assert tv == pytest.approx(best, abs=1e-14)
    # and one minus the mass the two distributions share: checked against the acceptance rate that
    # the brute-force pin of speculative sampling measured for these two vectors
    yD, yT = np.array([0.70, 0.10, 0.15, 0.05]), np.array([0.10, 0.20, 0.30, 0.40])
    assert oracle.total_variation(yD, yT) == pytest.approx(0.6, abs=1e-15)


def test_extract_features_is_two_draft_steps_a_label_and_a_distance(oracle):
    rng = np.random.default_rng(12)
    V, dD, dT, N = 83, 16, 40, 6
    WD = bits_of(torch.from_numpy(rng.normal(size=(V, dD)).astype(np.float32)))
    WT = bits_of(torch.from_numpy(rng.normal(size=(V, dT)).astype(np.float32)))
    HD = bits_of(torch.from_numpy(rng.normal(size=(N, dD)).astype(np.float32)))
    HT = bits_of(torch.from_numpy(rng.normal(size=(N, dT)).astype(np.float32)))
    # make two positions agree by construction: both hidden states point along their head's row of one token
    for n, tok in ((1, 17), (4, 60)):
        HD[n] = bits_of(torch.tensor([6.0 * py_bf16(b) for b in WD[tok]], dtype=torch.float32))
        HT[n] = bits_of(torch.tensor([6.0 * py_bf16(b) for b in WT[tok]], dtype=torch.float32))
    pos = np.arange(N, dtype=np.int32) + 3
    res = oracle.extract_features(WD, HD, WT, HT, pos)
    clf = oracle.Classifier(np.zeros((4, 12), np.float32), np.zeros(4, np.float32), np.zeros(4, np.float32),
                            np.zeros(1, np.float32))
    dD_ = oracle.draft_step(WD, HD, pos, np.ones(N, np.int32), clf, 0.5, 9, want_probs=True)
    dT_ = oracle.draft_step(WT, HT, pos, np.ones(N, np.int32), clf, 0.5, 9, want_probs=True)
    np.testing.assert_array_equal(res.feats_D, dD_.feats)
    np.testing.assert_array_equal(res.feats_T, dT_.feats)
    np.testing.assert_array_equal(res.token_D, dD_.token)
    np.testing.assert_array_equal(res.token_T, dT_.token)
    np.testing.assert_array_equal(res.label, (dD_.token == dT_.token).astype(np.uint8))
    assert res.label[1] == 1 and res.label[4] == 1 and res.token_D[1] == 17 and res.token_T[4] == 60
    for n in range(N):
        assert res.tv[n] == pytest.approx(0.5 * np.abs(dD_.probs[n] - dT_.probs[n]).sum(), abs=1e-14)
        assert 0.0 <= res.tv[n] <= 1.0
    # the label is what greedy verification would decide for a one-token look-ahead at that position
    for n in range(N):
        v = oracle.verify_ragged(WT, HT[n:n + 1], np.zeros(0, np.int32), np.array([0, 1], np.int32))
        assert (v.bonus[0] == res.token_D[n]) == bool(res.label[n])


# ------------------------------------------------------------------ whole iteration (Sec. 3)
def _position_classifier(oracle, cut: float, H: int = 4):
    """A hand-made 2-layer classifier that looks at the position feature only:
    C = sigmoid(6 - 30 * relu(pos - cut)), i.e. about 0.998 up to pos = cut and below 1e-10 from cut + 1 on."""
    W1 = np.zeros((H, 12), np.float32)
    b1 = np.zeros(H, np.float32)
    w2 = np.zeros(H, np.float32)
    W1[0, 11] = 1.0
    b1[0] = -cut
    w2[0] = -30.0
    return oracle.Classifier(W1, b1, w2, np.array([6.0], np.float32))


def _iteration_inputs(V, dD, dT, B, S, seed):
    g = torch.Generator().manual_seed(seed)
    W_D = (torch.randn(V, dD, generator=g) * 0.3).to(torch.bfloat16)
    W_T = (torch.randn(V, dT, generator=g) * 0.3).to(torch.bfloat16)
    h_D = torch.randn(S, B, dD, generator=g).to(torch.bfloat16)
    H_T = torch.randn(B, S + 1, dT, generator=g).to(torch.bfloat16)
    bits = lambda t: inputs.bf16_bits(t.reshape(-1, t.shape[-1])).reshape(t.shape)
    return bits(W_D), bits(W_T), bits(h_D), bits(H_T)


def test_draft_loop_look_ahead_from_a_position_classifier(oracle):
    """With a classifier that only reads the position, the look-ahead is known in closed form: drafting
    stops at the first token whose position exceeds the cut, SL = clip(cut + 1 - pos0, 1, SL_max)."""
    V, dD, dT, B, S = 50, 16, 24, 5, 6
    W_D, W_T, h_D, H_T = _iteration_inputs(V, dD, dT, B, S, seed=1)
    pos0 = np.array([0, 3, 7, 9, 20], np.int32)
    clf = _position_classifier(oracle, cut=9.0)
    res = oracle.draft_loop(W_D, h_D, pos0, clf, 0.5, S)
    np.testing.assert_array_equal(res.sl, np.clip(9 + 1 - pos0, 1, S))     # [6, 6, 3, 1, 1]
    for b in range(B):
        n = res.sl[b]
        assert np.all(res.halt[: n - 1, b] == 0) and res.halt[n - 1, b] == 1   # halts exactly at its last token
        assert np.all(res.token[n:, b] == -1) and np.all(res.halt[n:, b] == 255)   # later steps never ran
        np.testing.assert_array_equal(res.feats[:n, b, 11], pos0[b] + np.arange(1, n + 1))  # position feature
        # each token is the plain single draft step on that hidden state
        for i in range(n):
            one = oracle.draft_step(W_D, h_D[i, b:b + 1], [pos0[b] + i + 1], [i + 1], clf, 0.5, S)
            assert one.token[0] == res.token[i, b] and one.conf[0] == res.conf[i, b]


def test_draft_loop_degenerate_policies(oracle):
    """tau <= 0 never halts before the cap (static SL = SL_max); tau > 1 halts after the first token; a
    forced look-ahead overrules the classifier but leaves its outputs in place."""
    V, dD, dT, B, S = 40, 8, 8, 3, 5
    W_D, W_T, h_D, H_T = _iteration_inputs(V, dD, dT, B, S, seed=2)
    W1, b1, w2, b2 = inputs.classifier_params(8, 3)
    clf = oracle.Classifier(W1.numpy(), b1.numpy(), w2.numpy(), b2.numpy())
    pos0 = np.array([4, 0, 11], np.int32)
    static = oracle.draft_loop(W_D, h_D, pos0, clf, 0.0, S)
    np.testing.assert_array_equal(static.sl, [S] * B)
    assert np.all(static.halt[: S - 1] == 0) and np.all(static.halt[S - 1] == 1)      # only the cap halts
    np.testing.assert_array_equal(oracle.draft_loop(W_D, h_D, pos0, clf, 1.5, S).sl, [1] * B)
    forced = oracle.draft_loop(W_D, h_D, pos0, clf, 1.5, S, sl_forced=[2, 9, 4])
    np.testing.assert_array_equal(forced.sl, [2, S, 4])                                # capped at SL_max
    np.testing.assert_array_equal(forced.token[:2, 0], static.token[:2, 0])            # same tokens either way
    assert np.all(forced.halt[:2, 0] == 1)                                             # tau > 1: the classifier said halt
    # the look-ahead cannot grow with the threshold
    sls = [oracle.draft_loop(W_D, h_D, pos0, clf, t, S).sl for t in (0.3, 0.5, 0.7)]
    assert np.all(sls[0] >= sls[1]) and np.all(sls[1] >= sls[2])


def test_iteration_equals_the_host_closed_loop(oracle):
    """The iteration is the loop a host would run with the single-step calls: draft steps until the halt
    flag, then one ragged verification of the rows and ids kept.  Bit for bit."""
    V, dD, dT, B, S = 64, 16, 24, 4, 5
    W_D, W_T, h_D, H_T = _iteration_inputs(V, dD, dT, B, S, seed=3)
    pos0 = np.array([2, 5, 6, 1], np.int32)
    clf = _position_classifier(oracle, cut=7.0)
    g = np.random.default_rng(3)
    for ids in (None, g.integers(0, V, size=(B, S)).astype(np.int32)):
        res = oracle.iteration(W_D, h_D, W_T, H_T, pos0, clf, 0.5, S, draft_ids=ids)
        # host closed loop
        active = np.ones(B, np.uint8)
        sl = np.zeros(B, np.int64)
        toks = np.full((S, B), -1, np.int32)
        for j in range(S):
            st = oracle.draft_step(W_D, h_D[j], pos0 + j + 1, np.full(B, j + 1, np.int32), clf, 0.5, S, active=active)
            toks[j, active == 1] = st.token[active == 1]
            sl[active == 1] = j + 1
            active = (active.astype(bool) & (st.halt != 1)).astype(np.uint8)
            if not active.any():
                break
        off = np.concatenate([[0], np.cumsum(sl + 1)]).astype(np.int32)
        rows = np.concatenate([H_T[b, : sl[b] + 1] for b in range(B)])
        offered = toks.T if ids is None else ids
        packed = np.concatenate([offered[b, : sl[b]] for b in range(B)]).astype(np.int32)
        v = oracle.verify_ragged(W_T, rows, packed, off)
        np.testing.assert_array_equal(res.sl, sl)
        np.testing.assert_array_equal(res.token, toks)
        np.testing.assert_array_equal(res.n_accept, v.n_accept)
        np.testing.assert_array_equal(res.bonus, v.bonus)
        for b in range(B):
            np.testing.assert_array_equal(res.target_ids[b, : sl[b] + 1], v.target_ids[off[b]:off[b + 1]])
            assert np.all(res.target_ids[b, sl[b] + 1:] == -1)


def test_iteration_reproduces_the_worked_example_of_fig1(oracle):
    """Fig. 1 through the whole iteration: the look-ahead comes out as 5 (position classifier), the target
    agrees with the first three offered tokens and not with the fourth: 3 accepted, 4 tokens emitted."""
    with open(os.path.join(GOLDEN, "fig1_iteration.txt")) as f:
        gold = dict(line.split() for line in f if line.strip() and not line.startswith("#"))
    SL, accepted, emitted = int(gold["SL"]), int(gold["accepted"]), int(gold["emitted"])
    V, dD, dT, S = 80, 16, 32, 8
    W_D, W_T, h_D, H_T = _iteration_inputs(V, dD, dT, 1, S, seed=4)
    clf = _position_classifier(oracle, cut=float(SL - 1))            # pos0 = 0: tokens 1..SL are drafted
    free = oracle.verify_padded(W_T, H_T, [S], np.zeros((1, S), np.int32), S, 1)[2][0]    # the target's own tokens
    ids = free[:S].copy().reshape(1, S)
    ids[0, accepted] = (ids[0, accepted] + 1) % V                    # t4 wrong
    ids[0, accepted + 1] = (ids[0, accepted + 1] + 1) % V            # t5 wrong
    res = oracle.iteration(W_D, h_D, W_T, H_T, [0], clf, 0.5, S, draft_ids=ids)
    assert res.sl[0] == SL and res.n_accept[0] == accepted and res.n_accept[0] + 1 == emitted
    assert res.bonus[0] == free[accepted]
    # offering the draft phase's own tokens instead: a random draft head agrees with nothing here
    own = oracle.iteration(W_D, h_D, W_T, H_T, [0], clf, 0.5, S)
    n = 0
    while n < SL and own.token[n, 0] == free[n]:
        n += 1
    assert own.n_accept[0] == n and own.bonus[0] == free[n]


def test_verify_padded_strides_and_unused_rows(oracle):
    """The padded layout gives what the packed one gives; rows beyond sl[b] do not matter; the two id
    layouts ([B, S] and step-major [S, B]) are read through their strides."""
    V, dD, dT, B, S = 30, 8, 16, 3, 4
    W_D, W_T, h_D, H_T = _iteration_inputs(V, dD, dT, B, S, seed=5)
    sl = np.array([4, 0, 2], np.int32)
    g = np.random.default_rng(5)
    free = oracle.verify_padded(W_T, H_T, [S] * B, np.zeros((B, S), np.int32), S, 1)[2]
    ids = free[:, :S].copy()
    ids[0, 3] = (ids[0, 3] + 1) % V
    n, bonus, tid, gap = oracle.verify_padded(W_T, H_T, sl, ids, S, 1)
    np.testing.assert_array_equal(n, [3, 0, 2])
    np.testing.assert_array_equal(bonus, [free[0, 3], free[1, 0], free[2, 2]])
    n2, bonus2, _, _ = oracle.verify_padded(W_T, H_T, sl, np.ascontiguousarray(ids.T), 1, B)   # step-major ids
    np.testing.assert_array_equal(n2, n)
    np.testing.assert_array_equal(bonus2, bonus)
    junk = H_T.copy()
    junk[1, 1:] = g.integers(0, 65535, size=junk[1, 1:].shape).astype(np.uint16) & 0x7F7F   # rows no sequence owns
    junk[2, 3:] = 0
    n3, bonus3, _, _ = oracle.verify_padded(W_T, junk, sl, ids, S, 1)
    np.testing.assert_array_equal(n3, n)
    np.testing.assert_array_equal(bonus3, bonus)
