"""Shared helpers of the GPU parity tests: run the C-ABI calls on torch tensors and compare with
the CPU oracle under the stated tolerances.

Tolerances
  * integer results (token, n_accept, bonus, halt, target ids) are bit-exact, except that a position
    whose two largest oracle logits are closer than GAP_EXEMPT may return either of the two;
  * probabilities, features and the classifier output agree within PROB_TOL absolute (fp32 accumulation
    over bf16 inputs against the fp64 oracle);
  * a halt flag may differ only if the oracle's C lies within HALT_MARGIN of tau.
"""
from __future__ import annotations

import numpy as np
import torch

from paper_2405_04304_b200 import binding, inputs

GAP_EXEMPT = 1e-3
PROB_TOL = 2e-3
HALT_MARGIN = 1e-4


def make_clf(H: int, seed: int, b2=None, zero_head: bool = False):
    W1, b1, w2, b2_ = inputs.classifier_params(H, seed)
    if zero_head:
        w2 = torch.zeros_like(w2)
        b2_ = torch.zeros_like(b2_)
    if b2 is not None:
        b2_ = torch.tensor([b2], dtype=torch.float32)
    return W1, b1, w2, b2_


def to_oracle_clf(oracle, params):
    W1, b1, w2, b2 = params
    return oracle.Classifier(W1.numpy(), b1.numpy(), w2.numpy(), b2.numpy())


def to_gpu_clf(params):
    return binding.Classifier(*(t.cuda() for t in params))


def gpu_draft_step(ctx, W, h, pos, nd, clf, tau, sl_max, active=None, want_probs=False, host=False):
    """Run disco_draft_step (or the _host variant).  W is a CUDA bf16 tensor; the rest CPU tensors."""
    B = h.shape[0]
    V = W.shape[0]
    pos = torch.as_tensor(pos, dtype=torch.int32)
    nd = torch.as_tensor(nd, dtype=torch.int32)
    act = None if active is None else torch.as_tensor(active, dtype=torch.uint8)
    if host:
        token = torch.full((B,), -7, dtype=torch.int32).pin_memory()
        conf = torch.full((B,), -7.0, dtype=torch.float32).pin_memory()
        halt = torch.full((B,), 77, dtype=torch.uint8).pin_memory()
        feats = torch.full((B, binding.NFEAT), -7.0, dtype=torch.float32).pin_memory()
        ctx.draft_step_host(W, h.contiguous().pin_memory(), pos.pin_memory(), nd.pin_memory(), clf, tau, sl_max,
                            token, conf, halt, active=None if act is None else act.pin_memory(), feats=feats)
        probs = None
    else:
        token = torch.full((B,), -7, dtype=torch.int32, device="cuda")
        conf = torch.full((B,), -7.0, dtype=torch.float32, device="cuda")
        halt = torch.full((B,), 77, dtype=torch.uint8, device="cuda")
        feats = torch.full((B, binding.NFEAT), -7.0, dtype=torch.float32, device="cuda")
        probs = torch.full((B, V), -7.0, dtype=torch.float32, device="cuda") if want_probs else None
        ctx.draft_step(W, h.cuda(), pos.cuda(), nd.cuda(), clf, tau, sl_max, token, conf, halt,
                       active=None if act is None else act.cuda(), feats=feats, probs=probs)
        torch.cuda.synchronize()
    return dict(token=token.cpu().numpy(), conf=conf.cpu().numpy(), halt=halt.cpu().numpy(),
                feats=feats.cpu().numpy(), probs=None if probs is None else probs.cpu().numpy())


def check_draft(got, ref, tau, active=None):
    """Compare a GPU draft step with the oracle's DraftStepResult; returns the number of exemptions."""
    B = ref.token.shape[0]
    exempt = 0
    for b in range(B):
        if active is not None and not active[b]:
            assert got["token"][b] == -7 and got["halt"][b] == 77 and got["conf"][b] == -7.0, \
                f"inactive sequence {b} was written"
            assert np.all(got["feats"][b] == -7.0)
            continue
        if ref.gap[b] < GAP_EXEMPT:
            exempt += 1
            assert got["token"][b] in ref.topk_ids[b, :2], f"seq {b}: token not among the tied top-2"
        else:
            assert got["token"][b] == ref.token[b], f"seq {b}: token {got['token'][b]} != {ref.token[b]}"
        np.testing.assert_allclose(got["feats"][b], ref.feats[b], rtol=0, atol=PROB_TOL,
                                   err_msg=f"features of sequence {b}")
        assert got["feats"][b, 11] == ref.feats[b, 11]          # the position is copied exactly
        assert abs(float(got["conf"][b]) - ref.conf[b]) <= PROB_TOL, f"seq {b}: conf"
        if abs(ref.conf[b] - tau) >= HALT_MARGIN:
            assert got["halt"][b] == ref.halt[b], f"seq {b}: halt {got['halt'][b]} != {ref.halt[b]}"
        if got["probs"] is not None:
            np.testing.assert_allclose(got["probs"][b], ref.probs[b], rtol=0, atol=PROB_TOL)
            assert abs(float(got["probs"][b].astype(np.float64).sum()) - 1.0) < 1e-4
    return exempt


def gpu_verify(ctx, W, H, draft_ids, B=None, SL=None, row_off=None, host=False, want_ids=True):
    """Run disco_verify / disco_verify_ragged (or the _host variant)."""
    R = H.shape[0]
    ids = torch.as_tensor(draft_ids, dtype=torch.int32)
    if row_off is not None:
        off = torch.as_tensor(row_off, dtype=torch.int32)
        B = off.numel() - 1
    dev = "cpu" if host else "cuda"
    n_acc = torch.full((B,), -7, dtype=torch.int32, device=dev)
    bonus = torch.full((B,), -7, dtype=torch.int32, device=dev)
    tids = torch.full((R,), -7, dtype=torch.int32, device=dev) if want_ids else None
    if host:
        n_acc, bonus = n_acc.pin_memory(), bonus.pin_memory()
        tids = None if tids is None else tids.pin_memory()
        if row_off is None:
            off = torch.arange(B + 1, dtype=torch.int32) * (SL + 1)
        ctx.verify_ragged_host(W, H.contiguous().pin_memory(), ids.pin_memory() if ids.numel() else None,
                               off.pin_memory(), B, R, n_acc, bonus, tids)
    elif row_off is None:
        ctx.verify(W, H.cuda(), ids.cuda() if ids.numel() else None, B, SL, n_acc, bonus, tids)
    else:
        ctx.verify_ragged(W, H.cuda(), ids.cuda() if ids.numel() else None, off.cuda(), B, R, n_acc, bonus, tids)
    torch.cuda.synchronize()
    return dict(n_accept=n_acc.cpu().numpy(), bonus=bonus.cpu().numpy(),
                target_ids=None if tids is None else tids.cpu().numpy())


def check_verify(got, ref, row_off, draft_ids):
    """Compare with the oracle's VerifyResult.  Rows whose top-2 gap is below GAP_EXEMPT may differ; a
    sequence with such a row at or before min(n_oracle, n_gpu) is checked for self-consistency only."""
    row_off = np.asarray(row_off)
    draft_ids = np.asarray(draft_ids)
    B = row_off.shape[0] - 1
    exempt = 0
    tid = got["target_ids"]
    for b in range(B):
        r0, r1 = int(row_off[b]), int(row_off[b + 1])
        sl = r1 - r0 - 1
        tied = ref.gap[r0:r1] < GAP_EXEMPT
        if tid is not None:
            same = tid[r0:r1] == ref.target_ids[r0:r1]
            assert np.all(same | tied), f"seq {b}: target ids differ on rows that are not near-ties"
        n_g, n_o = int(got["n_accept"][b]), int(ref.n_accept[b])
        assert 0 <= n_g <= sl
        lim = min(n_g, n_o)
        if np.any(tied[: lim + 1]):
            exempt += 1
            if tid is not None:   # still has to be the prefix rule applied to the ids it reported
                d = draft_ids[r0 - b: r0 - b + sl]
                n = 0
                while n < sl and d[n] == tid[r0 + n]:
                    n += 1
                assert n_g == n and got["bonus"][b] == tid[r0 + n]
            continue
        assert n_g == n_o, f"seq {b}: n_accept {n_g} != {n_o}"
        assert got["bonus"][b] == ref.bonus[b], f"seq {b}: bonus"
    return exempt
