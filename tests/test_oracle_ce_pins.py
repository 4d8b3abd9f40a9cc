"""Pins for the masked target cross-entropy oracle (loss appendix: masked average of CE over the
target-response span, on the logits of the output head).  Library cross-entropy on library logits,
closed forms, and the invariances the definition implies."""
import math

import numpy as np
import pytest
import torch

import oracle


def make(rng, N, Lr, Dm, V, p_mask=0.6):
    h = rng.standard_normal((N, Lr, Dm))
    w = rng.standard_normal((V, Dm)) / math.sqrt(Dm)
    t = rng.integers(0, V, size=(N, Lr)).astype(np.int32)
    m = (rng.random((N, Lr)) < p_mask).astype(np.float64)
    return h, w, t, m


@pytest.mark.parametrize("shape", [(3, 4, 8, 11), (2, 5, 16, 50), (4, 1, 4, 3)])
def test_equals_library_cross_entropy_on_library_logits(shape):
    rng = np.random.default_rng(51)
    h, w, t, m = make(rng, *shape)
    nll, lse, loss = oracle.target_ce_fwd(h, w, t, m)
    logits = torch.from_numpy(h) @ torch.from_numpy(w).T                      # [N,Lr,V]
    ce = torch.nn.functional.cross_entropy(logits.reshape(-1, shape[3]), torch.from_numpy(t).long().reshape(-1),
                                           reduction="none").reshape(shape[0], shape[1]).numpy()
    assert np.max(np.abs(nll - m * ce)) < 1e-12
    assert np.max(np.abs(lse - torch.logsumexp(logits, dim=-1).numpy())) < 1e-12
    den = m.sum(axis=1)
    ref = np.where(den > 0, (m * ce).sum(axis=1) / np.maximum(den, 1), 0.0)
    assert np.max(np.abs(loss - ref)) < 1e-12
    # the paper's scalar objective (masked average over everything) from the per-candidate parts
    if m.sum() > 0:
        total = (loss * den).sum() / m.sum()
        assert abs(total - (m * ce).sum() / m.sum()) < 1e-12


def test_zero_hidden_state_gives_uniform_distribution():
    N, Lr, Dm, V = 2, 3, 4, 7
    rng = np.random.default_rng(52)
    _, w, t, _ = make(rng, N, Lr, Dm, V)
    nll, lse, loss = oracle.target_ce_fwd(np.zeros((N, Lr, Dm)), w, t, np.ones((N, Lr)))
    assert np.max(np.abs(lse - math.log(V))) < 1e-14 and np.max(np.abs(nll - math.log(V))) < 1e-14
    assert np.max(np.abs(loss - math.log(V))) < 1e-14


def test_two_word_vocabulary_is_the_logistic_loss():
    h = np.array([[[1.5, -0.5]]])
    w = np.array([[2.0, 1.0], [-1.0, 3.0]])          # logits 2.5 and -3.0
    nll, lse, loss = oracle.target_ce_fwd(h, w, np.array([[1]]), np.ones((1, 1)))
    assert abs(nll[0, 0] - math.log1p(math.exp(5.5))) < 1e-13      # -ln sigmoid(-3.0 - 2.5)
    assert abs(loss[0] - nll[0, 0]) < 1e-15


def test_masked_positions_and_their_targets_do_not_matter():
    rng = np.random.default_rng(53)
    h, w, t, m = make(rng, 3, 5, 8, 13)
    m[1] = 0.0                                        # a candidate without any weighted position
    nll, lse, loss = oracle.target_ce_fwd(h, w, t, m)
    t2 = t.copy(); t2[m == 0] = -7                    # even an illegal token id is ignored where mask = 0
    h2 = h.copy(); h2[m == 0] *= 3.0                  # their hidden states change only their own lse
    nll2, lse2, loss2 = oracle.target_ce_fwd(h2, w, t2, m)
    assert np.array_equal(nll, nll2) and np.array_equal(loss, loss2) and loss[1] == 0.0
    assert np.array_equal(lse[m != 0], lse2[m != 0])
    assert not nll[m == 0].any()


def test_shifting_all_logits_of_a_row_changes_lse_only():
    """Adding a vector u to the hidden state with W u = c * 1 shifts every logit by c."""
    rng = np.random.default_rng(54)
    N, Lr, Dm, V = 2, 2, 6, 5
    h, w, t, m = make(rng, N, Lr, Dm, V, p_mask=1.0)
    w[:, 0] = 1.0                                     # then u = c * e_0 gives W u = c * 1
    u = np.zeros(Dm); u[0] = 2.25
    nll, lse, _ = oracle.target_ce_fwd(h, w, t, m)
    nll2, lse2, _ = oracle.target_ce_fwd(h + u, w, t, m)
    assert np.max(np.abs(lse2 - lse - 2.25)) < 1e-12 and np.max(np.abs(nll2 - nll)) < 1e-12


def test_vocabulary_permutation_and_candidate_permutation():
    rng = np.random.default_rng(55)
    h, w, t, m = make(rng, 4, 3, 8, 9)
    nll, lse, loss = oracle.target_ce_fwd(h, w, t, m)
    perm = rng.permutation(9)
    inv = np.argsort(perm)
    nll2, lse2, loss2 = oracle.target_ce_fwd(h, w[perm], inv[t].astype(np.int32), m)
    assert np.max(np.abs(nll2 - nll)) < 1e-12 and np.max(np.abs(lse2 - lse)) < 1e-12
    cp = [2, 0, 3, 1]
    nll3, _, loss3 = oracle.target_ce_fwd(h[cp], w, t[cp], m[cp])
    assert np.array_equal(nll3, nll[cp]) and np.array_equal(loss3, loss[cp])


def test_fractional_weights_scale_the_terms():
    rng = np.random.default_rng(56)
    h, w, t, _ = make(rng, 2, 4, 8, 6)
    ones = np.ones((2, 4))
    nll1, _, _ = oracle.target_ce_fwd(h, w, t, ones)
    wts = np.array([[0.5, 2.0, 0.0, 1.0], [1.0, 1.0, 1.0, 1.0]])
    nll, _, loss = oracle.target_ce_fwd(h, w, t, wts)
    assert np.max(np.abs(nll - wts * nll1)) < 1e-13
    assert np.max(np.abs(loss - (wts * nll1).sum(axis=1) / wts.sum(axis=1))) < 1e-13


def test_bad_arguments_are_rejected():
    rng = np.random.default_rng(57)
    h, w, t, m = make(rng, 2, 2, 4, 5, p_mask=1.0)
    t[0, 0] = 5
    with pytest.raises(RuntimeError):
        oracle.target_ce_fwd(h, w, t, m)
    with pytest.raises(ValueError):
        oracle.target_ce_fwd(h, w, t[:1], m)
