"""Pins for the float64 oracle: brute force, closed forms, invariants, finite
differences and library second opinions.  CPU only."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import grpo_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _golden(name):
    vals = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, v = line.split()
            vals[k] = float(v)
    return vals


def _rng(seed):
    return np.random.default_rng(seed)


# ----------------------------------------------------------------------------- softmax / logp
def test_logits_index_order_tiny():
    # z[t, j] = sum_k H[t,k] W[j,k], checked with python loops on a non-square case
    H = _rng(0).normal(size=(3, 5))
    W = _rng(1).normal(size=(7, 5))
    Z = O.logits(H, W)
    assert Z.shape == (3, 7)
    for t in range(3):
        for j in range(7):
            assert abs(Z[t, j] - sum(H[t, k] * W[j, k] for k in range(5))) < 1e-13


def test_softmax_bruteforce_no_shift():
    rng = _rng(2)
    for V in (2, 5, 16):
        Z = rng.normal(size=(4, V)) * 3.0
        lse, LP, ent = O.log_softmax_stats(Z)
        for t in range(4):
            denom = sum(math.exp(z) for z in Z[t])
            for j in range(V):
                p = math.exp(Z[t, j]) / denom
                assert abs(math.exp(LP[t, j]) - p) < 1e-13
            assert abs(lse[t] - math.log(denom)) < 1e-12
            naive_ent = -sum((math.exp(z) / denom) * math.log(math.exp(z) / denom) for z in Z[t])
            assert abs(ent[t] - naive_ent) < 1e-12


def test_softmax_invariants_and_bounds():
    rng = _rng(3)
    V = 37
    Z = rng.normal(size=(9, V)) * 5.0
    lse, LP, ent = O.log_softmax_stats(Z)
    assert np.allclose(np.exp(LP).sum(axis=1), 1.0, atol=1e-13)
    assert np.all(lse >= Z.max(axis=1)) and np.all(lse <= Z.max(axis=1) + math.log(V))
    assert np.all(LP <= 0)
    assert np.all(ent >= 0) and np.all(ent <= math.log(V) + 1e-12)
    # shift invariance: adding a constant to every logit of a row changes lse by it, nothing else
    lse2, LP2, ent2 = O.log_softmax_stats(Z + 7.25)
    assert np.allclose(lse2, lse + 7.25, atol=1e-12)
    assert np.allclose(LP2, LP, atol=1e-12) and np.allclose(ent2, ent, atol=1e-12)
    # large logits must not overflow
    lse3, _, _ = O.log_softmax_stats(Z + 900.0)
    assert np.all(np.isfinite(lse3))


def test_special_cases_uniform_and_dominant():
    T, d, V = 5, 8, 11
    H = _rng(4).normal(size=(T, d))
    tokens = _rng(5).integers(0, V, size=T)
    logp, ent, lse = O.token_logprobs(H, np.zeros((V, d)), tokens)
    assert np.allclose(logp, -math.log(V), atol=1e-14)
    assert np.allclose(ent, math.log(V), atol=1e-14)
    # one dominant logit: logp -> 0, entropy -> 0
    W = np.zeros((V, d))
    W[3, 0] = 50.0
    H1 = np.zeros((1, d))
    H1[0, 0] = 1.0
    logp, ent, _ = O.token_logprobs(H1, W, np.array([3]))
    assert abs(logp[0]) < 1e-20 + 1e-15 and ent[0] < 1e-18 + 1e-15


def test_token_logprobs_vs_torch_library():
    T, d, V = 12, 16, 50
    rng = _rng(6)
    H = rng.normal(size=(T, d))
    W = rng.normal(size=(V, d)) * 0.3
    tokens = rng.integers(0, V, size=T)
    mask = np.ones(T, dtype=np.uint8)
    mask[[2, 7]] = 0
    logp, ent, lse = O.token_logprobs(H, W, tokens, mask)
    Zt = torch.from_numpy(H) @ torch.from_numpy(W).T
    lp_t = -torch.nn.functional.cross_entropy(Zt, torch.from_numpy(tokens), reduction="none")
    ent_t = torch.distributions.Categorical(logits=Zt).entropy()
    m = mask.astype(bool)
    assert np.allclose(logp[m], lp_t.numpy()[m], atol=1e-12)
    assert np.allclose(ent[m], ent_t.numpy()[m], atol=1e-12)
    assert np.allclose(lse[m], torch.logsumexp(Zt, dim=1).numpy()[m], atol=1e-12)
    assert np.all(logp[~m] == 0) and np.all(ent[~m] == 0)


# ----------------------------------------------------------------------------- advantages
def test_advantages_mean0_std1():
    rng = _rng(7)
    for G in (4, 5, 8, 16):
        for ddof in (0, 1):
            r = rng.uniform(size=6 * G)
            a = O.grpo_advantages(r, G, ddof=ddof, eps_std=1e-6).reshape(6, G)
            rs = r.reshape(6, G)
            sig = rs.std(axis=1, ddof=ddof)
            assert np.allclose(a.mean(axis=1), 0.0, atol=1e-12)
            assert np.allclose(a.std(axis=1, ddof=ddof), sig / (sig + 1e-6), atol=1e-12)


def test_advantages_bernoulli_closed_form():
    # k ones among G: sigma^2 = (k/G)(1-k/G) * G/(G-ddof)
    for G in (4, 8, 16):
        for k in range(1, G):
            for ddof in (0, 1):
                r = np.array([1.0] * k + [0.0] * (G - k))
                a = O.grpo_advantages(r, G, ddof=ddof, eps_std=1e-6)
                sigma = math.sqrt((k / G) * (1 - k / G) * G / (G - ddof))
                assert np.allclose(a[:k], (1 - k / G) / (sigma + 1e-6), atol=1e-12)
                assert np.allclose(a[k:], (0 - k / G) / (sigma + 1e-6), atol=1e-12)
    # the worked case G=4, k=1, sample std: sigma = 0.5 -> {+1.5, -0.5, -0.5, -0.5} / (1 + 2e-6)
    a = O.grpo_advantages(np.array([1.0, 0, 0, 0]), 4)
    assert np.allclose(a, np.array([1.5, -0.5, -0.5, -0.5]) / (1 + 2e-6), atol=1e-12)


def test_advantages_zero_variance_affine_permutation():
    assert np.all(O.grpo_advantages(np.array([0.3, 0.3, 0.3, 1.0, 1.0, 1.0]), 3) == 0.0)
    rng = _rng(8)
    r = rng.normal(size=16)
    a = O.grpo_advantages(r, 8, eps_std=0.0)
    a2 = O.grpo_advantages(3.5 * r - 2.0, 8, eps_std=0.0)
    assert np.allclose(a, a2, atol=1e-12)
    perm = rng.permutation(8)
    r2 = r.copy()
    r2[:8] = r[:8][perm]
    a3 = O.grpo_advantages(r2, 8, eps_std=0.0)
    assert np.allclose(a3[:8], a[:8][perm], atol=1e-12)
    assert np.allclose(a3[8:], a[8:], atol=1e-12)       # groups do not interact
    with pytest.raises(ValueError):
        O.grpo_advantages(r, 1)
    with pytest.raises(ValueError):
        O.grpo_advantages(r, 5)


def test_other_estimators_closed_forms():
    rng = _rng(21)
    G = 5
    r = rng.normal(size=3 * G)
    # RLOO: leaving one out of the mean equals scaling the centred reward by G/(G-1)
    a = O.rloo_advantages(r, G)
    mu = np.repeat(r.reshape(-1, G).mean(axis=1), G)
    assert np.allclose(a, (r - mu) * G / (G - 1), atol=1e-13)
    assert np.allclose(a.reshape(-1, G).sum(axis=1), 0.0, atol=1e-13)
    assert np.allclose(O.rloo_advantages(np.array([1.0, 0.0]), 2), [1.0, -1.0])
    # OPO: with equal lengths the length-weighted baseline is the plain mean; one long response pulls it
    assert np.allclose(O.opo_advantages(r, np.full(3 * G, 7), G), r - mu, atol=1e-13)
    o = O.opo_advantages(np.array([1.0, 0.0, 0.0, 0.0]), np.array([30, 10, 10, 10]), 4)
    assert np.allclose(o, np.array([1.0, 0, 0, 0]) - 0.5, atol=1e-15)
    # the length-weighted sum of OPO advantages vanishes in every group
    ln = rng.integers(1, 50, size=3 * G)
    o = O.opo_advantages(r, ln, G)
    assert np.allclose((o * ln).reshape(-1, G).sum(axis=1), 0.0, atol=1e-12)
    # REINFORCE++: zero mean, unit (population) std over the batch; invariant to per-group shifts
    p = O.reinforce_pp_advantages(r, G, eps_std=0.0)
    assert abs(p.mean()) < 1e-13 and abs(p.std() - 1.0) < 1e-13
    shifted = r + np.repeat(np.array([3.0, -2.0, 10.0]), G)
    assert np.allclose(O.reinforce_pp_advantages(shifted, G, eps_std=0.0), p, atol=1e-12)
    with pytest.raises(ValueError):
        O.rloo_advantages(r, 1)


def test_broadcast_to_tokens():
    offs = np.array([0, 3, 3, 7])
    adv = O.broadcast_to_tokens(np.array([1.0, 2.0, -1.0]), offs, 9)
    assert adv.tolist() == [1, 1, 1, -1, -1, -1, -1, 0, 0]


# ----------------------------------------------------------------------------- clip / k3 / loss
def test_clip_branches_constructed():
    eps_lo, eps_hi = 0.2, 0.28
    old = np.zeros(6)
    rho = np.array([1.0, 1.5, 0.5, 1.0, 1.5, 0.5])
    adv = np.array([2.0, 2.0, 2.0, -2.0, -2.0, -2.0])
    s, k3, r, active, dlogp = O.per_token_terms(np.log(rho), old, old, adv, eps_lo, eps_hi, 0.0)
    # A>0: inside -> rho*A; above -> (1+eps_hi)*A clipped; below -> rho*A (unclipped is smaller)
    # A<0: inside -> rho*A; above -> rho*A (more negative); below -> (1-eps_lo)*A clipped
    assert np.allclose(s, [2.0, 1.28 * 2, 0.5 * 2, -2.0, -3.0, -0.8 * 2], atol=1e-14)
    assert active.tolist() == [True, False, True, True, True, False]
    assert np.allclose(dlogp, -adv * rho * active, atol=1e-14)
    assert np.all(k3 == 0)
    # the surrogate as literally printed differs only for A<0
    s_lit, *_ = O.per_token_terms(np.log(rho), old, old, adv, eps_lo, eps_hi, 0.0, literal_clip=True)
    assert np.allclose(s_lit[:3], s[:3], atol=1e-14)
    assert np.allclose(s_lit[3:], [-2.0, -1.28 * 2, -1.0], atol=1e-14)


def test_k3_properties():
    logp = np.array([-1.0, -2.0, -3.0, -0.5])
    ref = logp + np.array([0.0, 1e-4, -0.7, 1.3])
    _, k3, _, _, dlogp = O.per_token_terms(logp, logp, ref, np.zeros(4), 0.2, 0.2, 1.0)
    assert k3[0] == 0 and dlogp[0] == 0
    assert np.all(k3 >= 0)
    assert abs(k3[1] - 0.5e-8) < 1e-11                   # Taylor: delta^2/2
    d = ref - logp
    assert np.allclose(k3, np.exp(d) - d - 1, atol=1e-15)


def _tiny_problem(seed, T=6, d=8, V=16, masked=(4,)):
    rng = _rng(seed)
    H = rng.normal(size=(T, d))
    W = rng.normal(size=(V, d)) * 0.5
    tokens = rng.integers(0, V, size=T)
    mask = np.ones(T, dtype=np.uint8)
    for i in masked:
        mask[i] = 0
    logp, _, _ = O.token_logprobs(H, W, tokens)
    old = logp + rng.normal(size=T) * 0.3
    ref = logp + rng.normal(size=T) * 0.2
    adv = rng.normal(size=T)
    return H, W, tokens, old, ref, adv, mask


def test_two_token_worked_example():
    g = _golden("two_token_worked_example.txt")
    H = np.array([[1.0]])
    W = np.array([[0.0], [math.log(3.0)]])
    tok = np.array([1])
    m = np.array([1], dtype=np.uint8)
    old = np.array([math.log(0.5)])
    ref = np.array([math.log(0.375)])
    A = O.policy_loss_fwd_bwd(H, W, tok, old, ref, np.array([1.0]), m, 0.2, 0.2, 0.5)
    assert abs(A["logp"][0] - g["logp"]) < 1e-14 and abs(A["entropy"][0] - g["entropy"]) < 1e-14
    assert abs(A["rho"][0] - g["rho"]) < 1e-14 and abs(A["kl_mean"] - g["k3"]) < 1e-14
    assert abs(A["loss"] - g["A_loss"]) < 1e-14
    assert np.allclose(A["G"][0], [g["A_g0"], g["A_g1"]], atol=1e-14)
    assert abs(A["dH"][0, 0] - g["A_dH"]) < 1e-14
    assert np.allclose(A["dW"][:, 0], [g["A_g0"], g["A_g1"]], atol=1e-14)
    B = O.policy_loss_fwd_bwd(H, W, tok, old, ref, np.array([-1.0]), m, 0.2, 0.2, 0.5)
    assert abs(B["loss"] - g["B_loss"]) < 1e-14
    assert np.allclose(B["G"][0], [g["B_g0"], g["B_g1"]], atol=1e-14)
    Bl = O.policy_loss_fwd_bwd(H, W, tok, old, ref, np.array([-1.0]), m, 0.2, 0.2, 0.5, literal_clip=True)
    assert abs(Bl["loss"] - g["B_literal_loss"]) < 1e-14
    C = O.policy_loss_fwd_bwd(H, W, tok, old, ref, np.array([1.0]), m, 0.2, 0.2, 0.5, ent_coef=0.1)
    assert abs(C["loss"] - g["C_loss"]) < 1e-13
    assert np.allclose(C["G"][0], [g["C_g0"], g["C_g1"]], atol=1e-13)


def test_loss_identities():
    H, W, tokens, old, ref, adv, mask = _tiny_problem(10)
    logp, ent, _ = O.token_logprobs(H, W, tokens)
    w = O.token_weights(mask)
    assert abs(w.sum() - 1.0) < 1e-15 and w[4] == 0
    # on-policy (rho = 1), no regulariser: loss = - sum w_t A_t
    base = O.policy_loss_fwd_bwd(H, W, tokens, logp, None, adv, mask, 0.2, 0.2, 0.0)
    assert abs(base["loss"] + (w * adv).sum()) < 1e-14
    # switching beta / ent_coef on moves the loss by exactly beta*sum(w k3) / -c*sum(w Ent)
    d = ref - logp
    k3 = np.exp(d) - d - 1
    withkl = O.policy_loss_fwd_bwd(H, W, tokens, logp, ref, adv, mask, 0.2, 0.2, 0.04)
    assert abs(withkl["loss"] - base["loss"] - 0.04 * (w * k3).sum()) < 1e-14
    withent = O.policy_loss_fwd_bwd(H, W, tokens, logp, None, adv, mask, 0.2, 0.2, 0.0, ent_coef=1e-3)
    assert abs(withent["loss"] - base["loss"] + 1e-3 * (w * ent).sum()) < 1e-14
    # equal-length unpadded groups: group advantages sum to zero, so the on-policy loss is 0
    T = 8
    rng = _rng(11)
    Hh = rng.normal(size=(T, 4))
    Ww = rng.normal(size=(5, 4))
    tk = rng.integers(0, 5, size=T)
    lp, _, _ = O.token_logprobs(Hh, Ww, tk)
    a_seq = O.grpo_advantages(np.array([1.0, 0, 0, 1.0]), 4)
    a_tok = O.broadcast_to_tokens(a_seq, np.array([0, 2, 4, 6, 8]), T)
    out = O.policy_loss_fwd_bwd(Hh, Ww, tk, lp, None, a_tok, np.ones(T), 0.2, 0.2, 0.0)
    assert abs(out["loss"]) < 1e-14
    # empty batch
    e = O.policy_loss_fwd_bwd(H, W, tokens, old, ref, adv, np.zeros(6), 0.2, 0.2, 0.04)
    assert e["loss"] == 0 and not e["dH"].any() and not e["dW"].any()


# ----------------------------------------------------------------------------- gradients
def test_gradient_closed_form_on_policy():
    # Eq. 3: at rho = 1, no clipping, beta = 0 the gradient is the advantage-weighted
    # score function: g_tj = -w_t A_t (1[j=y_t] - p_tj)
    H, W, tokens, old, ref, adv, mask = _tiny_problem(12)
    logp, _, _ = O.token_logprobs(H, W, tokens)
    out = O.policy_loss_fwd_bwd(H, W, tokens, logp, None, adv, mask, 0.2, 0.2, 0.0)
    w = O.token_weights(mask)
    rows = np.nonzero(mask)[0]
    Z = H[rows] @ W.T
    P = np.exp(Z) / np.exp(Z).sum(axis=1, keepdims=True)
    onehot = np.eye(W.shape[0])[tokens[rows]]
    G = -(w[rows] * adv[rows])[:, None] * (onehot - P)
    assert np.allclose(out["G"], G, atol=1e-14)
    dH = np.zeros_like(H)
    dH[rows] = G @ W
    assert np.allclose(out["dH"], dH, atol=1e-14)
    assert np.allclose(out["dW"], G.T @ H[rows], atol=1e-14)


@pytest.mark.parametrize("beta,ent_coef,eps", [(0.0, 0.0, (0.2, 0.2)), (0.3, 0.0, (0.2, 0.2)),
                                               (0.0, 0.05, (0.2, 0.28)), (0.3, 0.05, (0.2, 0.28)),
                                               (0.3, 0.05, (10.0, 10.0))])
def test_gradient_finite_differences(beta, ent_coef, eps):
    H, W, tokens, old, ref, adv, mask = _tiny_problem(13)
    kw = dict(eps_low=eps[0], eps_high=eps[1], beta=beta, ent_coef=ent_coef)
    refp = ref if beta != 0 else None
    out = O.policy_loss_fwd_bwd(H, W, tokens, old, refp, adv, mask, **kw)
    # the problem must exercise both clipped and unclipped tokens when eps is small
    if eps[0] < 1:
        assert out["active"].any() and (~out["active"]).any()

    def loss(Hx, Wx):
        return O.policy_loss_fwd_bwd(Hx, Wx, tokens, old, refp, adv, mask, **kw)["loss"]

    h = 1e-6
    for (X, dX, which) in ((H, out["dH"], 0), (W, out["dW"], 1)):
        num = np.zeros_like(X)
        for idx in np.ndindex(*X.shape):
            Xp = X.copy(); Xp[idx] += h
            Xm = X.copy(); Xm[idx] -= h
            num[idx] = ((loss(Xp, W) - loss(Xm, W)) if which == 0 else (loss(H, Xp) - loss(H, Xm))) / (2 * h)
        denom = max(np.abs(num).max(), 1e-12)
        assert np.abs(num - dX).max() / denom < 1e-6


def test_gradient_vs_torch_autograd():
    H, W, tokens, old, ref, adv, mask = _tiny_problem(14, T=10, d=6, V=20, masked=(1, 8))
    eps_lo, eps_hi, beta, c_ent = 0.2, 0.28, 0.04, 0.01
    out = O.policy_loss_fwd_bwd(H, W, tokens, old, ref, adv, mask, eps_lo, eps_hi, beta, ent_coef=c_ent)
    Ht = torch.tensor(H, requires_grad=True)
    Wt = torch.tensor(W, requires_grad=True)
    m = torch.tensor(mask.astype(np.float64))
    lsm = torch.log_softmax(Ht @ Wt.T, dim=1)
    lp = lsm.gather(1, torch.tensor(tokens)[:, None])[:, 0]
    ent = -(lsm.exp() * lsm).sum(1)
    ratio = (lp - torch.tensor(old)).exp()
    A = torch.tensor(adv)
    s = torch.minimum(ratio * A, ratio.clamp(1 - eps_lo, 1 + eps_hi) * A)
    dl = torch.tensor(ref) - lp
    lt = -s + beta * (dl.exp() - dl - 1) - c_ent * ent
    L = (lt * m).sum() / m.sum()
    L.backward()
    assert abs(L.item() - out["loss"]) < 1e-13
    assert np.allclose(Ht.grad.numpy(), out["dH"], atol=1e-13)
    assert np.allclose(Wt.grad.numpy(), out["dW"], atol=1e-13)


def test_gradient_identities():
    H, W, tokens, old, ref, adv, mask = _tiny_problem(15, T=9, d=5, V=13, masked=(0,))
    out = O.policy_loss_fwd_bwd(H, W, tokens, old, ref, adv, mask, 0.2, 0.2, 0.04, ent_coef=0.02)
    assert np.allclose(out["G"].sum(axis=1), 0.0, atol=1e-15)        # softmax gradient rows sum to 0
    assert np.allclose(out["dW"].sum(axis=0), 0.0, atol=1e-14)
    assert abs((out["dH"] * H).sum() - (out["dW"] * W).sum()) < 1e-13  # both equal sum g_tj z_tj
    assert not out["dH"][0].any()


def test_custom_token_weight_and_sampled_helpers():
    H, W, tokens, old, ref, adv, mask = _tiny_problem(16, T=9, d=5, V=13, masked=(3,))
    rng = _rng(17)
    tw = rng.uniform(size=9)
    kw = dict(eps_low=0.2, eps_high=0.28, beta=0.04, ent_coef=0.02)
    out = O.policy_loss_fwd_bwd(H, W, tokens, old, ref, adv, mask, token_weight=tw, **kw)
    # linearity in the weights: sum over single-token problems
    acc = 0.0
    for t in np.nonzero(mask)[0]:
        one = np.zeros(9); one[t] = 1
        acc += tw[t] * O.policy_loss_fwd_bwd(H, W, tokens, old, ref, adv, one, **kw)["loss"]
    assert abs(acc - out["loss"]) < 1e-13
    rows = np.nonzero(mask)[0]
    w = tw * mask
    sub = rows[[1, 4, 6]]
    r = O.dH_rows(H[sub], W, tokens[sub], old[sub], ref[sub], adv[sub], w[sub], **kw)
    assert np.allclose(r["dH"], out["dH"][sub], atol=1e-14)
    assert np.allclose(r["logp"], out["logp"][sub], atol=1e-14)
    sel = np.array([0, 5, 12, int(tokens[rows[0]])])
    _, _, _, _, dlogp = O.per_token_terms(out["logp"][rows], old[rows], ref[rows], adv[rows], 0.2, 0.28, 0.04)
    dWs = O.dW_rows(H[rows], W[sel], sel, tokens[rows], out["lse"][rows], out["entropy"][rows],
                    w[rows] * dlogp, w[rows] * 0.02)
    assert np.allclose(dWs, out["dW"][sel], atol=1e-14)


# ----------------------------------------------------------------------------- aggregation / sequence level
def test_aggregation_weights():
    mask = np.array([1, 1, 0, 1, 0, 0, 1, 1, 1], dtype=np.uint8)
    off = np.array([0, 3, 6, 9])
    w0 = O.aggregation_weights(mask, off, 0)
    assert np.allclose(w0, mask / 6.0)
    w1 = O.aggregation_weights(mask, off, 1)
    assert np.allclose(w1, [1 / 6, 1 / 6, 0, 1 / 3, 0, 0, 1 / 9, 1 / 9, 1 / 9])
    assert abs(w1.sum() - 1.0) < 1e-15                      # every sequence has a valid token
    w2 = O.aggregation_weights(mask, off, 2)
    assert np.allclose(w2, mask / 9.0)
    # equal, fully valid sequences: the three modes coincide
    full = np.ones(12)
    offs = np.array([0, 4, 8, 12])
    for mode in (1, 2):
        assert np.allclose(O.aggregation_weights(full, offs, mode), O.aggregation_weights(full, offs, 0))
    # a sequence without valid tokens contributes nothing
    assert np.allclose(O.aggregation_weights(np.array([1, 1, 0, 0]), np.array([0, 2, 4]), 1), [0.25, 0.25, 0, 0])


def test_sequence_ratio_is_geometric_mean():
    logp = np.log(np.array([0.5, 0.25, 0.1, 0.2]))
    old = np.log(np.array([0.25, 0.25, 0.2, 0.2]))
    rho, ln = O.sequence_ratio(logp, old, np.array([1, 1, 1, 0]), np.array([0, 2, 4]))
    assert np.allclose(rho, [math.sqrt(2.0 * 1.0), math.sqrt(2.0), 0.5, 1.0]) and ln.tolist() == [2, 2, 1, 0]


@pytest.mark.parametrize("agg_mode", [0, 1, 2])
def test_sequence_level_gradient_finite_differences_and_autograd(agg_mode):
    rng = _rng(31)
    T, d, V = 9, 6, 12
    off = np.array([0, 4, 5, 9])
    H = rng.normal(size=(T, d))
    W = rng.normal(size=(V, d)) * 0.5
    tokens = rng.integers(0, V, size=T)
    mask = np.array([1, 1, 0, 1, 1, 1, 1, 1, 0], dtype=np.uint8)
    lp, _, _ = O.token_logprobs(H, W, tokens)
    old = lp + rng.normal(size=T) * 0.4
    ref = lp + rng.normal(size=T) * 0.2
    adv = rng.normal(size=T)
    kw = dict(eps_low=0.15, eps_high=0.2, beta=0.1, ent_coef=0.02, seq_offsets=off, agg_mode=agg_mode,
              sequence_level=True)
    out = O.policy_loss_fwd_bwd(H, W, tokens, old, ref, adv, mask, **kw)
    assert out["active"].any() and (~out["active"]).any()

    def loss(Hx, Wx):
        return O.policy_loss_fwd_bwd(Hx, Wx, tokens, old, ref, adv, mask, **kw)["loss"]

    h = 1e-6
    for (X, dX, which) in ((H, out["dH"], 0), (W, out["dW"], 1)):
        num = np.zeros_like(X)
        for idx in np.ndindex(*X.shape):
            Xp = X.copy(); Xp[idx] += h
            Xm = X.copy(); Xm[idx] -= h
            num[idx] = ((loss(Xp, W) - loss(Xm, W)) if which == 0 else (loss(H, Xp) - loss(H, Xm))) / (2 * h)
        assert np.abs(num - dX).max() / max(np.abs(num).max(), 1e-12) < 1e-6
    # library second opinion: float64 autograd of the sequence-level objective
    Ht = torch.tensor(H, requires_grad=True)
    Wt = torch.tensor(W, requires_grad=True)
    lsm = torch.log_softmax(Ht @ Wt.T, dim=1)
    lpt = lsm.gather(1, torch.tensor(tokens)[:, None])[:, 0]
    ent = -(lsm.exp() * lsm).sum(1)
    mt = torch.tensor(mask.astype(np.float64))
    wt = torch.tensor(O.aggregation_weights(mask, off, agg_mode))
    total = 0.0
    for i in range(3):
        sl = slice(off[i], off[i + 1])
        mi = mt[sl]
        ratio = (((lpt[sl] - torch.tensor(old[sl])) * mi).sum() / mi.sum()).exp()
        A = torch.tensor(adv[sl])
        s = torch.minimum(ratio * A, ratio.clamp(1 - 0.15, 1 + 0.2) * A)
        dl = torch.tensor(ref[sl]) - lpt[sl]
        total = total + (wt[sl] * (-s + 0.1 * (dl.exp() - dl - 1) - 0.02 * ent[sl])).sum()
    total.backward()
    assert abs(total.item() - out["loss"]) < 1e-13
    assert np.allclose(Ht.grad.numpy(), out["dH"], atol=1e-13) and np.allclose(Wt.grad.numpy(), out["dW"], atol=1e-13)


def test_sequence_level_reduces_to_token_level_for_single_token_sequences():
    H, W, tokens, old, ref, adv, mask = _tiny_problem(33, T=6, d=8, V=16, masked=())
    off = np.arange(7)
    a = O.policy_loss_fwd_bwd(H, W, tokens, old, ref, adv, mask, 0.2, 0.2, 0.04, seq_offsets=off, sequence_level=True)
    b = O.policy_loss_fwd_bwd(H, W, tokens, old, ref, adv, mask, 0.2, 0.2, 0.04)
    assert abs(a["loss"] - b["loss"]) < 1e-15 and np.allclose(a["dH"], b["dH"], atol=1e-15)
    assert np.allclose(a["dW"], b["dW"], atol=1e-15)


# ----------------------------------------------------------------------------- full-distribution KL
def test_full_kl_values():
    rng = _rng(41)
    Z = rng.normal(size=(5, 9))
    Zr = rng.normal(size=(5, 9))
    _, LP, ent = O.log_softmax_stats(Z)
    _, LQ, _ = O.log_softmax_stats(Zr)
    kl = O.full_kl(LP, LQ)
    for t in range(5):
        p = np.exp(Z[t]) / np.exp(Z[t]).sum()
        q = np.exp(Zr[t]) / np.exp(Zr[t]).sum()
        assert abs(kl[t] - sum(p[j] * math.log(p[j] / q[j]) for j in range(9))) < 1e-13
    assert np.all(kl >= 0)
    assert np.allclose(O.full_kl(LP, LP), 0.0, atol=1e-15)
    _, LU, _ = O.log_softmax_stats(np.zeros((5, 9)))
    assert np.allclose(O.full_kl(LP, LU), math.log(9) - ent, atol=1e-13)       # uniform reference
    ref = torch.nn.functional.kl_div(torch.tensor(LQ), torch.tensor(LP), log_target=True, reduction="none").sum(1)
    assert np.allclose(kl, ref.numpy(), atol=1e-13)                             # library second opinion


def test_full_kl_loss_and_gradient():
    rng = _rng(42)
    T, d, dr, V = 7, 6, 5, 11
    H = rng.normal(size=(T, d)); W = rng.normal(size=(V, d)) * 0.6
    Hr = rng.normal(size=(T, dr)); Wr = rng.normal(size=(V, dr)) * 0.6
    tokens = rng.integers(0, V, size=T)
    mask = np.array([1, 1, 0, 1, 1, 1, 1], dtype=np.uint8)
    lp, _, _ = O.token_logprobs(H, W, tokens)
    old = lp + rng.normal(size=T) * 0.3
    adv = rng.normal(size=T)
    kw = dict(eps_low=0.2, eps_high=0.2, beta=0.3, ent_coef=0.02, H_ref=Hr, W_ref=Wr)
    out = O.policy_loss_fwd_bwd(H, W, tokens, old, None, adv, mask, **kw)
    base = O.policy_loss_fwd_bwd(H, W, tokens, old, None, adv, mask, 0.2, 0.2, 0.0, ent_coef=0.02)
    w = O.token_weights(mask)
    Z, Zr = H @ W.T, Hr @ Wr.T
    _, LP, _ = O.log_softmax_stats(Z)
    _, LQ, _ = O.log_softmax_stats(Zr)
    assert abs(out["loss"] - base["loss"] - 0.3 * (w * O.full_kl(LP, LQ)).sum()) < 1e-14
    # same policy and reference: the KL term and its gradient vanish
    same = O.policy_loss_fwd_bwd(H, W, tokens, old, None, adv, mask, 0.2, 0.2, 0.3, ent_coef=0.02, H_ref=H, W_ref=W)
    assert abs(same["loss"] - base["loss"]) < 1e-14 and np.allclose(same["dH"], base["dH"], atol=1e-15)

    def loss(Hx, Wx):
        return O.policy_loss_fwd_bwd(Hx, Wx, tokens, old, None, adv, mask, **kw)["loss"]

    h = 1e-6
    for (X, dX, which) in ((H, out["dH"], 0), (W, out["dW"], 1)):
        num = np.zeros_like(X)
        for idx in np.ndindex(*X.shape):
            Xp = X.copy(); Xp[idx] += h
            Xm = X.copy(); Xm[idx] -= h
            num[idx] = ((loss(Xp, W) - loss(Xm, W)) if which == 0 else (loss(H, Xp) - loss(H, Xm))) / (2 * h)
        assert np.abs(num - dX).max() / max(np.abs(num).max(), 1e-12) < 1e-6
    Ht = torch.tensor(H, requires_grad=True); Wt = torch.tensor(W, requires_grad=True)
    lsm = torch.log_softmax(Ht @ Wt.T, dim=1)
    lq = torch.log_softmax(torch.tensor(Hr) @ torch.tensor(Wr).T, dim=1)
    lpt = lsm.gather(1, torch.tensor(tokens)[:, None])[:, 0]
    ratio = (lpt - torch.tensor(old)).exp()
    A = torch.tensor(adv)
    s = torch.minimum(ratio * A, ratio.clamp(0.8, 1.2) * A)
    kl = (lsm.exp() * (lsm - lq)).sum(1)
    ent = -(lsm.exp() * lsm).sum(1)
    L = ((-s + 0.3 * kl - 0.02 * ent) * torch.tensor(w)).sum()
    L.backward()
    assert abs(L.item() - out["loss"]) < 1e-13
    assert np.allclose(Ht.grad.numpy(), out["dH"], atol=1e-13) and np.allclose(Wt.grad.numpy(), out["dW"], atol=1e-13)
    # the sampled-row helper agrees with autograd on a subset of rows, and returns KL_t itself
    sub = np.array([1, 4, 6])
    r = O.dH_rows(H[sub], W, tokens[sub], old[sub], None, adv[sub], w[sub], 0.2, 0.2, 0.3, ent_coef=0.02,
                  H_ref_rows=Hr[sub], W_ref=Wr)
    assert np.allclose(r["dH"], Ht.grad.numpy()[sub], atol=1e-13)
    assert np.allclose(r["kl"], kl.detach().numpy()[sub], atol=1e-13)


# ----------------------------------------------------------------------------- vocabulary-parallel head
def _shard_problem(seed):
    rng = _rng(seed)
    T, d, V = 9, 6, 23
    H = rng.normal(size=(T, d)); W = rng.normal(size=(V, d)) * 0.8
    tokens = rng.integers(0, V, size=T)
    tokens[0], tokens[1] = 0, V - 1                      # first and last id of the vocabulary
    mask = np.array([1, 1, 1, 0, 1, 1, 0, 1, 1], dtype=np.uint8)
    lp, _, _ = O.token_logprobs(H, W, tokens)
    old = lp + rng.normal(size=T) * 0.3
    ref = lp + rng.normal(size=T) * 0.2
    adv = rng.normal(size=T)
    return H, W, tokens, mask, old, ref, adv


def test_shard_statistics_brute_force():
    # one slice, tiny: the four numbers against python sums without any shift
    H, W, tokens, mask, *_ = _shard_problem(50)
    off, Vs = 5, 7
    st = O.shard_logit_stats(H, W[off:off + Vs], tokens, off, mask)
    for t in range(H.shape[0]):
        if not mask[t]:
            assert np.all(st[t] == 0)
            continue
        z = [sum(H[t, k] * W[off + j, k] for k in range(H.shape[1])) for j in range(Vs)]
        M, S, A, zy = st[t]
        assert abs(M - max(z)) < 1e-14
        assert abs(S * math.exp(M) - sum(math.exp(v) for v in z)) < 1e-12
        assert abs(A * math.exp(M) - sum(math.exp(v) * v for v in z)) < 1e-12
        inside = off <= tokens[t] < off + Vs
        assert abs(zy - (z[tokens[t] - off] if inside else 0.0)) < 1e-14


@pytest.mark.parametrize("cuts", [(0, 23), (0, 11, 23), (0, 1, 22, 23), (0, 4, 9, 17, 23)])
def test_merged_shard_statistics_equal_the_full_softmax(cuts):
    # any partition of the vocabulary reproduces the single-device definition (one slice: trivially)
    H, W, tokens, mask, *_ = _shard_problem(51)
    stats = [O.shard_logit_stats(H, W[a:b], tokens, a, mask) for a, b in zip(cuts[:-1], cuts[1:])]
    logp, ent, lse = O.merge_logit_stats(stats, mask)
    lp0, ent0, lse0 = O.token_logprobs(H, W, tokens, mask)
    assert np.abs(logp - lp0).max() < 1e-13 and np.abs(ent - ent0).max() < 1e-13 and np.abs(lse - lse0).max() < 1e-13
    # library second opinion on the merged result
    ref = -torch.nn.functional.cross_entropy(torch.tensor(H @ W.T), torch.tensor(tokens), reduction="none").numpy()
    assert np.abs(logp - ref * mask).max() < 1e-13
    # a slice whose logits are far below the others' must not disturb the sums (shift by the largest M)
    Wlow = W.copy(); Wlow[cuts[-2]:] *= 0.0; Hs = H * 30.0
    stats = [O.shard_logit_stats(Hs, Wlow[a:b], tokens, a, mask) for a, b in zip(cuts[:-1], cuts[1:])]
    lp1, ent1, lse1 = O.merge_logit_stats(stats, mask)
    lp2, ent2, lse2 = O.token_logprobs(Hs, Wlow, tokens, mask)
    assert np.all(np.isfinite(lp1)) and np.abs(lp1 - lp2).max() < 1e-10 and np.abs(ent1 - ent2).max() < 1e-10


@pytest.mark.parametrize("cuts", [(0, 23), (0, 10, 23), (0, 1, 8, 23)])
def test_shard_backward_sums_to_the_full_gradient(cuts):
    H, W, tokens, mask, old, ref, adv = _shard_problem(52)
    kw = dict(eps_low=0.2, eps_high=0.3, beta=0.1, ent_coef=0.03)
    full = O.policy_loss_fwd_bwd(H, W, tokens, old, ref, adv, mask, **kw)
    dH = np.zeros_like(H)
    for a, b in zip(cuts[:-1], cuts[1:]):
        o = O.policy_loss_shard_bwd(H, W[a:b], tokens, a, full["logp"], full["entropy"], full["lse"], old, ref, adv,
                                    mask, **kw)
        assert abs(o["loss"] - full["loss"]) < 1e-14                 # every slice sees the same loss
        assert np.abs(o["dW_shard"] - full["dW"][a:b]).max() < 1e-13  # its rows of dW
        dH += o["dH_partial"]
    assert np.abs(dH - full["dH"]).max() < 1e-13
    assert np.all(dH[mask == 0] == 0)
    # caller-supplied weights take the place of the token mean
    tw = np.linspace(0.5, 1.5, H.shape[0]) / 7.0
    full = O.policy_loss_fwd_bwd(H, W, tokens, old, ref, adv, mask, token_weight=tw, **kw)
    o = O.policy_loss_shard_bwd(H, W[3:15], tokens, 3, full["logp"], full["entropy"], full["lse"], old, ref, adv,
                                mask, token_weight=tw, **kw)
    assert np.abs(o["dW_shard"] - full["dW"][3:15]).max() < 1e-13 and abs(o["loss"] - full["loss"]) < 1e-14


# ----------------------------------------------------------------------------- padding-free row map
def test_valid_row_map():
    assert O.valid_row_map([0, 3, 0, 1, 255, 0]) == [1, 3, 4]          # any non-zero byte counts
    assert O.valid_row_map([]) == [] and O.valid_row_map([0, 0]) == [] and O.valid_row_map(None, 3) == [0, 1, 2]
    m = (_rng(60).uniform(size=1000) < 0.3).astype(np.uint8)
    rm = O.valid_row_map(m)
    assert rm == sorted(rm) and len(rm) == int(m.sum()) and all(m[t] for t in rm)
    assert rm == np.flatnonzero(m).tolist()                             # library second opinion
    # the compacted rows are what the masked functions work on: same log-probs either way
    H = _rng(61).normal(size=(12, 4)); W = _rng(62).normal(size=(7, 4)); tok = _rng(63).integers(0, 7, size=12)
    mk = np.array([1, 0, 1, 1, 0, 0, 1, 0, 1, 1, 0, 1], dtype=np.uint8)
    idx = O.valid_row_map(mk)
    lp_masked, _, _ = O.token_logprobs(H, W, tok, mk)
    lp_compact, _, _ = O.token_logprobs(H[idx], W, tok[idx])
    assert np.array_equal(lp_masked[idx], lp_compact)


# ----------------------------------------------------------------------------- token-level KL reward shaping
def _shaping_case():
    ln = math.log
    logp = np.array([ln(0.5), -7.0, ln(0.25), ln(0.5)])
    ref = np.array([ln(0.25), 3.0, ln(0.25), ln(1.0)])
    mask = np.array([1, 0, 1, 1], dtype=np.uint8)
    return logp, ref, mask, np.array([0, 4]), np.array([2.0])


def test_kl_shaping_hand_worked_example():
    g = _golden("kl_shaping_worked_example.txt")
    logp, ref, mask, off, R = _shaping_case()
    r, ret = O.kl_shaped_returns(R, logp, ref, mask, off, beta=0.5, kind="k1")
    assert abs(r[0] - g["k1_r0"]) < 1e-14 and abs(r[3] - g["k1_r3"]) < 1e-14 and r[1] == 0 and r[2] == 0
    assert abs(ret[0] - g["k1_ret0"]) < 1e-14 and abs(ret[2] - g["k1_ret2"]) < 1e-14 and abs(ret[3] - g["k1_ret3"]) < 1e-14
    assert ret[1] == 0
    r, ret = O.kl_shaped_returns(R, logp, ref, mask, off, beta=0.5, kind="k3")
    assert abs(r[0] - g["k3_r0"]) < 1e-14 and abs(r[3] - g["k3_r3"]) < 1e-14
    assert abs(ret[0] - g["k3_ret0"]) < 1e-14 and abs(ret[2] - g["k3_ret2"]) < 1e-14 and abs(ret[3] - g["k3_ret3"]) < 1e-14
    _, ret = O.kl_shaped_returns(R, logp, ref, mask, off, beta=0.5, gamma=0.5, kind="k3")
    assert abs(ret[2] - g["k3_half_ret2"]) < 1e-14 and abs(ret[0] - g["k3_half_ret0"]) < 1e-14 and ret[1] == 0


def test_kl_shaping_beta_zero_gives_every_valid_token_the_trajectory_value():
    rng = _rng(70)
    off = np.array([0, 5, 5, 12, 20])                # the second response is empty
    T = 23                                           # rows 20..22 lie outside every response
    mask = (rng.random(T) < 0.7).astype(np.uint8)
    mask[5:12] = 0                                   # the third response has no valid token
    R = rng.normal(size=4)
    logp, ref = rng.normal(size=T), rng.normal(size=T)
    r, ret = O.kl_shaped_returns(R, logp, ref, mask, off, beta=0.0)
    for i in (0, 3):
        for t in range(off[i], off[i + 1]):
            assert ret[t] == (R[i] if mask[t] else 0.0)
    assert np.all(ret[5:12] == 0) and np.all(ret[20:] == 0) and np.all(r[5:12] == 0)
    # the reward itself sits on the last valid token only
    for i in (0, 3):
        valid = [t for t in range(off[i], off[i + 1]) if mask[t]]
        assert r[valid[-1]] == R[i] and all(r[t] == 0 for t in valid[:-1])


def test_kl_shaping_matches_library_cumsum_and_closed_form():
    # no mask, gamma = 1: the return-to-go is a reversed cumulative sum (numpy's routine) ...
    rng = _rng(71)
    off = np.array([0, 7, 19])
    logp, ref = rng.normal(size=19), rng.normal(size=19)
    R = np.array([1.0, -0.5])
    for kind in ("k1", "k3"):
        r, ret = O.kl_shaped_returns(R, logp, ref, None, off, beta=0.3, kind=kind)
        for i in range(2):
            seg = r[off[i]:off[i + 1]]
            assert np.allclose(ret[off[i]:off[i + 1]], np.cumsum(seg[::-1])[::-1], atol=1e-13)
    # ... and with a constant log-ratio c the k1 return of position p of n is R - beta*c*(n - p)
    c = 0.25
    _, ret = O.kl_shaped_returns(R, logp, logp - c, None, off, beta=0.3, kind="k1")
    for i in range(2):
        n = off[i + 1] - off[i]
        for p in range(n):
            assert abs(ret[off[i] + p] - (R[i] - 0.3 * c * (n - p))) < 1e-13
    # k3 is the estimator of the loss: non-negative, zero iff ref == logp, ~ delta^2 / 2
    k3 = O.token_kl_estimate(logp, ref, "k3")
    assert np.all(k3 >= 0) and np.all(O.token_kl_estimate(logp, logp, "k3") == 0)
    assert abs(O.token_kl_estimate(np.zeros(1), np.array([1e-4]), "k3")[0] - 0.5e-8) < 1e-12
    # a per-token divergence handed in is used as it is
    kl = rng.random(19)
    r, _ = O.kl_shaped_returns(np.zeros(2), logp, ref, None, off, beta=2.0, kind="given", kl_tok=kl)
    assert np.allclose(r, -2.0 * kl, atol=0)


def test_kl_shaping_discounted_bruteforce_with_mask():
    # ret_t = sum over the valid tokens u >= t of the response of gamma^(valid tokens between) r_u
    rng = _rng(72)
    off = np.array([0, 9, 9, 30, 41])
    T = 41
    mask = (rng.random(T) < 0.6).astype(np.uint8)
    logp, ref = rng.normal(size=T) * 0.3, rng.normal(size=T) * 0.3
    R = rng.normal(size=4)
    for gamma in (1.0, 0.9, 0.5):
        r, ret = O.kl_shaped_returns(R, logp, ref, mask, off, beta=0.1, gamma=gamma, kind="k3")
        for i in range(4):
            valid = [t for t in range(off[i], off[i + 1]) if mask[t]]
            for a, t in enumerate(valid):
                brute = sum(gamma ** (b - a) * r[u] for b, u in enumerate(valid) if b >= a)
                assert abs(ret[t] - brute) < 1e-12
            # telescoping: consecutive valid tokens differ by exactly one shaped reward
            for a in range(len(valid) - 1):
                assert abs(ret[valid[a]] - gamma * ret[valid[a + 1]] - r[valid[a]]) < 1e-12
        assert np.all(ret[mask == 0] == 0) and np.all(r[mask == 0] == 0)


def test_valid_rows_outside_every_response_range_take_no_part():
    # response-aware paths (sequence-level ratio, per-response aggregation): a valid row that belongs to
    # no response is as good as masked - same loss, same gradients, and the token mean is over the rest
    rng = _rng(80)
    T, d, V = 14, 6, 11
    H, W = rng.normal(size=(T, d)), rng.normal(size=(V, d)) * 0.5
    tok = rng.integers(0, V, size=T)
    old, ref, adv = rng.normal(size=T) * 0.1 - 2.0, rng.normal(size=T) * 0.1 - 2.0, rng.normal(size=T)
    off = np.array([2, 6, 11])                        # rows 0, 1 and 11..13 belong to no response
    mask = np.ones(T, dtype=np.uint8)
    mask[4] = 0
    masked_out = mask.copy()
    masked_out[:2] = 0
    masked_out[11:] = 0
    for kw in (dict(sequence_level=True), dict(agg_mode=1), dict(agg_mode=2), dict(sequence_level=True, agg_mode=1)):
        a = O.policy_loss_fwd_bwd(H, W, tok, old, ref, adv, mask, 0.2, 0.3, 0.05, ent_coef=0.01, seq_offsets=off, **kw)
        b = O.policy_loss_fwd_bwd(H, W, tok, old, ref, adv, masked_out, 0.2, 0.3, 0.05, ent_coef=0.01, seq_offsets=off, **kw)
        assert abs(a["loss"] - b["loss"]) < 1e-14 and np.allclose(a["dW"], b["dW"], atol=1e-14)
        assert not a["dH"][:2].any() and not a["dH"][11:].any()
    # token mean with the sequence-level ratio: weights are 1 / (valid rows inside ranges) = 1/8
    a = O.policy_loss_fwd_bwd(H, W, tok, old, None, adv, mask, 0.2, 0.3, 0.0, seq_offsets=off, sequence_level=True)
    lp = a["logp"]
    rho, _ = O.sequence_ratio(lp, old, masked_out, off)
    s = np.minimum(rho * adv, np.clip(rho, 0.8, 1.3) * adv)
    assert abs(a["loss"] - (-(s * masked_out).sum() / 8.0)) < 1e-13
    # the plain path (no response structure) keeps every valid row
    c = O.policy_loss_fwd_bwd(H, W, tok, old, ref, adv, mask, 0.2, 0.3, 0.05)
    assert c["dH"][:2].any() and c["dH"][11:].any()


# ----------------------------------------------------------------------------- per-token loss on its own
def test_token_loss_worked_example():
    # the two-word example of tests/golden: the per-token call has to reproduce its loss and d loss / d logp
    # from logp, entropy, old, ref alone (cases A, B: dloss/dlogp = 0.25 and 1.75; case C adds -0.1 * entropy)
    g = _golden("two_token_worked_example.txt")
    lp, ent = np.array([g["logp"]]), np.array([g["entropy"]])
    old, ref = np.array([math.log(0.5)]), np.array([math.log(0.375)])
    A = O.token_loss(lp, ent, old, ref, np.array([1.0]), None, 0.2, 0.2, 0.5)
    assert abs(A["loss"] - g["A_loss"]) < 1e-14 and abs(A["dlogp"][0] - 0.25) < 1e-14 and A["dentropy"][0] == 0.0
    assert A["clip_frac"] == 1.0 and abs(A["ratio_mean"] - 1.5) < 1e-14 and abs(A["kl_mean"] - g["k3"]) < 1e-14
    B = O.token_loss(lp, ent, old, ref, np.array([-1.0]), None, 0.2, 0.2, 0.5)
    assert abs(B["loss"] - g["B_loss"]) < 1e-14 and abs(B["dlogp"][0] - 1.75) < 1e-14 and B["clip_frac"] == 0.0
    C = O.token_loss(lp, ent, old, ref, np.array([1.0]), None, 0.2, 0.2, 0.5, ent_coef=0.1)
    assert abs(C["loss"] - g["C_loss"]) < 1e-13 and abs(C["dentropy"][0] + 0.1) < 1e-15


@pytest.mark.parametrize("beta,ent_coef,weights", [(0.0, 0.0, False), (0.3, 0.0, False), (0.3, 0.05, False),
                                                   (0.3, 0.05, True)])
def test_token_loss_agrees_with_the_full_loss_and_finite_differences(beta, ent_coef, weights):
    H, W, tokens, old, ref, adv, mask = _tiny_problem(31, T=9, masked=(2, 7))
    rng = _rng(5)
    tw = rng.uniform(0.1, 1.0, size=9) if weights else None
    full = O.policy_loss_fwd_bwd(H, W, tokens, old, ref, adv, mask, 0.2, 0.3, beta, ent_coef=ent_coef, token_weight=tw)
    lp, ent = full["logp"], full["entropy"]
    t = O.token_loss(lp, ent, old, ref, adv, mask, 0.2, 0.3, beta, ent_coef=ent_coef, token_weight=tw)
    # same loss and metrics as the whole path computes from H and W
    assert abs(t["loss"] - full["loss"]) < 1e-14
    for k in ("pg_loss", "kl_mean", "entropy_mean", "clip_frac"):
        assert abs(t[k] - full[k]) < 1e-14
    # the chain rule through logp and entropy gives the whole path's logit gradient: row sums of G * z vanish,
    # so compare through dH = sum_j g_j W_j with g built from (dlogp, dentropy)
    Z = O.logits(H, W)
    _, LP, _ = O.log_softmax_stats(Z)
    P = np.exp(LP)
    onehot = np.zeros_like(P)
    onehot[np.arange(9), tokens] = 1.0
    G = t["dlogp"][:, None] * (onehot - P) + t["dentropy"][:, None] * (-P * (LP + ent[:, None]))
    assert np.abs(G @ W - full["dH"]).max() < 1e-13
    # central differences in logp and in the entropy, valid and masked rows alike
    h = 1e-6
    for i in range(9):
        for key, arr in (("dlogp", lp), ("dentropy", ent)):
            up, dn = arr.copy(), arr.copy()
            up[i] += h
            dn[i] -= h
            a = (up, ent) if key == "dlogp" else (lp, up)
            b = (dn, ent) if key == "dlogp" else (lp, dn)
            fd = (O.token_loss(a[0], a[1], old, ref, adv, mask, 0.2, 0.3, beta, ent_coef=ent_coef, token_weight=tw)["loss"] -
                  O.token_loss(b[0], b[1], old, ref, adv, mask, 0.2, 0.3, beta, ent_coef=ent_coef, token_weight=tw)["loss"]) / (2 * h)
            assert abs(fd - t[key][i]) < 1e-8, (key, i, fd, t[key][i])
    assert t["dlogp"][2] == 0.0 and t["dlogp"][7] == 0.0 and t["dentropy"][2] == 0.0
    # nothing valid: zero loss, zero derivatives
    z = O.token_loss(lp, ent, old, ref, adv, np.zeros(9, dtype=np.uint8), 0.2, 0.3, beta, ent_coef=ent_coef)
    assert z["loss"] == 0.0 and not z["dlogp"].any() and z["ratio_max"] == 0.0
