"""Float64 CPU oracle for the LM-head log-probability + GRPO policy-loss path.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain definition that the
CUDA library is checked against.  Nothing in the product path may import it;
it imports nothing from the product.  Every function works on float64 numpy
arrays (bf16 inputs are widened exactly by the caller) and follows the
definitions in the order the paper states them; the only library primitive
used as a step is a dense matrix product.

Notation (paper section 2.2 and 3.1): T token rows, d hidden size, V vocabulary
size; h_t the hidden state whose next-token distribution scores the sampled
token y_t; z_t = W h_t the logits; pi_theta(.|s_t) = softmax(z_t).

Readings of the paper that this oracle fixes (the paper prints no formula or
leaves a choice open for each of them):
  * GRPO normalisation within a group of responses (section 4.2): A_i = (r_i - mean_g) /
    (std_g + eps_std) with the sample standard deviation (ddof=1) by default.
  * PPO clipped surrogate (section 3.1): the standard pessimistic form
    min(r*A, clip(r, 1-eps_low, 1+eps_high)*A).  The form as literally printed,
    min(r, clip(r))*A, is available with literal_clip=True for a test that
    documents the difference; the two agree for A >= 0.
  * KL-to-reference (section 2.2 "Regularization", section 3.1 Omega): the
    sampled-token k3 estimator exp(delta) - delta - 1, delta = ref_logp - logp.
  * Eq. 6 is maximised; the loss returned here is its negative, to be minimised.
  * Entropy bonus (section 2.2): natural-log entropy of the full next-token
    distribution, entering the loss as  - ent_coef * H.
  * Token aggregation: weights w_t = m_t / sum(m) (token mean) unless the caller
    passes token_weight.
  * Token-level KL reward shaping (section 2.2): shaped reward -beta * kl_t per
    valid token plus the response's scalar on its last valid token, then the
    return-to-go (see kl_shaped_returns).

Parity pins: every function here is pinned by tests/test_oracle_pins.py against
brute force, closed forms, finite differences and library second opinions.
What cannot be pinned from the paper is WHICH estimator / aggregation the
authors' code uses (the three readings above): parity unpinned with respect to
the authors' repository, pinned with respect to the readings stated here.
"""
from __future__ import annotations

import numpy as np


# --------------------------------------------------------------------------- #
# Algorithm 1, advantage-estimation step; section 3.2.2 advantage estimation
# stage; section 4.2 (GRPO: rewards normalised within each group).
# --------------------------------------------------------------------------- #
def grpo_advantages(rewards, group_size, ddof=1, eps_std=1e-6):
    """Per-response GRPO advantages.

    rewards: [B] one scalar per trajectory (section 3.2.2 scoring stage), the
    K = group_size responses of one prompt stored consecutively.
    Returns adv[B] with adv_i = (r_i - mean_g) / (std_g + eps_std).
    A group whose rewards are all equal gets advantage exactly 0.
    """
    r = np.asarray(rewards, dtype=np.float64)
    B = r.shape[0]
    if group_size < 2 or B % group_size != 0:
        raise ValueError("group_size must be >= 2 and divide the number of responses")
    adv = np.zeros(B, dtype=np.float64)
    for g in range(B // group_size):
        grp = r[g * group_size:(g + 1) * group_size]
        mu = grp.sum() / group_size
        var = ((grp - mu) ** 2).sum() / (group_size - ddof)
        sigma = np.sqrt(var)
        if np.all(grp == grp[0]):
            adv[g * group_size:(g + 1) * group_size] = 0.0
        else:
            adv[g * group_size:(g + 1) * group_size] = (grp - mu) / (sigma + eps_std)
    return adv


# --------------------------------------------------------------------------- #
# Other critic-free estimators the paper names in section 4.2 without printing a
# formula (the leave-one-out baseline of RLOO, the length-weighted baseline of
# OPO, REINFORCE++).  Readings, stated here because the paper is silent:
#   RLOO          A_i = r_i - mean of the OTHER responses of the group
#   OPO           A_i = r_i - sum_j(len_j r_j) / sum_j(len_j) over the group
#   REINFORCE++   A_i = (c_i - mean(c)) / (std(c) + eps_std) over the whole batch,
#                 c_i = r_i - mean of its group (population std)
# Parity unpinned with respect to the authors' code; pinned to these readings.
# --------------------------------------------------------------------------- #
def rloo_advantages(rewards, group_size):
    r = np.asarray(rewards, dtype=np.float64)
    B = r.shape[0]
    if group_size < 2 or B % group_size != 0:
        raise ValueError("group_size must be >= 2 and divide the number of responses")
    adv = np.zeros(B)
    for g in range(B // group_size):
        for i in range(group_size):
            others = [r[g * group_size + j] for j in range(group_size) if j != i]
            adv[g * group_size + i] = r[g * group_size + i] - sum(others) / (group_size - 1)
    return adv


def opo_advantages(rewards, lengths, group_size):
    r = np.asarray(rewards, dtype=np.float64)
    ln = np.asarray(lengths, dtype=np.float64)
    B = r.shape[0]
    if group_size < 1 or B % group_size != 0:
        raise ValueError("group_size must divide the number of responses")
    adv = np.zeros(B)
    for g in range(B // group_size):
        sl = slice(g * group_size, (g + 1) * group_size)
        tot = ln[sl].sum()
        base = (ln[sl] * r[sl]).sum() / tot if tot > 0 else 0.0
        adv[sl] = r[sl] - base
    return adv


def reinforce_pp_advantages(rewards, group_size, eps_std=1e-6):
    r = np.asarray(rewards, dtype=np.float64)
    B = r.shape[0]
    if group_size < 1 or B % group_size != 0:
        raise ValueError("group_size must divide the number of responses")
    c = r - np.repeat(r.reshape(-1, group_size).mean(axis=1), group_size)
    mu = c.sum() / B
    sigma = np.sqrt(((c - mu) ** 2).sum() / B)
    return (c - mu) / (sigma + eps_std)


def broadcast_to_tokens(adv_seq, seq_offsets, T):
    """Outcome supervision: every token of response i carries A_i
    (Algorithm 1: one advantage per time step from one reward per trajectory)."""
    adv_tok = np.zeros(T, dtype=np.float64)
    for i in range(len(adv_seq)):
        adv_tok[seq_offsets[i]:seq_offsets[i + 1]] = adv_seq[i]
    return adv_tok


# --------------------------------------------------------------------------- #
# Section 2.2 "Regularization" mentions that the KL-to-reference term is commonly
# applied as token-level shaping, i.e. folded into per-token rewards instead of (or
# beside) the loss.  The paper prints no formula for the shaped reward; reading:
#   kl_t  = per-token divergence estimate of a valid token t, one of
#             "k1"  logp_t - ref_logp_t              (signed sampled log-ratio)
#             "k3"  exp(delta) - delta - 1, delta = ref_logp_t - logp_t
#                                                    (the estimator of the loss)
#             "given"  a per-token value handed in (e.g. the full-distribution KL_t)
#   r_t   = -beta * kl_t, and the last VALID token of response i additionally
#           receives the response's scalar seq_value_i (its trajectory reward,
#           section 3.2.2 scoring stage, or its group-normalised advantage)
#   ret_t = r_t + gamma * ret_{next valid token of the same response}
#           (return-to-go; gamma = 1 is the plain reverse cumulative sum)
# Masked rows take no part: they get 0, carry no reward and are not counted as a
# discount step.  Rows outside every response range get 0.  A response without a
# valid token gets nothing (its seq_value is dropped).
# Parity unpinned with respect to the authors' code; pinned to this reading.
# --------------------------------------------------------------------------- #
def token_kl_estimate(logp, ref_logp, kind="k3", kl_tok=None):
    """Per-token divergence estimate used for reward shaping (see above)."""
    if kind == "given":
        return np.asarray(kl_tok, dtype=np.float64)
    logp = np.asarray(logp, dtype=np.float64)
    ref = np.asarray(ref_logp, dtype=np.float64)
    if kind == "k1":
        return logp - ref
    if kind == "k3":
        delta = ref - logp
        return np.exp(delta) - delta - 1.0
    raise ValueError("unknown KL estimate")


def kl_shaped_returns(seq_value, logp, ref_logp, mask, seq_offsets, beta, gamma=1.0,
                      kind="k3", kl_tok=None):
    """Token-level KL reward shaping.  Returns (shaped_reward[T], returns[T])."""
    off = np.asarray(seq_offsets)
    T = len(mask) if mask is not None else int(off[-1])
    m = np.ones(T, dtype=bool) if mask is None else np.asarray(mask).astype(bool)
    kl = token_kl_estimate(logp, ref_logp, kind, kl_tok)
    v = np.asarray(seq_value, dtype=np.float64)
    shaped = np.zeros(T)
    ret = np.zeros(T)
    for i in range(len(off) - 1):
        valid = [t for t in range(int(off[i]), int(off[i + 1])) if m[t]]
        if not valid:
            continue
        for t in valid:
            shaped[t] = -beta * kl[t]
        shaped[valid[-1]] += v[i]
        running = 0.0
        for t in reversed(valid):
            running = shaped[t] + gamma * running
            ret[t] = running
    return shaped, ret


# --------------------------------------------------------------------------- #
# Section 4.4 (training without padding tokens): only rows whose mask is non-zero are
# worked on; the row map lists them in ascending order.
# --------------------------------------------------------------------------- #
def valid_row_map(mask, T=None):
    """Indices of the rows with mask != 0, ascending (mask None: every row 0..T-1)."""
    if mask is None:
        return list(range(T))
    return [t for t in range(len(mask)) if mask[t] != 0]


# --------------------------------------------------------------------------- #
# Section 2.2: the policy is the next-token distribution over the vocabulary.
# --------------------------------------------------------------------------- #
def logits(H, W):
    """z[t, j] = sum_k H[t, k] * W[j, k]."""
    H = np.asarray(H, dtype=np.float64)
    W = np.asarray(W, dtype=np.float64)
    return H @ W.T


def log_softmax_stats(Z):
    """From logits Z[T, V]: lse[T], log-probabilities LP[T, V], entropy[T].

    lse_t = log sum_j exp(z_tj) (computed with the usual max shift),
    LP_tj = z_tj - lse_t,  Ent_t = - sum_j p_tj * LP_tj with p = exp(LP)
    (section 2.2 "Regularization": entropy of pi_theta(.|s_t)).
    """
    M = Z.max(axis=1, keepdims=True)
    lse = M[:, 0] + np.log(np.exp(Z - M).sum(axis=1))
    LP = Z - lse[:, None]
    P = np.exp(LP)
    ent = -(P * LP).sum(axis=1)
    return lse, LP, ent


def token_logprobs(H, W, tokens, mask=None):
    """log pi_theta(y_t | s_t), entropy and lse per row; masked rows give 0.

    Section 2.2 (off-policy adaptation): the log-probability of the sampled
    token is what enters the importance ratio.
    """
    T = H.shape[0]
    tokens = np.asarray(tokens)
    m = np.ones(T, dtype=bool) if mask is None else np.asarray(mask).astype(bool)
    logp = np.zeros(T)
    ent = np.zeros(T)
    lse = np.zeros(T)
    rows = np.nonzero(m)[0]
    if rows.size:
        Z = logits(np.asarray(H, dtype=np.float64)[rows], W)
        lse_r, LP, ent_r = log_softmax_stats(Z)
        logp[rows] = LP[np.arange(rows.size), tokens[rows]]
        ent[rows] = ent_r
        lse[rows] = lse_r
    return logp, ent, lse


# --------------------------------------------------------------------------- #
# Eq. 6 with L^PG = PPO clipped surrogate (section 3.1) and Omega = KL-to-
# reference + entropy bonus (section 2.2 "Regularization").
# --------------------------------------------------------------------------- #
def token_weights(mask):
    """Token-mean weights w_t = m_t / sum(m) (length-masked token mean)."""
    m = np.asarray(mask).astype(np.float64)
    n = m.sum()
    return m / n if n > 0 else np.zeros_like(m)


def aggregation_weights(mask, seq_offsets, mode):
    """Token weights w_t of the loss (length normalisation by token weights, section 2.2).

    mode 0: token mean over the call, w_t = m_t / sum(m).
    mode 1: mean over sequences of each sequence's token mean, w_t = m_t / (B * len_i).
    mode 2: mean over sequences of the token sum divided by the longest row range,
            w_t = m_t / (B * L_max).
    B = number of sequences, len_i = valid tokens of sequence i, L_max = max_i(off[i+1] - off[i]).
    """
    m = np.asarray(mask).astype(np.float64)
    if mode == 0:
        return token_weights(m)
    off = np.asarray(seq_offsets)
    B = len(off) - 1
    w = np.zeros_like(m)
    L_max = max(int(off[i + 1] - off[i]) for i in range(B)) if B else 0
    for i in range(B):
        sl = slice(off[i], off[i + 1])
        n = m[sl].sum()
        if mode == 1:
            if n > 0:
                w[sl] = m[sl] / (B * n)
        elif mode == 2:
            if L_max > 0:
                w[sl] = m[sl] / (B * L_max)
        else:
            raise ValueError("unknown aggregation mode")
    return w


def sequence_ratio(logp, old_logp, mask, seq_offsets):
    """Sequence-level importance ratio (the GSPO variant named in section 4.2; the
    paper prints no formula - reading): rho_i = exp(mean over the valid tokens of sequence i of
    (logp_t - old_logp_t)), i.e. the geometric mean of the token ratios; every token of the
    sequence uses rho_i.  Returns (rho per row, len per row); rows outside any sequence get 1, 0."""
    T = len(logp)
    m = np.asarray(mask).astype(bool)
    rho = np.ones(T)
    ln = np.zeros(T)
    off = np.asarray(seq_offsets)
    for i in range(len(off) - 1):
        idx = np.arange(off[i], off[i + 1])[m[off[i]:off[i + 1]]]
        if idx.size:
            rho[idx] = np.exp((logp[idx] - old_logp[idx]).sum() / idx.size)
            ln[idx] = idx.size
    return rho, ln


def per_token_terms(logp, old_logp, ref_logp, adv, eps_low, eps_high, beta,
                    literal_clip=False):
    """Per-token surrogate s_t, k3_t, ratio rho_t and d(loss_t)/d(logp_t) (unweighted).

    rho = exp(logp - old)                       (section 2.2, importance ratio)
    s   = min(rho*A, clip(rho,1-eps_low,1+eps_high)*A)      (section 3.1)
    k3  = exp(delta) - delta - 1, delta = ref - logp        (reading of Omega)
    loss_t = -s + beta*k3 (entropy handled by the caller).
    """
    rho = np.exp(logp - old_logp)
    clipped = np.clip(rho, 1.0 - eps_low, 1.0 + eps_high)
    if literal_clip:
        s = np.minimum(rho, clipped) * adv
        active = (rho <= clipped)
    else:
        s = np.minimum(rho * adv, clipped * adv)
        # the unclipped branch is the minimum (ties count as unclipped)
        active = (rho * adv <= clipped * adv)
    if beta != 0.0:
        delta = ref_logp - logp
        k3 = np.exp(delta) - delta - 1.0
        dk3 = 1.0 - np.exp(delta)          # d k3 / d logp
    else:
        k3 = np.zeros_like(logp)
        dk3 = np.zeros_like(logp)
    # d s / d logp = A * rho on the unclipped branch, 0 on the clipped one
    dlogp = -(adv * rho * active) + beta * dk3
    return s, k3, rho, active, dlogp


def token_loss(logp, entropy, old_logp, ref_logp, adv, mask, eps_low, eps_high, beta,
               ent_coef=0.0, token_weight=None):
    """Eq. 6 (negated) from per-token quantities alone, for a caller that already holds the
    log-probability (and entropy) of every token:

        loss = sum_t w_t * ( -s_t + beta * k3_t - ent_coef * Ent_t ),   w_t = m_t / sum(m)

    with s_t, k3_t of per_token_terms (section 3.1 surrogate, k3 reading of Omega).  Returns the
    loss and its derivatives with respect to logp_t and Ent_t (zero on rows with mask 0):

        d loss / d logp_t = w_t * ( -A_t rho_t [unclipped] + beta (1 - exp(delta_t)) )
        d loss / d Ent_t  = -w_t * ent_coef
    """
    logp = np.asarray(logp, dtype=np.float64)
    T = logp.shape[0]
    m = np.ones(T) if mask is None else (np.asarray(mask) != 0).astype(np.float64)
    w = token_weights(m) if token_weight is None else np.asarray(token_weight, dtype=np.float64) * m
    ent = np.zeros(T) if entropy is None else np.asarray(entropy, dtype=np.float64)
    ref = np.zeros(T) if ref_logp is None else np.asarray(ref_logp, dtype=np.float64)
    s, k3, rho, active, dlogp = per_token_terms(logp, np.asarray(old_logp, dtype=np.float64), ref,
                                                np.asarray(adv, dtype=np.float64), eps_low, eps_high, beta)
    rows = m != 0
    loss_t = -s + beta * k3 - ent_coef * ent
    out = dict(loss=float((w[rows] * loss_t[rows]).sum()),
               dlogp=np.where(rows, w * dlogp, 0.0),
               dentropy=np.where(rows, -w * ent_coef, 0.0),
               pg_loss=float((w[rows] * -s[rows]).sum()),
               kl_mean=float((w[rows] * k3[rows]).sum()),
               entropy_mean=float((w[rows] * ent[rows]).sum()),
               clip_frac=float((w[rows] * (~active[rows])).sum()),
               ratio_mean=float((w[rows] * rho[rows]).sum()),
               ratio_max=float(rho[rows].max()) if rows.any() else 0.0)
    return out


def full_kl(LP, LQ):
    """KL(pi_theta(.|s_t) || pi_ref(.|s_t)) per row from the two log-probability matrices: the
    regulariser exactly as section 2.2 / 3.1 print it, sum_j p_j (log p_j - log q_j)."""
    return (np.exp(LP) * (LP - LQ)).sum(axis=1)


def policy_loss_fwd_bwd(H, W, tokens, old_logp, ref_logp, adv, mask,
                        eps_low, eps_high, beta, ent_coef=0.0,
                        token_weight=None, literal_clip=False,
                        seq_offsets=None, agg_mode=0, sequence_level=False,
                        H_ref=None, W_ref=None):
    """Loss of Eq. 6 (negated) and its gradients with respect to H and W.

    Returns a dict with loss, dH[T,d], dW[V,d], logp, entropy, lse, G (the
    gradient with respect to the logits on valid rows, [n_valid, V]) and the
    usual scalar metrics.  Rows with mask 0 contribute nothing and get dH = 0.
    """
    H = np.asarray(H, dtype=np.float64)
    W = np.asarray(W, dtype=np.float64)
    tokens = np.asarray(tokens)
    T, d = H.shape
    V = W.shape[0]
    m = np.asarray(mask).astype(bool)
    if seq_offsets is not None and (sequence_level or agg_mode != 0):
        # response-aware paths: a valid row that lies outside every response range takes no part
        # in the loss (it has no response to be aggregated with), exactly as if it were masked
        off_ = np.asarray(seq_offsets)
        inside = np.zeros(T, dtype=bool)
        inside[int(off_[0]):int(off_[-1])] = True
        m = m & inside
    if token_weight is not None:
        w = np.asarray(token_weight, dtype=np.float64) * m
    else:
        w = aggregation_weights(m, seq_offsets, agg_mode)
    old_logp = np.asarray(old_logp, dtype=np.float64)
    adv = np.asarray(adv, dtype=np.float64)
    ref = np.zeros(T) if ref_logp is None else np.asarray(ref_logp, dtype=np.float64)

    rows = np.nonzero(m)[0]
    out = dict(loss=0.0, dH=np.zeros((T, d)), dW=np.zeros((V, d)),
               logp=np.zeros(T), entropy=np.zeros(T), lse=np.zeros(T),
               G=np.zeros((0, V)), rows=rows)
    if rows.size == 0:
        out.update(pg_loss=0.0, kl_mean=0.0, entropy_mean=0.0, clip_frac=0.0)
        return out

    Hr = H[rows]
    y = tokens[rows]
    Z = logits(Hr, W)                               # [n, V]
    lse, LP, ent = log_softmax_stats(Z)
    P = np.exp(LP)
    logp = LP[np.arange(rows.size), y]

    wr = w[rows]
    if not sequence_level:
        s, k3, rho, active, dlogp = per_token_terms(
            logp, old_logp[rows], ref[rows], adv[rows], eps_low, eps_high, beta, literal_clip)
        wdlogp = wr * dlogp                       # weighted d loss / d logp_t
    else:
        # sequence-level ratio: the surrogate of every token uses rho_i of its sequence
        logp_full = np.zeros(T)
        logp_full[rows] = logp
        rho_full, len_full = sequence_ratio(logp_full, old_logp, m, seq_offsets)
        rho = rho_full[rows]
        a = adv[rows]
        clipped = np.clip(rho, 1.0 - eps_low, 1.0 + eps_high)
        s = np.minimum(rho * a, clipped * a)
        active = (rho * a <= clipped * a)
        # d rho_i / d logp_u = rho_i / len_i for every valid token u of sequence i, hence
        # d loss / d logp_u = -(rho_i / len_i) * sum over the sequence of w_t A_t active_t
        contrib = np.zeros(T)
        contrib[rows] = wr * a * active
        off = np.asarray(seq_offsets)
        seq_sum = np.zeros(T)
        for i in range(len(off) - 1):
            seq_sum[off[i]:off[i + 1]] = contrib[off[i]:off[i + 1]].sum()
        wdlogp = -(rho / np.maximum(len_full[rows], 1.0)) * seq_sum[rows]
        if beta != 0.0:
            delta = ref[rows] - logp
            k3 = np.exp(delta) - delta - 1.0
            wdlogp = wdlogp + wr * beta * (1.0 - np.exp(delta))
        else:
            k3 = np.zeros_like(logp)
    kl_full = None
    if H_ref is not None:
        # full-distribution KL to the (frozen) reference policy softmax(W_ref h_ref) replaces the
        # sampled-token k3 estimate: remove what k3 contributed, add beta * KL_t and its gradient
        Zr = logits(np.asarray(H_ref, dtype=np.float64)[rows], W_ref)
        _, LQ, _ = log_softmax_stats(Zr)
        kl_full = full_kl(LP, LQ)
        if beta != 0.0:
            delta_k3 = ref[rows] - logp
            wdlogp = wdlogp - wr * beta * (1.0 - np.exp(delta_k3))
        k3 = kl_full
    loss_t = -s + beta * k3 - ent_coef * ent
    loss = float((wr * loss_t).sum())

    # gradient with respect to the logits:
    #   d logp_t / d z_tj = 1[j = y_t] - p_tj
    #   d Ent_t  / d z_tj = -p_tj * (log p_tj + Ent_t)
    onehot = np.zeros_like(P)
    onehot[np.arange(rows.size), y] = 1.0
    G = wdlogp[:, None] * (onehot - P)
    if ent_coef != 0.0:
        G += (wr * ent_coef)[:, None] * P * (LP + ent[:, None])
    if kl_full is not None and beta != 0.0:
        # d KL_t / d z_tj = p_tj (log p_tj - log q_tj - KL_t)
        G += (wr * beta)[:, None] * P * (LP - LQ - kl_full[:, None])

    out["dH"][rows] = G @ W                         # dH_tk = sum_j g_tj W_jk
    out["dW"] = G.T @ Hr                            # dW_jk = sum_t g_tj H_tk
    out["loss"] = loss
    out["logp"][rows] = logp
    out["entropy"][rows] = ent
    out["lse"][rows] = lse
    out["G"] = G
    out["pg_loss"] = float((wr * -s).sum())
    out["kl_mean"] = float((wr * k3).sum())
    out["entropy_mean"] = float((wr * ent).sum())
    out["clip_frac"] = float((wr * (~active)).sum())
    out["rho"] = rho
    out["active"] = active
    return out


# --------------------------------------------------------------------------- #
# Sampled checks at sizes where the full gradient is too slow to form: one
# row of dH needs only that row; one row of dW needs that vocabulary row of
# the logits for every valid token plus per-token statistics.
# --------------------------------------------------------------------------- #
def dH_rows(H_rows, W, tokens_rows, old_rows, ref_rows, adv_rows, w_rows,
            eps_low, eps_high, beta, ent_coef=0.0, H_ref_rows=None, W_ref=None):
    """dH for a subset of valid rows whose token weights w_rows are given.

    With H_ref_rows / W_ref the regulariser is the full-distribution KL to
    softmax(W_ref h_ref) as in policy_loss_fwd_bwd (ref_rows is then unused)."""
    H_rows = np.asarray(H_rows, dtype=np.float64)
    W = np.asarray(W, dtype=np.float64)
    n = H_rows.shape[0]
    Z = logits(H_rows, W)
    lse, LP, ent = log_softmax_stats(Z)
    P = np.exp(LP)
    y = np.asarray(tokens_rows)
    logp = LP[np.arange(n), y]
    ref = np.zeros(n) if ref_rows is None else np.asarray(ref_rows, dtype=np.float64)
    s, k3, rho, active, dlogp = per_token_terms(
        logp, np.asarray(old_rows, dtype=np.float64), ref,
        np.asarray(adv_rows, dtype=np.float64), eps_low, eps_high, beta)
    onehot = np.zeros_like(P)
    onehot[np.arange(n), y] = 1.0
    w_rows = np.asarray(w_rows, dtype=np.float64)
    kl = None
    if H_ref_rows is not None:
        _, LQ, _ = log_softmax_stats(logits(np.asarray(H_ref_rows, dtype=np.float64), W_ref))
        kl = full_kl(LP, LQ)
        # the sampled-token estimate plays no part: take its derivative back out
        dlogp = dlogp - beta * (1.0 - np.exp(ref - logp)) if beta != 0.0 else dlogp
        k3 = kl
    G = (w_rows * dlogp)[:, None] * (onehot - P)
    if ent_coef != 0.0:
        G += (w_rows * ent_coef)[:, None] * P * (LP + ent[:, None])
    if kl is not None and beta != 0.0:
        G += (w_rows * beta)[:, None] * P * (LP - LQ - kl[:, None])
    return dict(dH=G @ W, logp=logp, entropy=ent, lse=lse, kl=kl,
                loss_t=-s + beta * k3 - ent_coef * ent)


def dW_rows(H_valid, W_sel, sel, tokens_valid, lse, ent, dlogp_w, ent_w):
    """dW[j, :] for the vocabulary rows j in `sel`.

    H_valid [n,d]: hidden states of every valid token; W_sel = W[sel];
    lse, ent [n]: per-token log-sum-exp and entropy; dlogp_w[n] = w_t * d loss_t /
    d logp_t; ent_w[n] = w_t * ent_coef.  g_tj as in policy_loss_fwd_bwd.
    """
    H_valid = np.asarray(H_valid, dtype=np.float64)
    Zs = H_valid @ np.asarray(W_sel, dtype=np.float64).T        # [n, |sel|]
    LP = Zs - np.asarray(lse, dtype=np.float64)[:, None]
    P = np.exp(LP)
    onehot = (np.asarray(tokens_valid)[:, None] == np.asarray(sel)[None, :]).astype(np.float64)
    G = np.asarray(dlogp_w, dtype=np.float64)[:, None] * (onehot - P)
    G += np.asarray(ent_w, dtype=np.float64)[:, None] * P * (LP + np.asarray(ent, dtype=np.float64)[:, None])
    return G.T @ H_valid


# --------------------------------------------------------------------------- #
# Vocabulary-parallel LM head (section 4.3 / 4.4: sharded training, model states
# not fully resident on one GPU): the rows of W are partitioned over ranks, rank
# s holding vocabulary ids [off_s, off_s + V_s).  Nothing new is computed - the
# results must equal the single-device definitions above - so each function
# below is the plain definition restricted to one slice of the vocabulary.
# --------------------------------------------------------------------------- #
def shard_logit_stats(H, W_shard, tokens, vocab_offset, mask=None):
    """Per-row statistics of one vocabulary slice: stats[t] = (M, S, A, z_y) with
    z_j = W_shard[j] . h_t for the slice's rows, M = max_j z_j, S = sum_j exp(z_j - M),
    A = sum_j exp(z_j - M) z_j, and z_y the logit of the sampled token when its id lies in
    [vocab_offset, vocab_offset + V_s), else 0.  Masked rows give (0, 0, 0, 0)."""
    H = np.asarray(H, dtype=np.float64)
    W_shard = np.asarray(W_shard, dtype=np.float64)
    T = H.shape[0]
    Vs = W_shard.shape[0]
    tokens = np.asarray(tokens)
    m = np.ones(T, dtype=bool) if mask is None else np.asarray(mask).astype(bool)
    stats = np.zeros((T, 4))
    for t in np.nonzero(m)[0]:
        z = W_shard @ H[t]
        M = z.max()
        e = np.exp(z - M)
        y = int(tokens[t]) - int(vocab_offset)
        stats[t] = (M, e.sum(), (e * z).sum(), z[y] if 0 <= y < Vs else 0.0)
    return stats


def merge_logit_stats(stats_per_shard, mask=None):
    """From the statistics of every slice of a partition of the vocabulary: lse_t = log of the
    sum over slices of S_s exp(M_s), logp_t = (sum of z_y over slices) - lse_t, and
    Ent_t = lse_t - (sum_s A_s exp(M_s)) / (sum_s S_s exp(M_s)); sums are shifted by the largest M_s.
    Returns (logp, entropy, lse); masked rows give 0."""
    st = np.asarray(stats_per_shard, dtype=np.float64)      # [n_shards, T, 4]
    T = st.shape[1]
    m = np.ones(T, dtype=bool) if mask is None else np.asarray(mask).astype(bool)
    logp, ent, lse = np.zeros(T), np.zeros(T), np.zeros(T)
    for t in np.nonzero(m)[0]:
        M = st[:, t, 0].max()
        S = (st[:, t, 1] * np.exp(st[:, t, 0] - M)).sum()
        A = (st[:, t, 2] * np.exp(st[:, t, 0] - M)).sum()
        lse[t] = M + np.log(S)
        logp[t] = st[:, t, 3].sum() - lse[t]
        ent[t] = lse[t] - A / S
    return logp, ent, lse


def policy_loss_shard_bwd(H, W_shard, tokens, vocab_offset, logp, entropy, lse, old_logp, ref_logp, adv,
                          mask, eps_low, eps_high, beta, ent_coef=0.0, token_weight=None):
    """One vocabulary slice's share of the backward pass, given the merged per-token
    log-probability, entropy and log-sum-exp of the whole vocabulary.

    The loss (identical on every slice, it only needs per-token quantities) and, for the
    columns j of the slice, g_tj exactly as in policy_loss_fwd_bwd with p_tj = exp(z_tj - lse_t);
    dH_partial = G_slice W_shard (summing it over the slices gives dH) and
    dW_shard = G_slice^T H (the slice's rows of dW)."""
    H = np.asarray(H, dtype=np.float64)
    W_shard = np.asarray(W_shard, dtype=np.float64)
    T, d = H.shape
    Vs = W_shard.shape[0]
    tokens = np.asarray(tokens)
    m = np.asarray(mask).astype(bool)
    w = token_weights(m) if token_weight is None else np.asarray(token_weight, dtype=np.float64) * m
    rows = np.nonzero(m)[0]
    out = dict(loss=0.0, dH_partial=np.zeros((T, d)), dW_shard=np.zeros((Vs, d)))
    if rows.size == 0:
        return out
    ref = np.zeros(T) if ref_logp is None else np.asarray(ref_logp, dtype=np.float64)
    lp = np.asarray(logp, dtype=np.float64)[rows]
    en = np.asarray(entropy, dtype=np.float64)[rows]
    s, k3, rho, active, dlogp = per_token_terms(lp, np.asarray(old_logp, dtype=np.float64)[rows], ref[rows],
                                                np.asarray(adv, dtype=np.float64)[rows], eps_low, eps_high, beta)
    wr = w[rows]
    out["loss"] = float((wr * (-s + beta * k3 - ent_coef * en)).sum())
    LP = H[rows] @ W_shard.T - np.asarray(lse, dtype=np.float64)[rows][:, None]     # log p_tj on the slice
    P = np.exp(LP)
    y = tokens[rows] - int(vocab_offset)
    onehot = np.zeros_like(P)
    inside = (y >= 0) & (y < Vs)
    onehot[np.nonzero(inside)[0], y[inside]] = 1.0
    G = (wr * dlogp)[:, None] * (onehot - P)
    if ent_coef != 0.0:
        G += (wr * ent_coef)[:, None] * P * (LP + en[:, None])
    out["dH_partial"][rows] = G @ W_shard
    out["dW_shard"] = G.T @ H[rows]
    return out
