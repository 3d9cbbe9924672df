"""GPU parity of the vocabulary-parallel head and of multi-model scoring, through the C ABI, against
the float64 oracle of the WHOLE vocabulary.  One GPU plays the ranks one after the other (the slice
calls are independent launches: nothing waits on another rank), so what is checked is exactly what
each rank would compute; the exchanges between ranks (all-gather of the statistics, sum of the
partial dH) are done here with torch.stack / addition and, across real processes, by the gloo test."""
import numpy as np
import pytest
import torch

from oracle import grpo_oracle as O

pytestmark = pytest.mark.gpu

TOL_LOGP = 2e-3
TOL_ENT = 2e-3
TOL_LOSS_REL = 1e-3
TOL_GRAD_REL = 1e-2


@pytest.fixture(scope="module")
def ctx():
    from paper_2512_21450_b200 import Context
    c = Context(0)
    yield c
    c.close()


def _np64(t):
    return t.detach().double().cpu().numpy()


def _rel(a, b):
    nb = np.linalg.norm(b)
    return np.linalg.norm(a - b) / nb if nb > 0 else np.linalg.norm(a)


def _status_ok(ctx):
    s, detail = ctx.last_device_status()
    assert s == 0, f"device status {s} detail {detail:#x}"


def _run_sharded(ctx, w, cuts, adv_tok, **kw):
    """Plays the ranks of a vocabulary partition one after the other on this GPU."""
    stats = []
    for a, b in zip(cuts[:-1], cuts[1:]):
        stats.append(ctx.rl_shard_logit_stats(w.H, w.W[a:b], w.tokens, w.mask, a, w.V).clone())
    logp, ent, lse = ctx.rl_merge_logit_stats(torch.stack(stats).contiguous(), w.mask)
    dH = torch.zeros(w.T, w.d, dtype=torch.float32, device=w.H.device)
    dW = torch.empty(w.V, w.d, dtype=torch.float32, device=w.H.device)
    losses = []
    for a, b in zip(cuts[:-1], cuts[1:]):
        o = ctx.rl_policy_loss_shard_bwd(w.H, w.W[a:b], w.tokens, w.old_logp, w.ref_logp, adv_tok, w.mask, a, w.V,
                                         logp, ent, lse, w.eps_low, w.eps_high, w.beta, ent_coef=w.ent_coef, **kw)
        dH += o["dH"]
        dW[a:b] = o["dW"]
        losses.append(float(o["loss"].item()))
    _status_ok(ctx)
    return logp, ent, lse, dH, dW, losses


@pytest.mark.parametrize("cfg_id,kwargs,cuts", [
    (0, dict(), (0, 4096)),                                   # one slice: the single-device result
    (0, dict(), (0, 2048, 4096)),
    (0, dict(V=4100, L_max=13, seed=910), (0, 1536, 1537, 4100)),   # a one-row slice and a ragged tail
    (4, dict(prompts=2, L_max=24, V=40000, seed=911), (0, 18944, 40000)),   # entropy bonus, several slabs per slice
    (1, dict(prompts=1, L_max=48, seed=912), (0, 75776, 151936)),   # the full 3B-class head on two ranks
])
def test_vocab_parallel_matches_full_vocabulary_oracle(ctx, cfg_id, kwargs, cuts):
    from paper_2512_21450_b200.workloads import make_workload
    w = make_workload(cfg_id, **kwargs)
    assert cuts[-1] == w.V
    o_adv = O.grpo_advantages(w.rewards.cpu().numpy(), w.G)
    o_adv_tok = O.broadcast_to_tokens(o_adv, w.seq_offsets.cpu().numpy(), w.T)
    _, adv_tok = ctx.rl_grpo_advantages(w.rewards, w.G, seq_offsets=w.seq_offsets, T=w.T)
    logp, ent, lse, dH, dW, losses = _run_sharded(ctx, w, cuts, adv_tok)
    oo = O.policy_loss_fwd_bwd(_np64(w.H), _np64(w.W), w.tokens.cpu().numpy(), _np64(w.old_logp),
                               None if w.ref_logp is None else _np64(w.ref_logp), o_adv_tok, w.mask.cpu().numpy(),
                               w.eps_low, w.eps_high, w.beta, ent_coef=w.ent_coef)
    m = w.mask.cpu().numpy().astype(bool)
    assert np.abs(_np64(logp) - oo["logp"]).max() <= TOL_LOGP
    assert np.abs(_np64(ent) - oo["entropy"]).max() <= TOL_ENT
    assert np.abs(_np64(lse) - oo["lse"]).max() <= TOL_LOGP
    assert not _np64(logp)[~m].any() and not _np64(dH)[~m].any()
    for ls in losses:                                          # every rank reports the loss of the whole vocabulary
        assert abs(ls - oo["loss"]) <= TOL_LOSS_REL * abs(oo["loss"]) + 1e-7
        assert ls == losses[0]
    assert _rel(_np64(dH), oo["dH"]) <= TOL_GRAD_REL
    assert _rel(_np64(dW), oo["dW"]) <= TOL_GRAD_REL
    # slice by slice against the oracle's slice functions as well (statistics and dW rows)
    a, b = cuts[-2], cuts[-1]
    st = ctx.rl_shard_logit_stats(w.H, w.W[a:b], w.tokens, w.mask, a, w.V)
    o_st = O.shard_logit_stats(_np64(w.H), _np64(w.W[a:b]), w.tokens.cpu().numpy(), a, w.mask.cpu().numpy())
    g = _np64(st)
    # (M, S) and (M, A) are each fixed only up to a common shift of M: compare what is unique
    assert np.abs((g[m, 0] + np.log(g[m, 1])) - (o_st[m, 0] + np.log(o_st[m, 1]))).max() <= TOL_LOGP
    assert np.abs(g[m, 2] / g[m, 1] - o_st[m, 2] / o_st[m, 1]).max() <= TOL_ENT
    assert np.abs(g[m, 3] - o_st[m, 3]).max() <= TOL_LOGP
    assert not g[~m].any()


def test_vocab_parallel_options_and_errors(ctx):
    from paper_2512_21450_b200.binding import RLHeadError
    from paper_2512_21450_b200.workloads import make_workload
    w = make_workload(0, V=4352, L_max=12, seed=920)
    o_adv_tok = O.broadcast_to_tokens(O.grpo_advantages(w.rewards.cpu().numpy(), w.G), w.seq_offsets.cpu().numpy(), w.T)
    _, adv_tok = ctx.rl_grpo_advantages(w.rewards, w.G, seq_offsets=w.seq_offsets, T=w.T)
    tw = (torch.rand(w.T, device="cuda") + 0.5) / w.T
    cuts = (0, 1024, 4352)
    logp, ent, lse, dH, dW, losses = _run_sharded(ctx, w, cuts, adv_tok, token_weight=tw)
    oo = O.policy_loss_fwd_bwd(_np64(w.H), _np64(w.W), w.tokens.cpu().numpy(), _np64(w.old_logp), _np64(w.ref_logp),
                               o_adv_tok, w.mask.cpu().numpy(), w.eps_low, w.eps_high, w.beta, token_weight=_np64(tw))
    assert abs(losses[0] - oo["loss"]) <= TOL_LOSS_REL * abs(oo["loss"]) + 1e-7
    assert _rel(_np64(dH), oo["dH"]) <= TOL_GRAD_REL and _rel(_np64(dW), oo["dW"]) <= TOL_GRAD_REL
    # bf16 partial dH and accumulation into an existing dW slice
    o1 = ctx.rl_policy_loss_shard_bwd(w.H, w.W[:1024], w.tokens, w.old_logp, w.ref_logp, adv_tok, w.mask, 0, w.V,
                                      logp, ent, lse, w.eps_low, w.eps_high, w.beta, token_weight=tw, dH_fp32=False)
    assert o1["dH"].dtype == torch.bfloat16
    o2 = ctx.rl_policy_loss_shard_bwd(w.H, w.W[:1024], w.tokens, w.old_logp, w.ref_logp, adv_tok, w.mask, 0, w.V,
                                      logp, ent, lse, w.eps_low, w.eps_high, w.beta, token_weight=tw,
                                      dW=o1["dW"].clone(), accumulate_dW=True)
    assert _rel(_np64(o2["dW"]), 2 * _np64(o1["dW"])) <= 1e-6
    _status_ok(ctx)
    # a token id outside the whole vocabulary is reported, one outside the slice is not
    bad = w.tokens.clone()
    bad[0] = w.V
    ctx.rl_shard_logit_stats(w.H, w.W[:1024], bad, w.mask, 0, w.V)
    s, _ = ctx.last_device_status()
    assert s == 7
    ctx.rl_shard_logit_stats(w.H, w.W[:1024], w.tokens, w.mask, 0, w.V)
    _status_ok(ctx)
    # slice outside the vocabulary
    with pytest.raises(RLHeadError) as e:
        ctx.rl_shard_logit_stats(w.H, w.W[:1024], w.tokens, w.mask, w.V - 100, w.V)
    assert e.value.status == 2
    with pytest.raises(RLHeadError) as e:
        ctx.rl_shard_logit_stats(w.H, w.W[:1024], w.tokens, w.mask, -1, w.V)
    assert e.value.status == 2
    # empty batch and all-masked batch
    z = torch.zeros(w.T, dtype=torch.uint8, device="cuda")
    st = ctx.rl_shard_logit_stats(w.H, w.W[:1024], w.tokens, z, 0, w.V)
    assert not st.any().item()
    lp, en, ls = ctx.rl_merge_logit_stats(torch.stack([st, st]).contiguous(), z)
    assert not lp.any().item() and not en.any().item() and not ls.any().item()
    o3 = ctx.rl_policy_loss_shard_bwd(w.H, w.W[:1024], w.tokens, w.old_logp, w.ref_logp, adv_tok, z, 0, w.V, lp, en, ls,
                                      w.eps_low, w.eps_high, w.beta)
    assert o3["loss"].item() == 0 and not o3["dH"].any().item() and not o3["dW"].any().item()
    _status_ok(ctx)


def test_multi_model_scoring(ctx):
    # old policy and reference scored in one call: each equals its own single-model result and the oracle
    from paper_2512_21450_b200.workloads import make_reference_model, make_workload
    w = make_workload(1, prompts=1, L_max=40, V=20000, seed=930)
    H_ref, W_ref = make_reference_model(w, d_ref=1024)
    (lp_a, lp_b), (en_a, en_b) = ctx.rl_token_logprobs_multi([w.H, H_ref], [w.W, W_ref], w.tokens, w.mask)
    _status_ok(ctx)
    m = w.mask.cpu().numpy()
    for (H, W, lp, en) in ((w.H, w.W, lp_a, en_a), (H_ref, W_ref, lp_b, en_b)):
        o_lp, o_en, _ = O.token_logprobs(_np64(H), _np64(W), w.tokens.cpu().numpy(), m)
        assert np.abs(_np64(lp) - o_lp).max() <= TOL_LOGP and np.abs(_np64(en) - o_en).max() <= TOL_ENT
        s_lp, s_en, _ = ctx.rl_token_logprobs(H, W, w.tokens, w.mask)
        assert torch.equal(s_lp, lp) and torch.equal(s_en, en)
    # without entropies, one model, and an empty batch
    (lp_only,), none = ctx.rl_token_logprobs_multi([w.H], [w.W], w.tokens, w.mask, want_entropy=False)
    assert none is None and torch.equal(lp_only, lp_a)
    _status_ok(ctx)
