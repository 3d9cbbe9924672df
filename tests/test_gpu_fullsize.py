"""Full-size parity, in the launch configuration the benchmark times (default context, default slab
sizes): the four large configurations are too big for a full float64 oracle pass, so the CUDA
output is checked on sampled outputs the oracle computes one by one, and on identities that hold
at any size.

  * sampled valid rows (random, first/last rows, tile-boundary rows): oracle log-prob, entropy and
    the dH row -- each needs only that row of H and all of W;
  * sampled vocabulary rows of dW (random, the most frequent targets, the last tail rows): the
    oracle forms g_tj for those j over all valid tokens; it takes lse/entropy/log-prob per token
    from the CUDA forward, which the sampled-row check has validated (semi-independent, by design);
  * loss: recomputed in float64 from the per-token log-probs and entropies;
  * identities: every column of dW sums to zero over the vocabulary, and <dH,H> = <dW,W>.
"""
import numpy as np
import pytest
import torch

from oracle import grpo_oracle as O

pytestmark = pytest.mark.gpu

TOL_LOGP = 2e-3
TOL_ENT = 2e-3
TOL_LOSS_REL = 1e-3
TOL_GRAD_REL = 1e-2


def _np64(t):
    return t.detach().double().cpu().numpy()


def _rel(a, b):
    return np.linalg.norm(a - b) / np.linalg.norm(b)


@pytest.mark.parametrize("cfg_id,n_rows,n_cols", [(1, 256, 96), (2, 192, 48), (3, 192, 48), (4, 192, 48)])
def test_full_size_sampled(cfg_id, n_rows, n_cols):
    from paper_2512_21450_b200 import Context
    from paper_2512_21450_b200.workloads import make_workload
    ctx = Context(0)
    try:
        w = make_workload(cfg_id)
        adv_seq, adv_tok = ctx.rl_grpo_advantages(w.rewards, w.G, seq_offsets=w.seq_offsets, T=w.T)
        out = ctx.rl_policy_loss_fwd_bwd(w.H, w.W, w.tokens, w.old_logp, w.ref_logp, adv_tok, w.mask,
                                         w.eps_low, w.eps_high, w.beta, ent_coef=w.ent_coef)
        status, detail = ctx.last_device_status()
        assert status == 0, (status, hex(detail & 0xffffffff))

        # advantages: full oracle (cheap)
        o_adv = O.grpo_advantages(w.rewards.cpu().numpy(), w.G)
        assert np.abs(_np64(adv_seq) - o_adv).max() <= 1e-6
        o_adv_tok = O.broadcast_to_tokens(o_adv, w.seq_offsets.cpu().numpy(), w.T)

        valid = torch.nonzero(w.mask, as_tuple=False)[:, 0].cpu().numpy()
        N = valid.size
        assert N == w.n_valid and N > 10000
        rng = np.random.default_rng(900 + cfg_id)
        special = [0, 1, 127, 128, 255, 256, N - 129, N - 128, N - 2, N - 1, 32767, 32768]
        idx = np.unique(np.concatenate([np.array([i for i in special if 0 <= i < N]),
                                        rng.choice(N, size=n_rows, replace=False)]))
        rows = valid[idx]
        W64 = _np64(w.W)
        wt = np.full(rows.size, 1.0 / N)
        ref_rows = None if w.ref_logp is None else _np64(w.ref_logp[rows])
        r = O.dH_rows(_np64(w.H[rows]), W64, w.tokens[rows].cpu().numpy(), _np64(w.old_logp[rows]), ref_rows,
                      o_adv_tok[rows], wt, w.eps_low, w.eps_high, w.beta, ent_coef=w.ent_coef)
        assert np.abs(_np64(out["logp"][rows]) - r["logp"]).max() <= TOL_LOGP
        assert np.abs(_np64(out["entropy"][rows]) - r["entropy"]).max() <= TOL_ENT
        assert _rel(_np64(out["dH"][rows]), r["dH"]) <= TOL_GRAD_REL
        # masked rows are exactly zero
        masked = torch.nonzero(w.mask == 0, as_tuple=False)[:, 0]
        if masked.numel():
            pick = masked[torch.randperm(masked.numel(), device=masked.device)[:4096]]
            assert not out["dH"][pick].any() and not out["logp"][pick].any()

        # per-token quantities of every valid row, in float64, from the CUDA forward outputs
        logp = _np64(out["logp"])[valid]
        ent = _np64(out["entropy"])[valid]
        old = _np64(w.old_logp)[valid]
        ref = np.zeros(N) if w.ref_logp is None else _np64(w.ref_logp)[valid]
        adv = o_adv_tok[valid]
        s, k3, rho, active, dlogp = O.per_token_terms(logp, old, ref, adv, w.eps_low, w.eps_high, w.beta)
        loss64 = float(((-s + w.beta * k3 - w.ent_coef * ent) / N).sum())
        assert abs(out["loss"].item() - loss64) <= TOL_LOSS_REL * abs(loss64) + 1e-7

        # sampled vocabulary rows of dW
        tok_valid = w.tokens.cpu().numpy()[valid]
        freq = np.argsort(np.bincount(tok_valid, minlength=w.V))[-8:]
        sel = np.unique(np.concatenate([rng.choice(w.V, size=n_cols, replace=False), freq,
                                        np.arange(w.V - 4, w.V), np.array([0, 255, 256, 18943, 18944, 37887, 37888])]))
        # the loss call does not return lse; the forward-only call does
        _, _, lse_t = ctx.rl_token_logprobs(w.H, w.W, w.tokens, w.mask)
        lse = _np64(lse_t)[valid]
        assert np.abs(lse[idx] - r["lse"]).max() <= TOL_LOGP
        Hv = _np64(w.H[torch.from_numpy(valid).to(w.H.device)])
        dWs = O.dW_rows(Hv, W64[sel], sel, tok_valid, lse, ent, dlogp / N, np.full(N, w.ent_coef / N))
        del Hv
        assert _rel(_np64(out["dW"][torch.from_numpy(sel).to(w.H.device)]), dWs) <= TOL_GRAD_REL

        # identities on the whole CUDA output
        dW = out["dW"]
        col_sum = dW.double().sum(dim=0)
        col_abs = dW.double().abs().sum(dim=0)
        assert (col_sum.abs() <= 1e-3 * col_abs + 1e-12).all()
        rowdot = torch.cat([(out["dH"][i:i + 65536].double() * w.H[i:i + 65536].double()).sum(dim=1)
                            for i in range(0, w.T, 65536)])
        lhs = rowdot.sum().item()
        rhs = (dW.double() * w.W.double()).sum().item()
        assert abs(lhs - rhs) <= 1e-2 * rowdot.abs().sum().item()
    finally:
        ctx.close()
        torch.cuda.empty_cache()


def test_full_size_full_kl():
    """Config 1 at full size with the full-distribution KL to a reference model (drifted copy of the
    policy): per-token KL, log-prob, entropy and dH on sampled rows, the loss recomputed in float64
    from the per-token outputs, and the two identities."""
    from paper_2512_21450_b200 import Context
    from paper_2512_21450_b200.workloads import make_workload, make_reference_model
    ctx = Context(0)
    try:
        w = make_workload(1)
        beta, ent_coef = 0.04, 0.001
        H_ref, W_ref = make_reference_model(w, drift=0.1)
        adv_seq, adv_tok = ctx.rl_grpo_advantages(w.rewards, w.G, seq_offsets=w.seq_offsets, T=w.T)
        out = ctx.rl_policy_loss_fwd_bwd(w.H, w.W, w.tokens, w.old_logp, None, adv_tok, w.mask, w.eps_low,
                                         w.eps_high, beta, ent_coef=ent_coef, H_ref=H_ref, W_ref=W_ref)
        status, detail = ctx.last_device_status()
        assert status == 0, (status, hex(detail & 0xffffffff))
        o_adv_tok = O.broadcast_to_tokens(O.grpo_advantages(w.rewards.cpu().numpy(), w.G),
                                          w.seq_offsets.cpu().numpy(), w.T)
        valid = torch.nonzero(w.mask, as_tuple=False)[:, 0].cpu().numpy()
        N = valid.size
        rng = np.random.default_rng(977)
        special = [0, 127, 128, 255, 256, N - 129, N - 1, 32767, 32768]
        idx = np.unique(np.concatenate([np.array([i for i in special if 0 <= i < N]),
                                        rng.choice(N, size=160, replace=False)]))
        rows = valid[idx]
        W64, Wr64 = _np64(w.W), _np64(W_ref)
        r = O.dH_rows(_np64(w.H[rows]), W64, w.tokens[rows].cpu().numpy(), _np64(w.old_logp[rows]), None,
                      o_adv_tok[rows], np.full(rows.size, 1.0 / N), w.eps_low, w.eps_high, beta, ent_coef=ent_coef,
                      H_ref_rows=_np64(H_ref[rows]), W_ref=Wr64)
        del W64, Wr64
        assert r["kl"].mean() > 1e-3
        assert np.abs(_np64(out["logp"][rows]) - r["logp"]).max() <= TOL_LOGP
        assert np.abs(_np64(out["entropy"][rows]) - r["entropy"]).max() <= TOL_ENT
        # KL_t = (A - D)/S - lse + lse_ref in fp32: a few ulp of quantities of size lse (about 12)
        assert np.abs(_np64(out["kl"][rows]) - r["kl"]).max() <= 2e-3 * np.abs(r["kl"]).max() + 2e-5
        assert _rel(_np64(out["dH"][rows]), r["dH"]) <= TOL_GRAD_REL
        masked = torch.nonzero(w.mask == 0, as_tuple=False)[:, 0]
        if masked.numel():
            assert not out["dH"][masked[:4096]].any() and not out["kl"][masked[:4096]].any()
        # loss from the per-token outputs, in float64
        logp = _np64(out["logp"])[valid]
        ent = _np64(out["entropy"])[valid]
        kl = _np64(out["kl"])[valid]
        s, _, _, _, _ = O.per_token_terms(logp, _np64(w.old_logp)[valid], np.zeros(N), o_adv_tok[valid],
                                          w.eps_low, w.eps_high, 0.0)
        loss64 = float(((-s + beta * kl - ent_coef * ent) / N).sum())
        assert abs(out["loss"].item() - loss64) <= TOL_LOSS_REL * abs(loss64) + 1e-7
        assert abs(out["metrics"][1].item() - kl.mean()) <= 1e-3 * kl.mean()
        dW = out["dW"]
        col_sum = dW.double().sum(dim=0)
        col_abs = dW.double().abs().sum(dim=0)
        assert (col_sum.abs() <= 1e-3 * col_abs + 1e-12).all()
        rowdot = torch.cat([(out["dH"][i:i + 65536].double() * w.H[i:i + 65536].double()).sum(dim=1)
                            for i in range(0, w.T, 65536)])
        rhs = (dW.double() * w.W.double()).sum().item()
        assert abs(rowdot.sum().item() - rhs) <= 1e-2 * rowdot.abs().sum().item()
    finally:
        ctx.close()
        torch.cuda.empty_cache()


def test_full_size_vocab_parallel():
    """Config 1 at full size with the head cut into two vocabulary slices (one GPU plays both ranks
    in turn): merged log-prob / entropy and the summed dH on sampled rows, sampled dW rows on both
    sides of the cut, the loss, and the two identities on the assembled gradients."""
    from paper_2512_21450_b200 import Context
    from paper_2512_21450_b200.workloads import make_workload
    ctx = Context(0)
    try:
        w = make_workload(1)
        cut = 296 * 256            # 75776: the first slice ends on a column-tile boundary, the second is ragged
        cuts = (0, cut, w.V)
        _, adv_tok = ctx.rl_grpo_advantages(w.rewards, w.G, seq_offsets=w.seq_offsets, T=w.T)
        stats = torch.stack([ctx.rl_shard_logit_stats(w.H, w.W[a:b], w.tokens, w.mask, a, w.V)
                             for a, b in zip(cuts[:-1], cuts[1:])]).contiguous()
        logp, ent, lse = ctx.rl_merge_logit_stats(stats, w.mask)
        dH = torch.zeros(w.T, w.d, dtype=torch.float32, device=w.H.device)
        dW = torch.empty(w.V, w.d, dtype=torch.float32, device=w.H.device)
        losses = []
        for a, b in zip(cuts[:-1], cuts[1:]):
            o = ctx.rl_policy_loss_shard_bwd(w.H, w.W[a:b], w.tokens, w.old_logp, w.ref_logp, adv_tok, w.mask, a, w.V,
                                             logp, ent, lse, w.eps_low, w.eps_high, w.beta, dW=dW[a:b])
            dH += o["dH"]
            losses.append(o["loss"].item())
        status, detail = ctx.last_device_status()
        assert status == 0, (status, hex(detail & 0xffffffff))
        assert losses[0] == losses[1]

        o_adv_tok = O.broadcast_to_tokens(O.grpo_advantages(w.rewards.cpu().numpy(), w.G),
                                          w.seq_offsets.cpu().numpy(), w.T)
        valid = torch.nonzero(w.mask, as_tuple=False)[:, 0].cpu().numpy()
        N = valid.size
        rng = np.random.default_rng(991)
        special = [0, 127, 128, 255, 256, N - 129, N - 1]
        idx = np.unique(np.concatenate([np.array(special), rng.choice(N, size=128, replace=False)]))
        rows = valid[idx]
        W64 = _np64(w.W)
        r = O.dH_rows(_np64(w.H[rows]), W64, w.tokens[rows].cpu().numpy(), _np64(w.old_logp[rows]),
                      _np64(w.ref_logp[rows]), o_adv_tok[rows], np.full(rows.size, 1.0 / N), w.eps_low, w.eps_high,
                      w.beta)
        assert np.abs(_np64(logp[rows]) - r["logp"]).max() <= TOL_LOGP
        assert np.abs(_np64(ent[rows]) - r["entropy"]).max() <= TOL_ENT
        assert np.abs(_np64(lse[rows]) - r["lse"]).max() <= TOL_LOGP
        assert _rel(_np64(dH[rows]), r["dH"]) <= TOL_GRAD_REL
        masked = torch.nonzero(w.mask == 0, as_tuple=False)[:, 0]
        assert not dH[masked[:4096]].any() and not logp[masked[:4096]].any()

        lp, en, ls = _np64(logp)[valid], _np64(ent)[valid], _np64(lse)[valid]
        s, k3, rho, active, dlogp = O.per_token_terms(lp, _np64(w.old_logp)[valid], _np64(w.ref_logp)[valid],
                                                      o_adv_tok[valid], w.eps_low, w.eps_high, w.beta)
        loss64 = float(((-s + w.beta * k3) / N).sum())
        assert abs(losses[0] - loss64) <= TOL_LOSS_REL * abs(loss64) + 1e-7

        tok_valid = w.tokens.cpu().numpy()[valid]
        sel = np.unique(np.concatenate([rng.choice(w.V, size=48, replace=False),
                                        np.array([0, cut - 2, cut - 1, cut, cut + 1, w.V - 2, w.V - 1])]))
        Hv = _np64(w.H[torch.from_numpy(valid).to(w.H.device)])
        dWs = O.dW_rows(Hv, W64[sel], sel, tok_valid, ls, en, dlogp / N, np.zeros(N))
        del Hv, W64
        assert _rel(_np64(dW[torch.from_numpy(sel).to(w.H.device)]), dWs) <= TOL_GRAD_REL

        col_sum = dW.double().sum(dim=0)
        col_abs = dW.double().abs().sum(dim=0)
        assert (col_sum.abs() <= 1e-3 * col_abs + 1e-12).all()
        rowdot = (dH.double() * w.H.double()).sum(dim=1)
        rhs = (dW.double() * w.W.double()).sum().item()
        assert abs(rowdot.sum().item() - rhs) <= 1e-2 * rowdot.abs().sum().item()
    finally:
        ctx.close()
        torch.cuda.empty_cache()
