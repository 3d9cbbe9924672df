"""GPU parity: the CUDA path, called through the C ABI, against the float64 oracle on the same
seeded inputs.  Tolerances are the stated ones for bf16 inputs with fp32 accumulation:
|dlogp| <= 2e-3, |dentropy| <= 2e-3, loss relative error <= 1e-3, dH and dW relative Frobenius
error <= 1e-2, advantages within 1e-6."""
import numpy as np
import pytest
import torch

from oracle import grpo_oracle as O

pytestmark = pytest.mark.gpu

TOL_LOGP = 2e-3
TOL_ENT = 2e-3
TOL_LOSS_REL = 1e-3
TOL_GRAD_REL = 1e-2
TOL_ADV = 1e-6


@pytest.fixture(scope="module")
def ctx():
    from paper_2512_21450_b200 import Context
    c = Context(0)
    yield c
    c.close()


def _np64(t):
    return t.detach().double().cpu().numpy()


def _assert_status_ok(ctx):
    s, detail = ctx.last_device_status()
    assert s == 0, f"device status {s} detail {detail:#x}"


def _rel(a, b):
    nb = np.linalg.norm(b)
    return np.linalg.norm(a - b) / nb if nb > 0 else np.linalg.norm(a)


def _assert_blockwise(got, want, block_rows, what):
    """Localised gradient check on top of the global Frobenius norm: every block of block_rows
    consecutive rows has to agree within 1e-2 of its own norm plus 1e-2 of an average block's norm
    (||tensor|| / sqrt(blocks)), so that one wrong row or tile cannot hide inside the global norm."""
    n = want.shape[0]
    n_blocks = (n + block_rows - 1) // block_rows
    pad = n_blocks * block_rows - n
    sq = lambda a: np.pad((a * a).sum(axis=1), (0, pad)).reshape(n_blocks, block_rows).sum(axis=1)  # noqa: E731
    err, ref = np.sqrt(sq(got - want)), np.sqrt(sq(want))
    bound = TOL_GRAD_REL * ref + TOL_GRAD_REL * np.linalg.norm(want) / np.sqrt(n_blocks)
    worst = int(np.argmax(err - bound))
    assert np.all(err <= bound), f"{what}: block {worst} (rows {worst * block_rows}..) off by {err[worst]:.3e} > {bound[worst]:.3e}"


def _poison(ctx, w, d_ref=0, dH_fp32=False):
    """Workspace and outputs filled with NaN bit patterns before a call: whatever a kernel forgets to
    write, or reads before writing, then shows up as NaN in the results."""
    ctx.ensure_workspace(w.T, w.d, w.V, d_ref=d_ref)
    ctx._ws.fill_(0xFF)
    dev = w.W.device
    return dict(dH=torch.full((w.T, w.d), float("nan"), dtype=torch.float32 if dH_fp32 else torch.bfloat16, device=dev),
                dW=torch.full((w.V, w.d), float("nan"), dtype=torch.float32, device=dev),
                loss=torch.full((1,), float("nan"), dtype=torch.float32, device=dev))


def _oracle_case(w, adv_tok_np, **kw):
    return O.policy_loss_fwd_bwd(
        _np64(w.H), _np64(w.W), w.tokens.cpu().numpy(), _np64(w.old_logp),
        None if w.ref_logp is None else _np64(w.ref_logp), adv_tok_np, w.mask.cpu().numpy(),
        w.eps_low, w.eps_high, w.beta, ent_coef=w.ent_coef, **kw)


def _check_against_oracle(ctx, w, token_weight=None, boundary_margin=1e-5, agg_mode=0, sequence_level=False,
                          dH_fp32=False):
    from paper_2512_21450_b200.workloads import Workload  # noqa: F401
    adv_seq, adv_tok = ctx.rl_grpo_advantages(w.rewards, w.G, seq_offsets=w.seq_offsets, T=w.T)
    o_adv = O.grpo_advantages(w.rewards.cpu().numpy(), w.G)
    assert np.abs(_np64(adv_seq) - o_adv).max() <= TOL_ADV
    o_adv_tok = O.broadcast_to_tokens(o_adv, w.seq_offsets.cpu().numpy(), w.T)
    assert np.abs(_np64(adv_tok) - o_adv_tok).max() <= TOL_ADV

    out = ctx.rl_policy_loss_fwd_bwd(w.H, w.W, w.tokens, w.old_logp, w.ref_logp, adv_tok, w.mask,
                                     w.eps_low, w.eps_high, w.beta, ent_coef=w.ent_coef,
                                     token_weight=token_weight, agg_mode=agg_mode, sequence_level=sequence_level,
                                     seq_offsets=w.seq_offsets if (agg_mode or sequence_level) else None,
                                     dH_fp32=dH_fp32, **_poison(ctx, w, dH_fp32=dH_fp32))
    _assert_status_ok(ctx)
    assert out["dH"].dtype == (torch.float32 if dH_fp32 else torch.bfloat16)
    for k in ("loss", "dH", "dW", "logp", "entropy", "metrics"):
        assert not torch.isnan(out[k]).any(), f"{k} holds NaN: something was left unwritten or read before written"
    # the oracle works from its own advantages; nothing it sees comes from the CUDA path
    oo = _oracle_case(w, o_adv_tok, token_weight=None if token_weight is None else _np64(token_weight),
                      seq_offsets=w.seq_offsets.cpu().numpy(), agg_mode=agg_mode, sequence_level=sequence_level)
    m = w.mask.cpu().numpy().astype(bool)
    assert np.abs(_np64(out["logp"]) - oo["logp"]).max() <= TOL_LOGP
    assert np.abs(_np64(out["entropy"]) - oo["entropy"]).max() <= TOL_ENT
    assert np.all(_np64(out["logp"])[~m] == 0) and np.all(_np64(out["entropy"])[~m] == 0)
    # the clip decision is taken in fp32 on the GPU: tokens whose ratio sits on a clip boundary
    # within rounding may legitimately fall on either side; the seeds used here have none
    rho = oo["rho"]
    if rho.size:
        dist = np.minimum(np.abs(rho - (1 - w.eps_low)), np.abs(rho - (1 + w.eps_high)))
        assert dist.min() > boundary_margin, "a token sits on the clip boundary; pick another seed"
    loss = float(out["loss"].item())
    assert abs(loss - oo["loss"]) <= TOL_LOSS_REL * abs(oo["loss"]) + 1e-7
    dH = _np64(out["dH"])
    assert not dH[~m].any()
    assert _rel(dH, oo["dH"]) <= TOL_GRAD_REL
    assert _rel(_np64(out["dW"]), oo["dW"]) <= TOL_GRAD_REL
    _assert_blockwise(dH[m], oo["dH"][m], 1, "dH row")
    _assert_blockwise(_np64(out["dW"]), oo["dW"], 128, "dW 128-row block")
    met = _np64(out["metrics"])
    assert abs(met[0] - oo["pg_loss"]) <= 1e-3 * abs(oo["pg_loss"]) + 1e-7
    assert abs(met[1] - oo["kl_mean"]) <= 1e-3 * abs(oo["kl_mean"]) + 1e-7
    assert abs(met[2] - oo["entropy_mean"]) <= 2e-3
    assert abs(met[3] - oo["clip_frac"]) <= 1e-6
    assert met[6] == m.sum()
    return out, oo


# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("cta_group", [1, 2])
def test_gemm_engine_layouts(cta_group):
    # operand layouts of the tensor-core engine (single CTAs and CTA pairs) against a library product
    from paper_2512_21450_b200 import Context
    ctx = Context(0)
    ctx.set_cta_group(cta_group)
    g = torch.Generator(device="cuda").manual_seed(1)
    for (M, N, K) in [(128, 256, 64), (256, 512, 200), (384, 768, 2048), (1280, 256, 72)]:
        A = torch.randn(M, K, generator=g, device="cuda").to(torch.bfloat16)
        B = torch.randn(N, K, generator=g, device="cuda").to(torch.bfloat16)
        ref = A.float() @ B.float().T
        for a_mn in (0, 1):
            for b_mn in (0, 1):
                C = ctx.rl_selftest_gemm(A.T.contiguous() if a_mn else A, B.T.contiguous() if b_mn else B,
                                         M, N, K, a_mn, b_mn)
                _assert_status_ok(ctx)
                assert (C - ref).abs().max().item() <= 1e-4 * ref.abs().max().item()
                C2 = ctx.rl_selftest_gemm(A.T.contiguous() if a_mn else A, B.T.contiguous() if b_mn else B,
                                          M, N, K, a_mn, b_mn, C=C.clone(), accumulate=True)
                assert (C2 - 2 * ref).abs().max().item() <= 2e-4 * ref.abs().max().item()
    ctx.close()


def test_wide_and_square_gradient_tiles():
    # dH and dW run on 256 x 512 tiles by default; the 256 x 256 tiles must give the same bits (every
    # output element is the same sum in the same order), on shapes where the last wide tile is half
    # empty (d = 256, 768, 2304) and where several slabs accumulate
    from paper_2512_21450_b200 import Context
    from paper_2512_21450_b200.workloads import make_workload
    wide, square = Context(0), Context(0)
    try:
        square.set_wide_tiles(False)
        g = torch.Generator(device="cuda").manual_seed(5)
        for (M, N, K) in [(256, 512, 64), (256, 256, 200), (384, 768, 2048), (1280, 1280, 72)]:
            A = torch.randn(M, K, generator=g, device="cuda").to(torch.bfloat16)
            B = torch.randn(N, K, generator=g, device="cuda").to(torch.bfloat16)
            ref = A.float() @ B.float().T
            for a_mn in (0, 1):
                for b_mn in (0, 1):
                    args = (A.T.contiguous() if a_mn else A, B.T.contiguous() if b_mn else B, M, N, K, a_mn, b_mn)
                    C = wide.rl_selftest_gemm(*args)
                    _assert_status_ok(wide)
                    assert (C - ref).abs().max().item() <= 1e-4 * ref.abs().max().item()
                    assert torch.equal(C, square.rl_selftest_gemm(*args))
                    C2 = wide.rl_selftest_gemm(*args, C=C.clone(), accumulate=True)
                    assert (C2 - 2 * ref).abs().max().item() <= 2e-4 * ref.abs().max().item()
        for kw in (dict(cfg_id=0, L_max=13, V=4100, seed=710), dict(cfg_id=1, prompts=1, L_max=40, d=768, V=30000, seed=711),
                   dict(cfg_id=1, prompts=1, L_max=24, d=2304, V=5000, seed=712)):
            w = make_workload(kw.pop("cfg_id"), **kw)
            a, _ = _check_against_oracle(wide, w)
            a = {k: v.clone() for k, v in a.items()}
            b, _ = _check_against_oracle(square, w)
            for k in ("loss", "dH", "dW"):
                assert torch.equal(a[k], b[k]), k
    finally:
        wide.close()
        square.close()


def test_single_cta_tiles_match_oracle():
    # the default context runs CTA pairs; the single-CTA tile shape must give the same results
    from paper_2512_21450_b200 import Context
    from paper_2512_21450_b200.workloads import make_workload
    c1 = Context(0)
    try:
        c1.set_cta_group(1)
        _check_against_oracle(c1, make_workload(0, L_max=13, V=4100, seed=700))
        _check_against_oracle(c1, make_workload(1, prompts=1, L_max=40, seed=701))
    finally:
        c1.close()


@pytest.mark.parametrize("T", [1, 15, 16, 17, 4095, 4096, 4097, 70001, (1 << 20) + 3])
def test_mask_scan_row_map_is_exact(ctx, T):
    # integer work: the row map and the count must equal the oracle's bit for bit
    rng = np.random.default_rng(T)
    for p_valid in (0.0, 0.55, 1.0):
        m_np = (rng.uniform(size=T) < p_valid).astype(np.uint8) * rng.integers(1, 256, size=T).astype(np.uint8)
        backing = torch.zeros(T + 1, dtype=torch.uint8, device="cuda")
        for off in (0, 1):                               # 16-byte aligned and unaligned mask pointers
            mask = backing[off:off + T]
            mask.copy_(torch.from_numpy(m_np))
            row_map, n_valid = ctx.rl_mask_scan(mask)
            expect = O.valid_row_map(m_np.tolist())
            assert n_valid.item() == len(expect)
            assert row_map[:len(expect)].cpu().tolist() == expect
    row_map, n_valid = ctx.rl_mask_scan(None, T=T)       # no mask: every row
    assert n_valid.item() == T and row_map.cpu().tolist() == O.valid_row_map(None, T)
    _assert_status_ok(ctx)


# from 2048 groups of 4, 8, ... 32 responses on, the library runs one thread per group instead of shuffle segments
@pytest.mark.parametrize("n_groups,G", [(4, 4), (8, 8), (64, 16), (7, 5), (3, 40), (1024, 8), (9, 2), (5, 32), (3, 33),
                                        (100, 3), (2048, 8), (5000, 4), (3001, 12), (2500, 16), (2049, 28), (2048, 32),
                                        (4000, 6), (2047, 8)])
def test_advantages(ctx, n_groups, G):
    rng = np.random.default_rng(100 + G)
    for kind in ("bernoulli", "uniform", "zero_var"):
        if kind == "bernoulli":
            r = (rng.uniform(size=n_groups * G) < 0.4).astype(np.float32)
        elif kind == "uniform":
            r = rng.uniform(size=n_groups * G).astype(np.float32)
        else:
            r = np.repeat(rng.uniform(size=n_groups).astype(np.float32), G)
        rt = torch.from_numpy(r).cuda()
        for ddof in (0, 1):
            a = ctx.rl_grpo_advantages(rt, G, ddof=ddof, eps_std=1e-6)
            o = O.grpo_advantages(r, G, ddof=ddof, eps_std=1e-6)
            assert np.abs(_np64(a) - o).max() <= TOL_ADV
            if kind == "zero_var":
                assert not _np64(a).any()


# the big_* cases have more than 2^20 rows: several 8192-row block shares per block, searches that span many responses
@pytest.mark.parametrize("case", ["long", "short", "ragged", "empty_ranges", "inner_span", "one_row",
                                  "big_long", "big_short", "big_tiny", "big_ragged", "big_empty_inner", "big_one"])
def test_advantage_broadcast_is_exact(ctx, case):
    # a copy: every row must carry exactly its response's value, rows outside the span of the ranges 0
    rng = np.random.default_rng(sum(map(ord, case)))
    G = 4
    if case == "long":
        lens = rng.integers(3000, 9000, size=16)
    elif case == "short":
        lens = rng.integers(1, 9, size=4096)
    elif case == "ragged":
        lens = np.concatenate([rng.integers(1, 5, size=300), rng.integers(500, 3000, size=20)])
        rng.shuffle(lens)
    elif case == "empty_ranges":
        lens = rng.integers(0, 40, size=2000) * (rng.uniform(size=2000) < 0.3)
        lens[:700] = 0
        lens[700] = 5
    elif case == "inner_span":
        lens = rng.integers(10, 2000, size=64)
    elif case == "big_long":
        lens = rng.integers(64, 4097, size=1024)            # about 2.1 M rows, a few responses per 8192-row block share
    elif case == "big_short":
        lens = rng.integers(1, 17, size=160000)             # about 1.4 M rows, a thousand responses per block share
    elif case == "big_tiny":
        lens = np.concatenate([np.ones(40000, dtype=np.int64), rng.integers(0, 3, size=600000),
                               rng.integers(2000, 9000, size=100)])   # thousands of responses per 8192-row block share
    elif case == "big_ragged":
        lens = np.concatenate([rng.integers(1, 5, size=3000), rng.integers(20000, 90000, size=24)])
        rng.shuffle(lens)
    elif case == "big_empty_inner":
        lens = rng.integers(100, 3000, size=900) * (rng.uniform(size=900) < 0.8)
        lens[:50] = 0                                       # the span starts with empty ranges, inside a block share
    elif case == "big_one":
        lens = np.array([1 << 20, 1, 0, 5], dtype=np.int64)
    else:
        lens = np.ones(4, dtype=np.int64)
    inner = case in ("inner_span", "big_empty_inner", "big_ragged")
    first = 1237 if inner else 0
    off = np.concatenate([[first], first + np.cumsum(lens)]).astype(np.int32)
    T = int(off[-1]) + (4321 if inner else 0)
    if case.startswith("big"):
        T = max(T, (1 << 20) + 13)
    if case == "ragged":
        T += 3                                              # rows past the last range, T not a multiple of 4
    n_seq = len(lens)
    r = rng.uniform(size=n_seq).astype(np.float32)
    adv_seq, adv_tok = ctx.rl_grpo_advantages(torch.from_numpy(r).cuda(), G, seq_offsets=torch.from_numpy(off).cuda(), T=T)
    _assert_status_ok(ctx)
    expect = O.broadcast_to_tokens(O.grpo_advantages(r, G), off, T)
    got = _np64(adv_tok)
    assert got.shape == (T,) and np.abs(got - expect).max() <= TOL_ADV
    outside = np.ones(T, dtype=bool)
    outside[off[0]:off[-1]] = False
    assert not got[outside].any()                             # rows outside the span of the ranges: exactly 0
    # property of the copy: a row holds bit for bit what the call returned for its response
    assert np.array_equal(got[off[0]:off[-1]], np.repeat(_np64(adv_seq), lens))


@pytest.mark.parametrize("n_groups,G", [(8, 8), (5, 3), (64, 16), (3, 40), (2048, 8)])
def test_other_advantage_estimators(ctx, n_groups, G):
    rng = np.random.default_rng(300 + G)
    r = rng.uniform(size=n_groups * G).astype(np.float32)
    ln = rng.integers(1, 513, size=n_groups * G).astype(np.int32)
    rt, lt = torch.from_numpy(r).cuda(), torch.from_numpy(ln).cuda()
    # rewards are O(1); fp32 arithmetic on them stays within the advantage tolerance
    assert np.abs(_np64(ctx.rl_advantages("rloo", rt, G)) - O.rloo_advantages(r, G)).max() <= TOL_ADV
    assert np.abs(_np64(ctx.rl_advantages("opo", rt, G, lengths=lt)) - O.opo_advantages(r, ln, G)).max() <= TOL_ADV
    assert np.abs(_np64(ctx.rl_advantages("grpo", rt, G)) - O.grpo_advantages(r, G)).max() <= TOL_ADV
    # batch-normalised values are O(3): allow a few fp32 ulps of that
    pp = _np64(ctx.rl_advantages("reinforce_pp", rt, G))
    assert np.abs(pp - O.reinforce_pp_advantages(r, G)).max() <= 4e-6


def test_config0_full(ctx):
    from paper_2512_21450_b200.workloads import make_workload
    w = make_workload(0)
    assert w.T == 256 and w.n_valid == 256
    lp, ent, lse = ctx.rl_token_logprobs(w.H, w.W, w.tokens, w.mask)
    _assert_status_ok(ctx)
    olp, oent, olse = O.token_logprobs(_np64(w.H), _np64(w.W), w.tokens.cpu().numpy(), w.mask.cpu().numpy())
    assert np.abs(_np64(lp) - olp).max() <= TOL_LOGP
    assert np.abs(_np64(ent) - oent).max() <= TOL_ENT
    assert np.abs(_np64(lse) - olse).max() <= TOL_LOGP
    _check_against_oracle(ctx, w)


@pytest.mark.parametrize("cfg_id,prompts,L_max", [(1, 1, 96), (2, 1, 64), (3, 2, 64), (4, 4, 24)])
def test_reduced_configs(ctx, cfg_id, prompts, L_max):
    # same d, V, distributions and masks as the full configuration, fewer prompts / shorter rows
    from paper_2512_21450_b200.workloads import make_workload
    w = make_workload(cfg_id, prompts=prompts, L_max=L_max)
    assert w.n_valid > 128 and w.n_valid % 128 != 0      # several row tiles and a ragged tail
    if cfg_id == 4:
        r = w.rewards.cpu().numpy().reshape(-1, w.G)
        assert (r.max(axis=1) == r.min(axis=1)).any()     # a zero-variance group is present
        assert w.ref_logp is None and w.ent_coef > 0
    _check_against_oracle(ctx, w)


@pytest.mark.parametrize("agg_mode,sequence_level", [(1, False), (2, False), (0, True), (1, True), (2, True)])
def test_aggregation_modes_and_sequence_level_ratio(ctx, agg_mode, sequence_level):
    from paper_2512_21450_b200.workloads import make_workload
    # ragged right-padded responses (3B-class head), and responses with masked spans inside
    def shift_behaviour_policy(w):
        # the sequence-level ratio averages the token noise away; a per-response offset of the
        # behaviour log-probs puts some responses outside the clip band and leaves others inside
        bias = torch.tensor([0.45, 0.0, -0.45, 0.1], device=w.old_logp.device).repeat(w.n_seq // 4 + 1)[:w.n_seq]
        w.old_logp = (w.old_logp + bias.repeat_interleave(w.L_max)) * w.mask

    w = make_workload(1, prompts=1, L_max=96, seed=800 + agg_mode, sigma_old=0.3)
    shift_behaviour_policy(w)
    out, oo = _check_against_oracle(ctx, w, agg_mode=agg_mode, sequence_level=sequence_level,
                                    dH_fp32=(agg_mode == 2))
    if sequence_level:
        assert 0.0 < oo["clip_frac"] < 1.0            # some responses clipped, some not
    w = make_workload(3, prompts=2, L_max=64, seed=810 + agg_mode, d=256, V=5000, sigma_old=0.3)
    shift_behaviour_policy(w)
    _check_against_oracle(ctx, w, agg_mode=agg_mode, sequence_level=sequence_level)


@pytest.mark.parametrize("agg_mode,sequence_level", [(0, True), (1, False), (2, True)])
def test_valid_rows_outside_every_response_range(ctx, agg_mode, sequence_level):
    # the response ranges cover only part of the rows: valid rows before the first and after the last
    # range take no part in the loss (outputs of the forward still cover them), and the token mean of
    # agg_mode 0 is over the rows inside ranges
    from paper_2512_21450_b200.workloads import make_workload
    w = make_workload(1, prompts=1, L_max=40, d=256, V=3000, seed=520 + agg_mode)
    off = w.seq_offsets.clone()
    inner = off[2:7].contiguous()                      # responses 2..5 only
    adv = torch.randn(w.T, device="cuda")
    out = ctx.rl_policy_loss_fwd_bwd(w.H, w.W, w.tokens, w.old_logp, w.ref_logp, adv, w.mask, w.eps_low, w.eps_high,
                                     w.beta, ent_coef=0.01, agg_mode=agg_mode, sequence_level=sequence_level,
                                     seq_offsets=inner)
    _assert_status_ok(ctx)
    oo = O.policy_loss_fwd_bwd(_np64(w.H), _np64(w.W), w.tokens.cpu().numpy(), _np64(w.old_logp), _np64(w.ref_logp),
                               _np64(adv), w.mask.cpu().numpy(), w.eps_low, w.eps_high, w.beta, ent_coef=0.01,
                               seq_offsets=inner.cpu().numpy(), agg_mode=agg_mode, sequence_level=sequence_level)
    assert abs(out["loss"].item() - oo["loss"]) <= TOL_LOSS_REL * abs(oo["loss"]) + 1e-7
    dH = _np64(out["dH"])
    lo, hi = int(inner[0]), int(inner[-1])
    assert not dH[:lo].any() and not dH[hi:].any()
    assert _rel(dH, oo["dH"]) <= TOL_GRAD_REL and _rel(_np64(out["dW"]), oo["dW"]) <= TOL_GRAD_REL


@pytest.mark.parametrize("cta_group", [2, 1])
@pytest.mark.parametrize("cfg_id,prompts,L_max,d_ref,V,ent", [
    (0, None, None, None, None, 0.0),      # config 0 as it stands, reference = drifted policy
    (1, 1, 40, 192, 4100, 0.01),           # reference model of another width, ragged vocabulary tail
    (3, 2, 64, None, 600, 0.0),            # several row slabs and column slabs (limits set below)
])
def test_full_distribution_kl(cta_group, cfg_id, prompts, L_max, d_ref, V, ent):
    """Regulariser = sum_j p_j (log p_j - log q_j) over the whole vocabulary (sections 2.2 / 3.1),
    q from a second hidden-state / LM-head pair; loss, metrics, dH and dW against the oracle."""
    from paper_2512_21450_b200 import Context
    from paper_2512_21450_b200.workloads import make_workload, make_reference_model
    c = Context(0)
    try:
        try:
            c.set_cta_group(cta_group)
        except RuntimeError:
            pytest.skip("CTA pairs cannot be co-scheduled on this device")
        kw = {} if cfg_id == 0 else dict(prompts=prompts, L_max=L_max, d=128, V=V)
        w = make_workload(cfg_id, **kw)
        if cfg_id == 3:
            c.set_slab_limits(128, 256)
        beta = w.beta if w.beta > 0 else 0.04
        H_ref, W_ref = make_reference_model(w, d_ref=d_ref, drift=0.3)
        adv_seq, adv_tok = c.rl_grpo_advantages(w.rewards, w.G, seq_offsets=w.seq_offsets, T=w.T)
        out = c.rl_policy_loss_fwd_bwd(w.H, w.W, w.tokens, w.old_logp, None, adv_tok, w.mask, w.eps_low,
                                       w.eps_high, beta, ent_coef=ent, H_ref=H_ref, W_ref=W_ref)
        status, detail = c.last_device_status()
        assert status == 0, (status, hex(detail & 0xffffffff))
        o_adv_tok = O.broadcast_to_tokens(O.grpo_advantages(w.rewards.cpu().numpy(), w.G),
                                          w.seq_offsets.cpu().numpy(), w.T)
        oo = O.policy_loss_fwd_bwd(_np64(w.H), _np64(w.W), w.tokens.cpu().numpy(), _np64(w.old_logp), None,
                                   o_adv_tok, w.mask.cpu().numpy(), w.eps_low, w.eps_high, beta, ent_coef=ent,
                                   H_ref=_np64(H_ref), W_ref=_np64(W_ref))
        assert oo["kl_mean"] > 1e-4          # the regulariser is really exercised
        assert np.abs(_np64(out["logp"]) - oo["logp"]).max() <= TOL_LOGP
        assert np.abs(_np64(out["entropy"]) - oo["entropy"]).max() <= TOL_ENT
        met = _np64(out["metrics"])
        # KL_t is a difference of fp32 quantities of the size of lse (about 10): a few ulp of that
        assert abs(met[1] - oo["kl_mean"]) <= 2e-3 * abs(oo["kl_mean"]) + 5e-6
        assert abs(out["loss"].item() - oo["loss"]) <= TOL_LOSS_REL * abs(oo["loss"]) + 1e-6
        m = w.mask.cpu().numpy().astype(bool)
        dH = _np64(out["dH"])
        assert not dH[~m].any()
        assert _rel(dH, oo["dH"]) <= TOL_GRAD_REL
        assert _rel(_np64(out["dW"]), oo["dW"]) <= TOL_GRAD_REL
        # the gradient of the regulariser alone (no advantage signal): compare at A = 0
        zero_adv = torch.zeros_like(adv_tok)
        out0 = c.rl_policy_loss_fwd_bwd(w.H, w.W, w.tokens, w.old_logp, None, zero_adv, w.mask, w.eps_low,
                                        w.eps_high, beta, H_ref=H_ref, W_ref=W_ref)
        oo0 = O.policy_loss_fwd_bwd(_np64(w.H), _np64(w.W), w.tokens.cpu().numpy(), _np64(w.old_logp), None,
                                    np.zeros(w.T), w.mask.cpu().numpy(), w.eps_low, w.eps_high, beta,
                                    H_ref=_np64(H_ref), W_ref=_np64(W_ref))
        assert _rel(_np64(out0["dH"]), oo0["dH"]) <= TOL_GRAD_REL
        assert _rel(_np64(out0["dW"]), oo0["dW"]) <= TOL_GRAD_REL
        assert abs(out0["loss"].item() - oo0["loss"]) <= TOL_LOSS_REL * abs(oo0["loss"]) + 1e-6
    finally:
        c.close()


def test_full_kl_argument_checks(ctx):
    from paper_2512_21450_b200.workloads import make_workload, make_reference_model
    w = make_workload(0)
    H_ref, W_ref = make_reference_model(w)
    adv = torch.zeros(w.T, device=w.H.device)
    # not combined with the sequence-level path
    with pytest.raises(RuntimeError):
        ctx.rl_policy_loss_fwd_bwd(w.H, w.W, w.tokens, w.old_logp, None, adv, w.mask, 0.2, 0.2, 0.04,
                                   H_ref=H_ref, W_ref=W_ref, sequence_level=True, seq_offsets=w.seq_offsets)
    # the reference hidden size must be a whole number of 64-element k-slices
    with pytest.raises(RuntimeError):
        ctx.rl_policy_loss_fwd_bwd(w.H, w.W, w.tokens, w.old_logp, None, adv, w.mask, 0.2, 0.2, 0.04,
                                   H_ref=H_ref[:, :40].contiguous(), W_ref=W_ref[:, :40].contiguous())
    _assert_status_ok(ctx)


def test_clip_exercised_and_peaked_rows(ctx):
    from paper_2512_21450_b200.workloads import make_workload
    w = make_workload(0, sigma_old=0.3, peaked_frac=0.05, seed=77)
    out, oo = _check_against_oracle(ctx, w)
    assert 0.05 < oo["clip_frac"] < 0.6                   # the clip is active on a real share of tokens
    assert oo["entropy"][w.mask.cpu().numpy().astype(bool)].min() < 1.0   # peaked rows present
    w = make_workload(4, prompts=2, L_max=16, sigma_old=0.3, seed=78, d=256, V=5000)
    _check_against_oracle(ctx, w)


@pytest.mark.parametrize("V,L_max", [(4096, 13), (4000, 16), (4100, 16), (300, 9), (37888 + 256 + 40, 11)])
def test_ragged_shapes(ctx, V, L_max):
    # rows not a multiple of 128, vocabulary not a multiple of 256 / 32, more than one vocabulary slab
    from paper_2512_21450_b200.workloads import make_workload
    w = make_workload(0, L_max=L_max, V=V, seed=500 + V)
    _check_against_oracle(ctx, w)


@pytest.mark.parametrize("d,V,L_max", [(64, 300, 16), (64, 1, 5), (128, 2, 16), (192, 777, 1), (64, 70000, 3)])
def test_extreme_shapes(ctx, d, V, L_max):
    # smallest hidden size the TMA layout allows, one- and two-word vocabularies (entropy 0 /
    # gradient exactly zero for V = 1), a single row per response, a vocabulary with many slabs
    from paper_2512_21450_b200.workloads import make_workload
    w = make_workload(0, L_max=L_max, d=d, V=V, seed=600 + V)
    out, oo = _check_against_oracle(ctx, w)
    if V == 1:
        assert not out["dH"].any() and not out["dW"].any() and not out["logp"].any()


@pytest.mark.parametrize("cta_group", [2, 1])
def test_row_groups(cta_group):
    # the rows-first passes take the row tiles in groups that fit an L2 budget: any grouping must give
    # bit for bit what one group gives (only the order in which tiles are visited changes), several
    # groups, a ragged last group, several vocabulary slabs and ranges
    from paper_2512_21450_b200 import Context
    from paper_2512_21450_b200.workloads import make_workload
    w = make_workload(1, prompts=1, L_max=400, d=256, V=3000, seed=87)
    assert w.n_valid > 1400                                   # at least 6 row tiles of 256 / 11 of 128
    panel = 128 * cta_group * w.d * 2
    c2 = Context(0)
    try:
        c2.set_cta_group(cta_group)
        c2.set_slab_limits(32768, 1024)
        c2.set_row_group_bytes(0)
        base, _ = _check_against_oracle(c2, w)
        base = {k: v.clone() for k, v in base.items()}
        for tiles in (1, 2, 4, 5, 1000):
            c2.set_row_group_bytes(tiles * panel)
            out, _ = _check_against_oracle(c2, w)
            for k in ("loss", "dH", "dW", "logp", "entropy"):
                assert torch.equal(out[k], base[k]), (tiles, k)
        # the two-product passes of the full-distribution KL walk their tiles through the same function
        from paper_2512_21450_b200.workloads import make_reference_model
        H_ref, W_ref = make_reference_model(w, d_ref=128)
        _, adv_tok = c2.rl_grpo_advantages(w.rewards, w.G, seq_offsets=w.seq_offsets, T=w.T)
        kl = []
        for nbytes in (0, 2 * 128 * cta_group * (w.d + 128) * 2):
            c2.set_row_group_bytes(nbytes)
            o = c2.rl_policy_loss_fwd_bwd(w.H, w.W, w.tokens, w.old_logp, None, adv_tok, w.mask, w.eps_low, w.eps_high,
                                          0.05, H_ref=H_ref, W_ref=W_ref)
            _assert_status_ok(c2)
            kl.append({k: v.clone() for k, v in o.items()})
        for k in ("loss", "dH", "dW", "kl"):
            assert torch.equal(kl[0][k], kl[1][k]), k
    finally:
        c2.close()


def test_wide_hidden_size(ctx):
    # d = 8192, four times the hidden size of the 3B-class head: 128 k-slices per logit tile, 32 column tiles in the dH and dW passes.  The entropy-bonus configuration keeps the loss
    # away from the near-zero value that equal-length GRPO groups otherwise cancel to.
    from paper_2512_21450_b200.workloads import make_workload
    _check_against_oracle(ctx, make_workload(4, prompts=1, L_max=5, d=8192, V=1500, seed=640))


def test_multiple_slabs(ctx):
    # force several row slabs and several vocabulary slabs on a small case
    from paper_2512_21450_b200 import Context
    from paper_2512_21450_b200.workloads import make_workload
    c2 = Context(0)
    try:
        c2.set_slab_limits(128, 512)
        w = make_workload(1, prompts=1, L_max=64, d=128, V=1500, seed=9)
        assert w.n_valid > 256
        _check_against_oracle(c2, w)
    finally:
        c2.close()


@pytest.mark.parametrize("slices", [2, 3, 4])
def test_dh_k_slices(slices):
    # dH tiles cut along K into separately accumulated slices: same result, several slabs and CTA shapes
    from paper_2512_21450_b200 import Context
    from paper_2512_21450_b200.workloads import make_workload
    c2 = Context(0)
    try:
        c2.set_dh_k_slices(slices)
        c2.set_slab_limits(256, 512)
        _check_against_oracle(c2, make_workload(1, prompts=1, L_max=64, d=256, V=1500, seed=19 + slices))
        c2.set_slab_limits(0, 0)
        _check_against_oracle(c2, make_workload(0, L_max=13, V=4100, seed=29 + slices))     # a 1-block K range
        if slices == 3:
            c2.set_cta_group(1)
            _check_against_oracle(c2, make_workload(1, prompts=1, L_max=40, seed=39))
    finally:
        c2.close()


@pytest.mark.parametrize("cta_group,wide", [(2, False), (2, True), (1, False)])
def test_dh_stream_k(cta_group, wide):
    # dH tiles balanced over the SMs by stream-K: a case with more tiles than workers and a ragged last
    # wave (10 row tiles of 256 x 8 column tiles = 80 tiles on 74 pairs; 160 on 148 single CTAs), several
    # vocabulary slabs (parts are added to what earlier slabs left) - against the oracle, against the
    # plain tile loop, and bitwise reproducible
    from paper_2512_21450_b200 import Context
    from paper_2512_21450_b200.workloads import make_workload
    # on 256 x 512 tiles the same ragged wave needs twice the rows: 20 row tiles x 4 wide tiles = 80 on 74 pairs
    w = make_workload(1, prompts=2 if wide else 1, L_max=640, V=1200, seed=83)
    assert (4864 < w.n_valid <= 5120) if wide else (2304 < w.n_valid <= 2560)
    c2 = Context(0)
    try:
        c2.set_cta_group(cta_group)
        c2.set_wide_tiles(wide)
        c2.set_slab_limits(32768, 512)
        c2.set_dh_stream_k(True)
        out, _ = _check_against_oracle(c2, w)
        first = out["dH"].clone()
        again, _ = _check_against_oracle(c2, w)
        assert torch.equal(first, again["dH"])
        c2.set_dh_stream_k(False)
        plain, _ = _check_against_oracle(c2, w)
        assert _rel(_np64(first), _np64(plain["dH"])) <= 1e-2
        # fp32 dH leaves the two accumulator buffers without a bf16 rounding in between
        c2.set_dh_stream_k(True)
        a32, _ = _check_against_oracle(c2, w, dH_fp32=True)
        c2.set_dh_stream_k(False)
        b32, _ = _check_against_oracle(c2, w, dH_fp32=True)
        assert _rel(_np64(a32["dH"]), _np64(b32["dH"])) <= 1e-5
    finally:
        c2.close()


def test_token_weight_accumulate_and_strides(ctx):
    from paper_2512_21450_b200.workloads import make_workload
    w = make_workload(0, seed=31)
    g = torch.Generator(device="cuda").manual_seed(5)
    tw = torch.rand(w.T, generator=g, device="cuda") / w.T
    _check_against_oracle(ctx, w, token_weight=tw)
    # accumulate_dW adds to what is there; strided H (ldH > d) is read correctly
    adv_seq, adv_tok = ctx.rl_grpo_advantages(w.rewards, w.G, seq_offsets=w.seq_offsets, T=w.T)
    base = ctx.rl_policy_loss_fwd_bwd(w.H, w.W, w.tokens, w.old_logp, w.ref_logp, adv_tok, w.mask,
                                      w.eps_low, w.eps_high, w.beta)
    dW0 = base["dW"].clone()
    Hwide = torch.zeros(w.T, w.d + 64, dtype=torch.bfloat16, device="cuda")
    Hwide[:, :w.d] = w.H
    acc = ctx.rl_policy_loss_fwd_bwd(Hwide[:, :w.d], w.W, w.tokens, w.old_logp, w.ref_logp, adv_tok, w.mask,
                                     w.eps_low, w.eps_high, w.beta, accumulate_dW=True, dW=dW0.clone())
    _assert_status_ok(ctx)
    assert torch.allclose(acc["dW"], 2 * dW0, rtol=1e-5, atol=1e-12)
    # a weight matrix that is a column slice of a wider one (ldW > d)
    Wwide = torch.zeros(w.V, w.d + 128, dtype=torch.bfloat16, device="cuda")
    Wwide[:, :w.d] = w.W
    strided = ctx.rl_policy_loss_fwd_bwd(w.H, Wwide[:, :w.d], w.tokens, w.old_logp, w.ref_logp, adv_tok, w.mask,
                                         w.eps_low, w.eps_high, w.beta)
    assert torch.equal(strided["dW"], dW0) and torch.equal(strided["dH"], base["dH"])
    assert torch.equal(acc["dH"], base["dH"])
    assert acc["loss"].item() == base["loss"].item()     # deterministic reductions


def test_degenerate_batches(ctx):
    from paper_2512_21450_b200.workloads import make_workload
    w = make_workload(0, seed=41)
    adv = torch.ones(w.T, device="cuda")
    # all rows masked: loss 0, gradients 0, no error
    zero_mask = torch.zeros_like(w.mask)
    out = ctx.rl_policy_loss_fwd_bwd(w.H, w.W, w.tokens, w.old_logp, w.ref_logp, adv, zero_mask,
                                     w.eps_low, w.eps_high, w.beta)
    _assert_status_ok(ctx)
    assert out["loss"].item() == 0 and not out["dH"].any() and not out["dW"].any()
    assert not out["logp"].any()
    # a single valid row
    one = torch.zeros_like(w.mask)
    one[37] = 1
    out = ctx.rl_policy_loss_fwd_bwd(w.H, w.W, w.tokens, w.old_logp, w.ref_logp, adv, one,
                                     w.eps_low, w.eps_high, w.beta)
    oo = O.policy_loss_fwd_bwd(_np64(w.H), _np64(w.W), w.tokens.cpu().numpy(), _np64(w.old_logp),
                               _np64(w.ref_logp), _np64(adv), one.cpu().numpy(), w.eps_low, w.eps_high, w.beta)
    assert abs(out["loss"].item() - oo["loss"]) <= TOL_LOSS_REL * abs(oo["loss"]) + 1e-7
    assert _rel(_np64(out["dH"]), oo["dH"]) <= TOL_GRAD_REL and _rel(_np64(out["dW"]), oo["dW"]) <= TOL_GRAD_REL
    # mask = NULL means all valid
    lp_all, _, _ = ctx.rl_token_logprobs(w.H, w.W, w.tokens, None)
    lp_m, _, _ = ctx.rl_token_logprobs(w.H, w.W, w.tokens, torch.ones_like(w.mask))
    assert torch.equal(lp_all, lp_m)
    # T = 0
    e = torch.empty(0, w.d, dtype=torch.bfloat16, device="cuda")
    ei = torch.empty(0, dtype=torch.int32, device="cuda")
    ef = torch.empty(0, dtype=torch.float32, device="cuda")
    out = ctx.rl_policy_loss_fwd_bwd(e, w.W, ei, ef, ef, ef, None, 0.2, 0.2, 0.04, want_aux=False)
    assert out["loss"].item() == 0 and not out["dW"].any()
    _assert_status_ok(ctx)


def test_error_reporting(ctx):
    from paper_2512_21450_b200 import Context, RLHeadError
    from paper_2512_21450_b200.workloads import make_workload
    w = make_workload(0, seed=51)
    adv = torch.ones(w.T, device="cuda")

    def status_of(fn):
        with pytest.raises(RLHeadError) as e:
            fn()
        return e.value.status

    args = (w.tokens, w.old_logp, w.ref_logp, adv, w.mask)
    assert status_of(lambda: ctx.rl_policy_loss_fwd_bwd(w.H, w.W, *args, 1.5, 0.2, 0.04)) == 1     # eps_low
    assert status_of(lambda: ctx.rl_policy_loss_fwd_bwd(w.H, w.W, *args, 0.2, -1.0, 0.04)) == 1    # eps_high
    assert status_of(lambda: ctx.rl_policy_loss_fwd_bwd(w.H, w.W, *args, 0.2, 0.2, -0.1)) == 1     # beta
    assert status_of(lambda: ctx.rl_policy_loss_fwd_bwd(w.H, w.W, w.tokens, w.old_logp, None, adv, w.mask,
                                                        0.2, 0.2, 0.04)) == 1                       # ref missing
    H_bad = torch.zeros(w.T, 96, dtype=torch.bfloat16, device="cuda")
    W_bad = torch.zeros(w.V, 96, dtype=torch.bfloat16, device="cuda")
    assert status_of(lambda: ctx.rl_token_logprobs(H_bad, W_bad, w.tokens, w.mask)) == 2           # d % 64
    H_off = torch.zeros(w.T * w.d + 8, dtype=torch.bfloat16, device="cuda")[4:4 + w.T * w.d].view(w.T, w.d)
    assert status_of(lambda: ctx.rl_token_logprobs(H_off, w.W, w.tokens, w.mask)) == 3             # 8-byte offset
    assert status_of(lambda: ctx.rl_grpo_advantages(w.rewards, 1)) == 2
    assert status_of(lambda: ctx.rl_grpo_advantages(w.rewards, 5)) == 2
    assert status_of(lambda: ctx.rl_grpo_advantages(w.rewards, 4, ddof=2, eps_std=1e-6)) == 1
    assert status_of(lambda: ctx.rl_advantages("opo", w.rewards, 4)) == 1                         # lengths missing
    assert status_of(lambda: ctx.rl_advantages("rloo", w.rewards, 1)) == 2
    assert status_of(lambda: ctx.set_cta_group(3)) == 1
    assert status_of(lambda: ctx.set_slab_limits(100, 256)) == 2
    assert status_of(lambda: ctx.rl_policy_loss_fwd_bwd(w.H, w.W, *args, 0.2, 0.2, 0.04, agg_mode=1)) == 1  # no offsets
    assert ctx.workspace_bytes(1024, 256, 4096) <= ctx.workspace_bytes(4096, 256, 4096) <= \
        ctx.workspace_bytes(4096, 512, 8192, host=True)
    # no workspace bound
    c2 = Context(0)
    try:
        lib = c2.lib
        import ctypes
        s = lib.rl_token_logprobs(c2.handle, ctypes.c_void_p(w.H.data_ptr()), w.d, ctypes.c_void_p(w.W.data_ptr()),
                                  w.d, ctypes.c_void_p(w.tokens.data_ptr()), None, w.T, w.d, w.V,
                                  ctypes.c_void_p(adv.data_ptr()), None, None)
        assert s == 4
    finally:
        c2.close()
    # token id outside the vocabulary on a valid row -> latched device status, context still usable
    bad = w.tokens.clone()
    bad[5] = w.V + 3
    ctx.rl_token_logprobs(w.H, w.W, bad, w.mask)
    s, detail = ctx.last_device_status()
    assert s == 7 and detail == 5
    masked = w.mask.clone()
    masked[5] = 0
    ctx.rl_token_logprobs(w.H, w.W, bad, masked)           # ignored on a masked row
    _assert_status_ok(ctx)
    lp, _, _ = ctx.rl_token_logprobs(w.H, w.W, w.tokens, w.mask)
    _assert_status_ok(ctx)
    assert torch.isfinite(lp).all()


def test_host_buffer_step_matches_device_call(ctx):
    # the host-buffer entry point (pinned inputs, advantages from rewards on the device) must give
    # exactly what the device-pointer calls give
    from paper_2512_21450_b200.workloads import make_workload
    for cfg_id, kw in ((0, dict(seed=91)), (4, dict(prompts=2, L_max=16, seed=92, d=256, V=5000))):
        w = make_workload(cfg_id, **kw)
        _, adv_tok = ctx.rl_grpo_advantages(w.rewards, w.G, seq_offsets=w.seq_offsets, T=w.T)
        ref = ctx.rl_policy_loss_fwd_bwd(w.H, w.W, w.tokens, w.old_logp, w.ref_logp, adv_tok, w.mask,
                                         w.eps_low, w.eps_high, w.beta, ent_coef=w.ent_coef)
        ref = {k: v.clone() for k, v in ref.items()}
        pin = lambda x: None if x is None else x.cpu().pin_memory()  # noqa: E731
        dH = torch.empty_like(ref["dH"])
        dW = torch.empty_like(ref["dW"])
        loss, metrics = ctx.rl_policy_loss_fwd_bwd_host(
            pin(w.H), w.W, pin(w.tokens), pin(w.old_logp), pin(w.ref_logp), None, pin(w.mask), w.eps_low,
            w.eps_high, w.beta, w.ent_coef, dH, dW, rewards_host=pin(w.rewards), group_size=w.G,
            seq_offsets_host=pin(w.seq_offsets))
        _assert_status_ok(ctx)
        assert loss == ref["loss"].item()
        assert torch.equal(dH, ref["dH"]) and torch.equal(dW, ref["dW"])
        assert np.allclose(metrics, ref["metrics"].cpu().numpy(), rtol=0, atol=0)
        # per-row advantages from the host instead of rewards
        loss2, _ = ctx.rl_policy_loss_fwd_bwd_host(
            pin(w.H), w.W, pin(w.tokens), pin(w.old_logp), pin(w.ref_logp), pin(adv_tok), pin(w.mask), w.eps_low,
            w.eps_high, w.beta, w.ent_coef, dH, dW)
        assert loss2 == ref["loss"].item() and torch.equal(dW, ref["dW"])


def test_pipelined_host_steps_match_the_blocking_call():
    # steps submitted two deep (the copies of step i+1 overlap the kernels of step i) must give exactly
    # what the blocking host call gives for each step's own inputs, with two workloads of the same shape
    # alternating so that a stale stage or result word would show; slot protocol errors are reported
    from paper_2512_21450_b200 import Context, RLHeadError
    from paper_2512_21450_b200.workloads import make_workload
    c = Context(0)
    try:
        ws = [make_workload(4, prompts=2, L_max=16, seed=95 + i, d=256, V=5000) for i in range(2)]
        pin = lambda x: None if x is None else x.cpu().pin_memory()  # noqa: E731
        hosts, expect = [], []
        for w in ws:
            h = dict(H=pin(w.H), tok=pin(w.tokens), old=pin(w.old_logp), ref=pin(w.ref_logp), mask=pin(w.mask),
                     rew=pin(w.rewards), off=pin(w.seq_offsets))
            hosts.append(h)
            dH = torch.empty(w.T, w.d, dtype=torch.bfloat16, device="cuda")
            dW = torch.empty(w.V, w.d, dtype=torch.float32, device="cuda")
            loss, metrics = c.rl_policy_loss_fwd_bwd_host(h["H"], w.W, h["tok"], h["old"], h["ref"], None, h["mask"], w.eps_low,
                                                          w.eps_high, w.beta, w.ent_coef, dH, dW, rewards_host=h["rew"],
                                                          group_size=w.G, seq_offsets_host=h["off"])
            expect.append((loss, metrics, dH.clone(), dW.clone()))
        assert expect[0][0] != expect[1][0]
        outs = [(torch.empty_like(expect[0][2]), torch.empty_like(expect[0][3])) for _ in range(2)]   # one dH / dW pair per slot

        def submit(step):
            k = step % 2
            w, h = ws[k], hosts[k]
            c.rl_policy_loss_fwd_bwd_host_submit(k, h["H"], w.W, h["tok"], h["old"], h["ref"], None, h["mask"], w.eps_low,
                                                 w.eps_high, w.beta, w.ent_coef, outs[k][0], outs[k][1],
                                                 rewards_host=h["rew"], group_size=w.G, seq_offsets_host=h["off"])

        n_steps = 7
        submit(0)
        for step in range(1, n_steps + 1):
            if step < n_steps:
                submit(step)
            k = (step - 1) % 2
            loss, metrics = c.rl_policy_loss_fwd_bwd_host_wait(k)
            assert loss == expect[k][0] and metrics == expect[k][1], step
            assert torch.equal(outs[k][0], expect[k][2]) and torch.equal(outs[k][1], expect[k][3]), step
        status, detail = c.last_device_status()
        assert status == 0, (status, detail)
        # protocol: waiting on an idle slot, submitting to a busy one, a slot that does not exist
        with pytest.raises(RLHeadError):
            c.rl_policy_loss_fwd_bwd_host_wait(0)
        submit(0)
        with pytest.raises(RLHeadError):
            submit(0)
        with pytest.raises(RLHeadError):
            c.rl_policy_loss_fwd_bwd_host_wait(2)
        c.rl_policy_loss_fwd_bwd_host_wait(0)
    finally:
        c.close()


def test_autograd_front_end(ctx):
    from paper_2512_21450_b200.autograd import fused_grpo_head_loss
    from paper_2512_21450_b200.workloads import make_workload
    w = make_workload(0, seed=95)
    o_adv = O.broadcast_to_tokens(O.grpo_advantages(w.rewards.cpu().numpy(), w.G), w.seq_offsets.cpu().numpy(), w.T)
    adv = torch.from_numpy(o_adv).float().cuda()
    H = w.H.clone().requires_grad_(True)
    W = w.W.clone().requires_grad_(True)
    loss, logp, ent, metrics = fused_grpo_head_loss(H, W, w.tokens, w.old_logp, w.ref_logp, adv, w.mask,
                                                    w.eps_low, w.eps_high, w.beta)
    (3.0 * loss).backward()
    oo = _oracle_case(w, o_adv)
    assert abs(loss.item() - oo["loss"]) <= TOL_LOSS_REL * abs(oo["loss"]) + 1e-7
    assert _rel(_np64(H.grad), 3.0 * oo["dH"]) <= TOL_GRAD_REL
    assert _rel(_np64(W.grad), 3.0 * oo["dW"]) <= TOL_GRAD_REL      # includes the rounding of dW to bf16
    assert not logp.requires_grad and np.abs(_np64(logp) - oo["logp"]).max() <= TOL_LOGP


def test_calls_can_be_captured_in_a_cuda_graph():
    # the calls neither allocate nor synchronise, so a whole step can be captured once and replayed
    from paper_2512_21450_b200 import Context
    from paper_2512_21450_b200.workloads import make_workload
    w = make_workload(0, seed=97)
    c2 = Context(0)
    try:
        c2.ensure_workspace(w.T, w.d, w.V)
        adv_seq = torch.empty_like(w.rewards)
        adv_tok = torch.empty(w.T, device="cuda")
        loss = torch.empty(1, device="cuda")
        dH = torch.empty(w.T, w.d, dtype=torch.bfloat16, device="cuda")
        dW = torch.empty(w.V, w.d, device="cuda")
        import ctypes
        P = ctypes.c_void_p

        def step():
            s1 = c2.lib.rl_grpo_advantages_ex(c2.handle, P(w.rewards.data_ptr()), w.n_seq, w.G, 1, 1e-6,
                                              P(w.seq_offsets.data_ptr()), w.T, P(adv_seq.data_ptr()),
                                              P(adv_tok.data_ptr()))
            s2 = c2.lib.rl_policy_loss_fwd_bwd(c2.handle, P(w.H.data_ptr()), w.d, P(w.W.data_ptr()), w.d,
                                               P(w.tokens.data_ptr()), P(w.old_logp.data_ptr()),
                                               P(w.ref_logp.data_ptr()), P(adv_tok.data_ptr()), P(w.mask.data_ptr()),
                                               w.T, w.d, w.V, w.eps_low, w.eps_high, w.beta, P(loss.data_ptr()),
                                               P(dH.data_ptr()), P(dW.data_ptr()))
            assert s1 == 0 and s2 == 0

        side = torch.cuda.Stream()
        with torch.cuda.stream(side):
            c2._bind_stream()
            step()                                   # eager reference run on the side stream
            torch.cuda.synchronize()
            ref = (loss.clone(), dH.clone(), dW.clone())
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                c2._bind_stream()
                step()
        for t in (loss, dH, dW):
            t.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(loss, ref[0]) and torch.equal(dH, ref[1]) and torch.equal(dW, ref[2])
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(dW, ref[2])
        assert c2.last_device_status()[0] == 0
    finally:
        c2.close()


def test_bounded_wait_times_out_cleanly(ctx):
    # a wait that nothing satisfies ends by itself, reports RL_ERR_TIMEOUT and leaves the context usable
    import time
    from paper_2512_21450_b200.workloads import make_workload
    t0 = time.time()
    ctx.selftest_wait_timeout(limit_ms=20)
    s, detail = ctx.last_device_status()
    assert s == 8 and (detail & 0xffffffff) == 0x70000000
    assert time.time() - t0 < 5.0
    assert ctx.last_device_status()[0] == 0           # cleared
    w = make_workload(0, seed=71)
    lp, _, _ = ctx.rl_token_logprobs(w.H, w.W, w.tokens, w.mask)
    _assert_status_ok(ctx)
    assert torch.isfinite(lp).all()


def test_run_to_run_determinism(ctx):
    from paper_2512_21450_b200.workloads import make_workload
    w = make_workload(1, prompts=1, L_max=40, seed=61)
    adv_seq, adv_tok = ctx.rl_grpo_advantages(w.rewards, w.G, seq_offsets=w.seq_offsets, T=w.T)
    a = ctx.rl_policy_loss_fwd_bwd(w.H, w.W, w.tokens, w.old_logp, w.ref_logp, adv_tok, w.mask, 0.2, 0.2, 0.04)
    a = {k: v.clone() for k, v in a.items()}
    b = ctx.rl_policy_loss_fwd_bwd(w.H, w.W, w.tokens, w.old_logp, w.ref_logp, adv_tok, w.mask, 0.2, 0.2, 0.04)
    for k in ("loss", "dH", "dW", "logp", "entropy"):
        assert torch.equal(a[k], b[k]), k


def test_global_token_count_and_gradient_hand_over(ctx):
    # data-parallel hooks on one GPU: (1) the token mean divided by a count handed in on the device equals
    # the same loss with explicit per-row weights 1 / count; (2) the dW slab hook reports every row of dW
    # exactly once, in ascending order, also with several row slabs; (3) a capped grid gives the same result
    from paper_2512_21450_b200 import Context
    from paper_2512_21450_b200.workloads import make_workload
    w = make_workload(1, prompts=1, L_max=64, d=256, V=3000, seed=905)
    adv_seq, adv_tok = ctx.rl_grpo_advantages(w.rewards, w.G, seq_offsets=w.seq_offsets, T=w.T)
    n_global = 3 * w.n_valid + 17                      # as if two more ranks held tokens
    cnt = torch.tensor([n_global], dtype=torch.int64, device="cuda")
    a = ctx.rl_policy_loss_fwd_bwd(w.H, w.W, w.tokens, w.old_logp, w.ref_logp, adv_tok, w.mask, w.eps_low, w.eps_high,
                                   w.beta, token_count=cnt)
    o_adv = O.broadcast_to_tokens(O.grpo_advantages(w.rewards.cpu().numpy(), w.G), w.seq_offsets.cpu().numpy(), w.T)
    oo = _oracle_case(w, o_adv, token_weight=np.full(w.T, 1.0 / n_global))
    assert abs(a["loss"].item() - oo["loss"]) <= TOL_LOSS_REL * abs(oo["loss"]) + 1e-7
    assert _rel(_np64(a["dH"]), oo["dH"]) <= TOL_GRAD_REL and _rel(_np64(a["dW"]), oo["dW"]) <= TOL_GRAD_REL
    _assert_status_ok(ctx)

    c2 = Context(0)
    try:
        seen = []
        c2.set_dw_slab_hook(lambda slab, r0, r1: seen.append((slab, r0, r1)))
        for limits in ((0, 0), (128, 512)):           # default slabs: one; small slabs: 6 column x several row slabs
            c2.set_slab_limits(*limits)
            seen.clear()
            b = c2.rl_policy_loss_fwd_bwd(w.H, w.W, w.tokens, w.old_logp, w.ref_logp, adv_tok, w.mask, w.eps_low,
                                          w.eps_high, w.beta, token_count=cnt)
            _assert_status_ok(c2)
            assert [s[0] for s in seen] == list(range(len(seen))) and seen[0][1] == 0 and seen[-1][2] == w.V
            assert all(seen[i][2] == seen[i + 1][1] for i in range(len(seen) - 1))
            assert len(seen) == (1 if limits == (0, 0) else -(-w.V // 512))
            assert _rel(_np64(b["dW"]), oo["dW"]) <= TOL_GRAD_REL
        c2.set_dw_slab_hook(None)
        c2.set_slab_limits(0, 0)
        seen.clear()
        c2.set_max_ctas(140)
        b = c2.rl_policy_loss_fwd_bwd(w.H, w.W, w.tokens, w.old_logp, w.ref_logp, adv_tok, w.mask, w.eps_low, w.eps_high,
                                      w.beta, token_count=cnt)
        _assert_status_ok(c2)
        assert not seen
        assert abs(b["loss"].item() - oo["loss"]) <= TOL_LOSS_REL * abs(oo["loss"]) + 1e-7
        assert _rel(_np64(b["dH"]), oo["dH"]) <= TOL_GRAD_REL and _rel(_np64(b["dW"]), oo["dW"]) <= TOL_GRAD_REL
        c2.set_max_ctas(0)
    finally:
        c2.close()


@pytest.mark.parametrize("mode,cluster,nbytes,px", [(0, 2, 0, 1), (0, 8, 0, 1), (1, 4, 8192, 2), (1, 8, 16384, 4)])
def test_cluster_exchange_probe_runs_and_returns(ctx, mode, cluster, nbytes, px):
    # the measurement kernels for cluster data movement: a short run must come back with a time, a cluster
    # count and a clean status word (their one mbarrier wait is bounded)
    ms, n_clusters = ctx.selftest_cluster_exchange(mode, cluster, 50, nbytes, px)
    _assert_status_ok(ctx)
    assert ms > 0 and 1 <= n_clusters <= 148 // cluster
