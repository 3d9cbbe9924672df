"""The allocation-free log-probability entry point (rl_token_logprobs_static), called through the
C ABI, must give what rl_token_logprobs gives.  It exists for callers that cannot allocate GPU
memory when they score tokens, for instance next to a rollout engine that has reserved nearly
all of the device: it takes no context and no workspace and keeps its scratch in a fixed 16 MiB
device array inside the library.  That array is shared by every call and keeps old contents, so
the check is made on two calls in a row with different inputs: the second must not see anything
of the first.  Collected last on purpose (file name), and it must pass alone in a fresh process
as well as after the other tests."""
import numpy as np
import pytest
import torch

from oracle import grpo_oracle as O

pytestmark = pytest.mark.gpu

TOL = 2e-3   # the log-prob / entropy tolerance of the parity tests


def _run_static(w, mask):
    from paper_2512_21450_b200.binding import rl_token_logprobs_static
    lp = torch.full((w.T,), 7.0, device="cuda")
    ent = torch.full((w.T,), 7.0, device="cuda")
    lse = torch.full((w.T,), 7.0, device="cuda")
    st = torch.full((2,), -1, dtype=torch.int32, device="cuda")
    rl_token_logprobs_static(w.H, w.W, w.tokens, mask, lp, ent, lse, st)
    torch.cuda.synchronize()
    return lp, ent, lse, st.cpu().tolist()


def test_static_entry_matches_workspace_entry_twice_in_a_row():
    from paper_2512_21450_b200 import Context, RLHeadError
    from paper_2512_21450_b200.binding import rl_token_logprobs_static
    from paper_2512_21450_b200.workloads import make_workload
    ctx = Context(0)
    try:
        # call 1: 3B-class head shapes, ragged masked rows; call 2: a smaller, different problem whose
        # scratch footprint lies inside call 1's, with a token id out of range to exercise the status word
        w1 = make_workload(1, prompts=1, L_max=96, seed=1234)
        w2 = make_workload(0, L_max=13, V=4100, seed=4321)
        for w in (w1, w2):
            ref_lp, ref_ent, ref_lse = ctx.rl_token_logprobs(w.H, w.W, w.tokens, w.mask)
            assert ctx.last_device_status()[0] == 0
            lp, ent, lse, st = _run_static(w, w.mask)
            assert st == [0, 0]
            assert (lp - ref_lp).abs().max().item() <= TOL
            assert (ent - ref_ent).abs().max().item() <= TOL
            assert (lse - ref_lse).abs().max().item() <= TOL
            m = w.mask.bool()
            assert not lp[~m].any() and not ent[~m].any()
            # and against the float64 oracle itself, so that the two CUDA entries cannot share a mistake
            f64 = lambda t: t.double().cpu().numpy()  # noqa: E731
            olp, oent, olse = O.token_logprobs(f64(w.H), f64(w.W), w.tokens.cpu().numpy(), w.mask.cpu().numpy())
            assert np.abs(f64(lp) - olp).max() <= TOL and np.abs(f64(ent) - oent).max() <= TOL
            assert np.abs(f64(lse) - olse).max() <= TOL
        # a latched error is reported through dev_status and does not leak into the next call
        bad = w2.tokens.clone()
        bad[3] = w2.V + 1
        w2.tokens, good = bad, w2.tokens
        _, _, _, st = _run_static(w2, w2.mask)
        assert st == [7, 3]
        w2.tokens = good
        lp, _, _, st = _run_static(w2, w2.mask)
        assert st == [0, 0]
        ref_lp, _, _ = ctx.rl_token_logprobs(w2.H, w2.W, w2.tokens, w2.mask)
        assert (lp - ref_lp).abs().max().item() <= TOL
        # sizes beyond the fixed scratch are refused before anything runs
        T_big, d = 4096, 2048
        Hb = torch.zeros(T_big, d, dtype=torch.bfloat16, device="cuda")
        out = torch.zeros(T_big, device="cuda")
        with pytest.raises(RLHeadError) as e:
            rl_token_logprobs_static(Hb, w1.W, torch.zeros(T_big, dtype=torch.int32, device="cuda"), None, out)
        assert e.value.status == 4
    finally:
        ctx.close()


@pytest.mark.parametrize("V,T_ok,T_refused", [(151936, 3072, 3200), (32768, 3712, 3840)])
def test_static_entry_size_limit_is_where_the_header_says(V, T_ok, T_refused):
    # d = 2048: the largest documented row count is accepted (all-zero operands: every logit is 0, so
    # logp = -log V exactly), the next multiple of 128 is refused before anything is enqueued
    import math
    from paper_2512_21450_b200 import RLHeadError
    from paper_2512_21450_b200.binding import rl_token_logprobs_static
    d = 2048
    W = torch.zeros(V, d, dtype=torch.bfloat16, device="cuda")
    for T, ok in ((T_ok, True), (T_refused, False)):
        H = torch.zeros(T, d, dtype=torch.bfloat16, device="cuda")
        tok = torch.zeros(T, dtype=torch.int32, device="cuda")
        lp = torch.full((T,), 7.0, device="cuda")
        st = torch.full((2,), -1, dtype=torch.int32, device="cuda")
        if ok:
            rl_token_logprobs_static(H, W, tok, None, lp, dev_status=st)
            torch.cuda.synchronize()
            assert st.cpu().tolist() == [0, 0]
            assert (lp + math.log(V)).abs().max().item() <= 1e-4
        else:
            with pytest.raises(RLHeadError) as e:
                rl_token_logprobs_static(H, W, tok, None, lp, dev_status=st)
            assert e.value.status == 4
            assert (lp == 7.0).all() and st.cpu().tolist() == [-1, -1]     # nothing ran


def test_static_entry_with_no_rows_clears_the_status_words():
    from paper_2512_21450_b200.binding import rl_token_logprobs_static
    W = torch.zeros(512, 64, dtype=torch.bfloat16, device="cuda")
    H = torch.zeros(0, 64, dtype=torch.bfloat16, device="cuda")
    st = torch.full((2,), -1, dtype=torch.int32, device="cuda")
    rl_token_logprobs_static(H, W, torch.zeros(0, dtype=torch.int32, device="cuda"), None,
                             torch.zeros(0, device="cuda"), dev_status=st)
    torch.cuda.synchronize()
    assert st.cpu().tolist() == [0, 0]
