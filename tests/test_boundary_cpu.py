"""CPU-only checks of the boundary and the host logic: the shared library builds, loads and
exports every symbol the header declares; the binding refuses to run without a GPU; the
synthetic workloads have the structure the configurations ask for."""
import ctypes
import os
import re

import numpy as np
import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "rlhead.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(rl_[a-z0-9_]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    from paper_2512_21450_b200 import build
    path = build.build()
    assert os.path.exists(path)
    lib = ctypes.CDLL(path)
    names = _declared_symbols()
    assert {"rl_grpo_advantages", "rl_token_logprobs", "rl_policy_loss_fwd_bwd"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} declared in rlhead.h but not exported"
    lib.rl_status_string.restype = ctypes.c_char_p
    assert lib.rl_status_string(0) == b"ok"
    assert b"token" in lib.rl_status_string(7)


def test_binding_declares_every_symbol_and_has_no_cpu_path():
    from paper_2512_21450_b200 import binding
    lib = binding.load_library()
    for n in _declared_symbols():
        assert getattr(lib, n).argtypes is not None or n == "rl_status_string"
    if not torch.cuda.is_available():
        with pytest.raises(RuntimeError):
            binding.Context(0)


def test_product_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2512_21450_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"^\s*(from|import)\s+oracle\b", src, flags=re.M), f
                assert "grpo_oracle" not in src and "oracle/" not in src and "oracle." not in src, f
    osrc = open(os.path.join(ROOT, "oracle", "grpo_oracle.py")).read()
    assert "paper_2512_21450_b200" not in osrc and "import torch" not in osrc


def test_workload_structure_cpu():
    from paper_2512_21450_b200.workloads import CONFIGS, make_workload
    w = make_workload(0, device="cpu")
    assert (w.T, w.d, w.V, w.G, w.n_seq, w.n_valid) == (256, 256, 4096, 4, 16, 256)
    assert w.H.dtype == torch.bfloat16 and w.W.dtype == torch.bfloat16 and w.tokens.dtype == torch.int32
    assert int(w.tokens.min()) >= 0 and int(w.tokens.max()) < w.V
    w2 = make_workload(0, device="cpu")
    assert torch.equal(w.H, w2.H) and torch.equal(w.tokens, w2.tokens) and torch.equal(w.old_logp, w2.old_logp)
    # perturbation scale of the behaviour / reference log-probabilities
    z = w.H.float() @ w.W.float().T
    lp = torch.log_softmax(z, 1).gather(1, w.tokens.long()[:, None])[:, 0]
    assert 0.03 < (w.old_logp - lp).std().item() < 0.07
    assert 0.07 < (w.ref_logp - lp).std().item() < 0.13
    # small-shape stand-ins of the other configurations keep their mask / reward structure
    w1 = make_workload(1, device="cpu", d=64, V=512)
    lens = w1.mask.view(w1.n_seq, w1.L_max).sum(1)
    assert w1.T == 64 * 512 and int(lens.min()) >= 64 and int(lens.max()) <= 512
    m = w1.mask.view(w1.n_seq, w1.L_max)
    assert all(bool((row[:n] == 1).all()) and not bool(row[n:].any()) for row, n in zip(m, lens))  # right-padded
    w3 = make_workload(3, device="cpu", prompts=1, d=64, V=512)
    frac = 1 - w3.n_valid / w3.T
    assert 0.28 < frac < 0.36 and bool(w3.mask.view(w3.n_seq, -1)[:, 0].all())
    w4 = make_workload(4, device="cpu", L_max=8, d=64, V=512)
    r = w4.rewards.view(-1, w4.G)
    zero_var = (r.max(1).values == r.min(1).values).float().mean().item()
    assert 0.1 < zero_var < 0.45 and w4.ref_logp is None and w4.ent_coef == 1e-3 and w4.eps_high == 0.28
    assert CONFIGS[2]["V"] == 152064 and CONFIGS[2]["d"] == 3584


def _check_schedule(n_valid, rows_cap, k_len, n_tiles, cta_group, n_workers, **kw):
    """Every (row tile, column tile, k-block) of the pass is covered exactly once."""
    from paper_2512_21450_b200.binding import debug_schedule
    u = debug_schedule(n_valid, rows_cap, k_len, n_tiles, cta_group=cta_group, n_workers=n_workers, **kw)
    rows = min(n_valid, rows_cap)
    m_units = -(-rows // (128 * cta_group))
    kb = -(-k_len // 64)
    cover = np.zeros((m_units, n_tiles, max(kb, 1)), dtype=np.int32)
    for worker, mu, c0, c1, ks, kb0, kb1, kpt in u:
        assert 0 <= worker < n_workers and 0 <= mu < m_units and 0 <= c0 < c1 <= n_tiles and kpt == kb
        assert 0 <= kb0 and kb1 <= kb               # kb1 <= kb0: an empty K slice, which the kernels fill with zeros
        cover[mu, c0:c1, kb0:kb1] += 1
        if kw.get("stream_k"):
            assert ks == (1 if kb0 > 0 else 0) and kb1 > kb0
    if kb > 0:
        assert (cover == 1).all(), (n_valid, k_len, n_tiles, kw)
    else:
        assert len(u) == m_units * len({(r[2], r[3]) for r in u}) or len(u) == 0
    return u


def test_tile_schedules_cover_every_tile_once():
    # the functions the kernels use to hand out work, run on the host: plain round-robin, column ranges,
    # row groups (equal groups, ragged last group), stream-K (last full wave + ragged wave cut by k-blocks,
    # at most two parts per tile) and K slices - on pairs and single CTAs, many sizes
    rng = np.random.default_rng(0)
    for _ in range(60):
        cg = int(rng.integers(1, 3))
        workers = int(rng.choice([3, 7, 74, 148]))
        n_valid = int(rng.integers(1, 40000))
        k_len = int(rng.choice([64, 72, 2048, 18944, 384]))
        n_tiles = int(rng.integers(1, 80))
        _check_schedule(n_valid, 32768, k_len, n_tiles, cg, workers)
        _check_schedule(n_valid, 32768, k_len, n_tiles, cg, workers, n_fastest=1)
        _check_schedule(n_valid, 32768, k_len, n_tiles, cg, workers, n_range=0)
        _check_schedule(n_valid, 32768, k_len, n_tiles, cg, workers, n_range=int(rng.integers(1, 9)),
                        m_group=int(rng.integers(1, 40)))
        _check_schedule(n_valid, 32768, k_len, n_tiles, cg, workers, n_range=-8, m_group=int(rng.integers(0, 40)))
        _check_schedule(n_valid, 32768, k_len, 8 * n_tiles, cg, workers, n_range=-112, m_group=int(rng.integers(0, 40)))
        _check_schedule(n_valid, 32768, k_len, n_tiles, cg, workers, n_fastest=1, k_split_max=int(rng.integers(2, 5)))
        u = _check_schedule(n_valid, 32768, k_len, n_tiles, cg, workers, n_fastest=1, stream_k=1)
        parts = {}
        for worker, mu, c0, c1, ks, kb0, kb1, kpt in u:
            parts.setdefault((mu, c0), []).append((kb0, kb1))
        assert max(len(v) for v in parts.values()) <= 2
    # the benchmark's dH pass with 256 x 256 tiles: 66 row tiles x 8 column tiles on 74 pairs, stream-K on
    u = _check_schedule(16896, 32768, 18944, 8, 2, 74, n_fastest=1, stream_k=1)
    work = np.zeros(74, dtype=np.int64)
    for worker, mu, c0, c1, ks, kb0, kb1, kpt in u:
        work[worker] += kb1 - kb0
    assert work.max() - work.min() <= 1 and work.sum() == 66 * 8 * 296
    # range lengths chosen on the device.  Gradient-of-the-logits pass of the benchmark (66 row tiles, 148 column
    # tiles per slab, 74 pairs): ranges of 4 tiles = 33 waves of equal units; 7B-class head (88 row tiles): the same.
    # A pass asked to choose in [8, 12] with plenty of work (594 column tiles): 9 tiles per unit (66 ranges x 66 row
    # tiles = 58.9 waves) rather than 8.
    for rows, tiles, nr_arg, expect in [(16896, 148, -8, 4), (22528, 148, -8, 4), (16896, 594, -112, 9),
                                        (16896, 2, -8, 2), (300, 148, -8, 4)]:
        u = _check_schedule(rows, 32768, 2048, tiles, 2, 74, n_range=nr_arg, m_group=36)
        assert max(r[3] - r[2] for r in u) == expect, (rows, tiles, expect, max(r[3] - r[2] for r in u))
    # a forward pass with few rows keeps the split that fills the machine (at most 16 ranges per row tile)
    u = _check_schedule(300, 32768, 2048, 594, 2, 74, n_range=-112)
    assert len({(r[2], r[3]) for r in u}) <= 16
    # the same pass on 256 x 512 tiles (the tile counter then counts 512-wide tiles: d = 2048 -> 4, 2560 -> 5,
    # 3584 -> 7): 264 tiles on 74 pairs are 3.57 waves; stream-K evens them out, K slices cover every k-block
    for d_tiles, n_valid in ((4, 16896), (5, 32768), (7, 32768), (4, 300), (7, 20001)):
        m_units = -(-n_valid // 256)
        u = _check_schedule(n_valid, 32768, 18944, d_tiles, 2, 74, n_fastest=1, stream_k=1)
        work = np.zeros(74, dtype=np.int64)
        for worker, mu, c0, c1, ks, kb0, kb1, kpt in u:
            work[worker] += kb1 - kb0
        assert work.sum() == m_units * d_tiles * 296
        if m_units * d_tiles >= 74 and (m_units * d_tiles) % 74:
            assert work.max() - work.min() <= 296      # full waves of whole tiles plus one balanced share each
            tail = work - (m_units * d_tiles // 74 - 1) * 296
            assert tail.max() - tail.min() <= 1
        _check_schedule(n_valid, 32768, 18944, d_tiles, 2, 74, n_fastest=1, k_split_max=4)
    # row groups: 66 row tiles with a budget of 36 tiles become two groups of 33; within a group all
    # column ranges are walked before the next group starts
    u = _check_schedule(16896, 32768, 2048, 74, 2, 74, m_group=36)
    assert {int(r[1]) for r in u} == set(range(66))
    for worker in (0, 37, 73):
        seen_second = False
        for r in u[u[:, 0] == worker]:
            if r[1] >= 33:
                seen_second = True
            else:
                assert not seen_second                 # a worker never returns to the first group
        assert seen_second
    # argument errors
    from paper_2512_21450_b200.binding import RLHeadError, debug_schedule
    with pytest.raises(RLHeadError):
        debug_schedule(10, 0, 64, 1)
