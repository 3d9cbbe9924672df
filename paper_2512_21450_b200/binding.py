"""ctypes binding of librlhead.so (C ABI declared in include/rlhead.h).

Argument marshalling only: every step of the path runs in the library's CUDA
kernels.  torch is used for device memory and streams.  There is no CPU
fallback: if the shared library is missing or the device is not sm_100, the
calls raise.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, byref, c_char_p, c_float, c_int, c_int32, c_int64, c_size_t, c_void_p

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "librlhead.so")

STATUS_NAMES = {
    0: "RL_OK", 1: "RL_ERR_INVALID_ARG", 2: "RL_ERR_SHAPE", 3: "RL_ERR_ALIGNMENT", 4: "RL_ERR_WORKSPACE",
    5: "RL_ERR_CUDA", 6: "RL_ERR_UNSUPPORTED_ARCH", 7: "RL_ERR_TOKEN_RANGE", 8: "RL_ERR_TIMEOUT",
}


class RLHeadError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)}")


class rl_loss_opts(ctypes.Structure):
    _fields_ = [
        ("struct_size", c_size_t),
        ("ent_coef", c_float),
        ("token_weight", c_void_p),
        ("accumulate_dW", c_int),
        ("logp_out", c_void_p),
        ("entropy_out", c_void_p),
        ("metrics_out", c_void_p),
        ("agg_mode", c_int),
        ("sequence_level", c_int),
        ("dH_dtype", c_int),
        ("seq_offsets", c_void_p),
        ("n_seq", c_int64),
        ("kl_full", c_int),
        ("H_ref", c_void_p),
        ("ldH_ref", c_int64),
        ("W_ref", c_void_p),
        ("ldW_ref", c_int64),
        ("d_ref", c_int64),
        ("kl_out", c_void_p),
        ("token_count", c_void_p),
    ]

DW_SLAB_HOOK = ctypes.CFUNCTYPE(None, c_void_p, c_int, c_int64, c_int64)


_lib = None


def load_library():
    """Load librlhead.so; raises if it has not been built (no fallback)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} not found: build it with `python -m paper_2512_21450_b200.build`")
    lib = ctypes.CDLL(LIB_PATH)
    P = c_void_p
    lib.rl_status_string.restype = c_char_p
    lib.rl_status_string.argtypes = [c_int]
    lib.rl_create.argtypes = [POINTER(c_void_p), c_int]
    lib.rl_destroy.argtypes = [P]
    lib.rl_set_stream.argtypes = [P, P]
    lib.rl_workspace_bytes.argtypes = [P, c_int64, c_int64, c_int64, POINTER(c_size_t)]
    lib.rl_workspace_bytes_host.argtypes = [P, c_int64, c_int64, c_int64, POINTER(c_size_t)]
    lib.rl_workspace_bytes_kl.argtypes = [P, c_int64, c_int64, c_int64, c_int64, POINTER(c_size_t)]
    lib.rl_set_workspace.argtypes = [P, P, c_size_t]
    lib.rl_set_slab_limits.argtypes = [P, c_int, c_int]
    lib.rl_set_dh_k_slices.argtypes = [P, c_int]
    lib.rl_set_dh_k_slices.restype = c_int
    lib.rl_set_row_group_bytes.argtypes = [P, c_int64]
    lib.rl_set_row_group_bytes.restype = c_int
    lib.rl_set_wide_tiles.argtypes = [P, c_int]
    lib.rl_set_wide_tiles.restype = c_int
    lib.rl_set_dh_stream_k.argtypes = [P, c_int]
    lib.rl_set_dh_stream_k.restype = c_int
    lib.rl_set_max_ctas.argtypes = [P, c_int]
    lib.rl_set_max_ctas.restype = c_int
    lib.rl_set_dw_slab_hook.argtypes = [P, DW_SLAB_HOOK, P]
    lib.rl_set_dw_slab_hook.restype = c_int
    lib.rl_set_cta_group.argtypes = [P, c_int]
    lib.rl_set_cta_group.restype = c_int
    lib.rl_last_device_status.argtypes = [P, POINTER(c_int32)]
    lib.rl_grpo_advantages.argtypes = [P, P, c_int64, c_int, P]
    lib.rl_grpo_advantages_ex.argtypes = [P, P, c_int64, c_int, c_int, c_float, P, c_int64, P, P]
    lib.rl_selftest_wait_timeout.argtypes = [P, c_int]
    lib.rl_selftest_wait_timeout.restype = c_int
    lib.rl_advantages.argtypes = [P, c_int, P, P, c_int64, c_int, c_float, P]
    lib.rl_advantages.restype = c_int
    lib.rl_token_logprobs.argtypes = [P, P, c_int64, P, c_int64, P, P, c_int64, c_int64, c_int64, P, P, P]
    loss_args = [P, P, c_int64, P, c_int64, P, P, P, P, P, c_int64, c_int64, c_int64,
                 c_float, c_float, c_float, P, P, P]
    lib.rl_policy_loss_fwd_bwd.argtypes = loss_args
    lib.rl_policy_loss_fwd_bwd_ex.argtypes = loss_args + [POINTER(rl_loss_opts)]
    lib.rl_policy_loss_fwd_bwd_host.argtypes = [P, P, c_int64, P, c_int64, P, P, P, P, P, c_int64, c_int, P, P,
                                                c_int64, c_int64, c_int64,
                                                c_float, c_float, c_float, c_float, P, P, P, P]
    lib.rl_workspace_bytes_host_pipelined.argtypes = [P, c_int64, c_int64, c_int64, POINTER(c_size_t)]
    lib.rl_workspace_bytes_host_pipelined.restype = c_int
    lib.rl_policy_loss_fwd_bwd_host_submit.argtypes = [P, c_int, P, c_int64, P, c_int64, P, P, P, P, P, c_int64, c_int, P, P,
                                                       c_int64, c_int64, c_int64, c_float, c_float, c_float, c_float, P, P]
    lib.rl_policy_loss_fwd_bwd_host_submit.restype = c_int
    lib.rl_policy_loss_fwd_bwd_host_wait.argtypes = [P, c_int, P, P]
    lib.rl_policy_loss_fwd_bwd_host_wait.restype = c_int
    lib.rl_launch_count.argtypes = [P, POINTER(c_int64)]
    lib.rl_set_profiling.argtypes = [P, c_int]
    lib.rl_profile_read.argtypes = [P, POINTER(ctypes.c_double), POINTER(c_int64)]
    lib.rl_selftest_gemm.argtypes = [P, P, P, P, c_int64, c_int64, c_int64, c_int, c_int, c_int]
    lib.rl_token_logprobs_static.argtypes = [P, P, c_int64, P, c_int64, P, P, c_int64, c_int64, c_int64, P, P, P, P]
    lib.rl_token_logprobs_static.restype = c_int
    lib.rl_debug_schedule.argtypes = [c_int64, c_int64, c_int64, c_int64, c_int, c_int, c_int, c_int, c_int, c_int, c_int,
                                      P, c_int64, POINTER(c_int64)]
    lib.rl_debug_schedule.restype = c_int
    lib.rl_selftest_cluster_exchange.argtypes = [P, c_int, c_int, c_int, c_int, c_int, POINTER(c_float), POINTER(c_int)]
    lib.rl_selftest_cluster_exchange.restype = c_int
    lib.rl_mask_scan.argtypes = [P, P, c_int64, P, P]
    lib.rl_mask_scan.restype = c_int
    lib.rl_kl_shaped_returns.argtypes = [P, P, P, P, P, P, P, c_int64, c_int64, c_float, c_float, c_int, P, P]
    lib.rl_kl_shaped_returns.restype = c_int
    lib.rl_token_loss.argtypes = [P, P, P, P, P, P, P, c_int64, c_float, c_float, c_float, c_float, P, P, P, P, P, P]
    lib.rl_token_loss.restype = c_int
    lib.rl_token_logprobs_multi.argtypes = [P, c_int, POINTER(c_void_p), POINTER(c_int64), POINTER(c_void_p),
                                            POINTER(c_int64), POINTER(c_int64), P, P, c_int64, c_int64,
                                            POINTER(c_void_p), POINTER(c_void_p)]
    lib.rl_token_logprobs_multi.restype = c_int
    lib.rl_shard_logit_stats.argtypes = [P, P, c_int64, P, c_int64, P, P, c_int64, c_int64, c_int64, c_int64, c_int64, P]
    lib.rl_shard_logit_stats.restype = c_int
    lib.rl_merge_logit_stats.argtypes = [P, P, c_int, P, c_int64, P, P, P]
    lib.rl_merge_logit_stats.restype = c_int
    lib.rl_policy_loss_shard_bwd.argtypes = [P, P, c_int64, P, c_int64, P, P, P, P, P, c_int64, c_int64, c_int64,
                                             c_int64, c_int64, P, P, P, c_float, c_float, c_float, P, P, P,
                                             POINTER(rl_loss_opts)]
    lib.rl_policy_loss_shard_bwd.restype = c_int
    for name in ("rl_create", "rl_destroy", "rl_set_stream", "rl_workspace_bytes", "rl_workspace_bytes_host",
                 "rl_workspace_bytes_kl",
                 "rl_set_workspace", "rl_set_slab_limits", "rl_last_device_status", "rl_grpo_advantages", "rl_grpo_advantages_ex",
                 "rl_token_logprobs", "rl_policy_loss_fwd_bwd", "rl_policy_loss_fwd_bwd_ex",
                 "rl_policy_loss_fwd_bwd_host", "rl_selftest_gemm", "rl_launch_count", "rl_set_profiling",
                 "rl_profile_read"):
        getattr(lib, name).restype = c_int
    _lib = lib
    return lib


def _ptr(t):
    return c_void_p(t.data_ptr()) if t is not None else c_void_p(0)


def _check(status, where):
    if status != 0:
        raise RLHeadError(status, where)


class Context:
    """One library context on one device; owns a torch-allocated workspace."""

    def __init__(self, device=0):
        if not torch.cuda.is_available():
            raise RuntimeError("rlhead needs a CUDA device (sm_100a); there is no CPU path")
        self.lib = load_library()
        self.device = torch.device("cuda", device)
        self.handle = c_void_p()
        _check(self.lib.rl_create(byref(self.handle), device), "rl_create")
        self._ws = None
        self._ws_key = None
        self._slot_busy = [False, False]

    def close(self):
        if self.handle:
            self.lib.rl_destroy(self.handle)
            self.handle = c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _bind_stream(self):
        _check(self.lib.rl_set_stream(self.handle, c_void_p(torch.cuda.current_stream(self.device).cuda_stream)),
               "rl_set_stream")

    def workspace_bytes(self, T, d, V, host=False, d_ref=0):
        n = c_size_t()
        if d_ref:
            _check(self.lib.rl_workspace_bytes_kl(self.handle, T, d, V, d_ref, byref(n)), "rl_workspace_bytes_kl")
            return n.value
        fn = self.lib.rl_workspace_bytes_host if host else self.lib.rl_workspace_bytes
        _check(fn(self.handle, T, d, V, byref(n)), "rl_workspace_bytes")
        return n.value

    def ensure_workspace(self, T, d, V, host=False, d_ref=0):
        need = self.workspace_bytes(T, d, V, host, d_ref)
        if self._ws is None or self._ws.numel() < need:
            self._ws = None
            self._ws = torch.empty(need, dtype=torch.uint8, device=self.device)
        _check(self.lib.rl_set_workspace(self.handle, _ptr(self._ws), self._ws.numel()), "rl_set_workspace")

    def set_slab_limits(self, max_rows=0, max_cols=0):
        _check(self.lib.rl_set_slab_limits(self.handle, max_rows, max_cols), "rl_set_slab_limits")

    def set_dh_k_slices(self, max_slices):
        _check(self.lib.rl_set_dh_k_slices(self.handle, max_slices), "rl_set_dh_k_slices")

    def set_row_group_bytes(self, nbytes):
        _check(self.lib.rl_set_row_group_bytes(self.handle, int(nbytes)), "rl_set_row_group_bytes")

    def set_wide_tiles(self, on):
        _check(self.lib.rl_set_wide_tiles(self.handle, int(on)), "rl_set_wide_tiles")

    def set_dh_stream_k(self, on):
        _check(self.lib.rl_set_dh_stream_k(self.handle, int(on)), "rl_set_dh_stream_k")

    def set_max_ctas(self, max_ctas):
        _check(self.lib.rl_set_max_ctas(self.handle, int(max_ctas)), "rl_set_max_ctas")

    def set_dw_slab_hook(self, fn):
        """fn(slab, row_begin, row_end) is called on the host right after the launch that completes those
        rows of dW has been enqueued; None removes the hook."""
        if fn is None:
            self._hook = DW_SLAB_HOOK(0)
        else:
            self._hook = DW_SLAB_HOOK(lambda user, slab, r0, r1: fn(slab, r0, r1))
        _check(self.lib.rl_set_dw_slab_hook(self.handle, self._hook, None), "rl_set_dw_slab_hook")

    def set_cta_group(self, cta_group):
        _check(self.lib.rl_set_cta_group(self.handle, cta_group), "rl_set_cta_group")

    def last_device_status(self):
        detail = c_int32()
        return self.lib.rl_last_device_status(self.handle, byref(detail)), detail.value

    # ------------------------------------------------------------------ calls
    def rl_grpo_advantages(self, rewards, group_size, ddof=1, eps_std=1e-6, seq_offsets=None, T=None):
        self._bind_stream()
        assert rewards.dtype == torch.float32 and rewards.is_cuda and rewards.is_contiguous()
        adv_seq = torch.empty_like(rewards)
        if seq_offsets is None:
            if ddof == 1 and eps_std == 1e-6:
                _check(self.lib.rl_grpo_advantages(self.handle, _ptr(rewards), rewards.numel(), group_size,
                                                   _ptr(adv_seq)), "rl_grpo_advantages")
            else:
                _check(self.lib.rl_grpo_advantages_ex(self.handle, _ptr(rewards), rewards.numel(), group_size, ddof,
                                                      eps_std, None, 0, _ptr(adv_seq), None),
                       "rl_grpo_advantages_ex")
            return adv_seq
        assert seq_offsets.dtype == torch.int32 and seq_offsets.is_cuda
        adv_tok = torch.empty(T, dtype=torch.float32, device=rewards.device)
        _check(self.lib.rl_grpo_advantages_ex(self.handle, _ptr(rewards), rewards.numel(), group_size, ddof, eps_std,
                                              _ptr(seq_offsets), T, _ptr(adv_seq), _ptr(adv_tok)),
               "rl_grpo_advantages_ex")
        return adv_seq, adv_tok

    ESTIMATORS = {"grpo": 0, "rloo": 1, "opo": 2, "reinforce_pp": 3}

    def rl_advantages(self, estimator, rewards, group_size, lengths=None, eps_std=1e-6):
        self._bind_stream()
        assert rewards.dtype == torch.float32 and rewards.is_cuda and rewards.is_contiguous()
        assert lengths is None or lengths.dtype == torch.int32
        adv_seq = torch.empty_like(rewards)
        _check(self.lib.rl_advantages(self.handle, self.ESTIMATORS[estimator], _ptr(rewards), _ptr(lengths),
                                      rewards.numel(), group_size, eps_std, _ptr(adv_seq)), "rl_advantages")
        return adv_seq

    def rl_token_logprobs(self, H, W, tokens, mask=None):
        self._bind_stream()
        T, d = H.shape
        V = W.shape[0]
        assert H.dtype == torch.bfloat16 and W.dtype == torch.bfloat16 and tokens.dtype == torch.int32
        assert H.stride(1) == 1 and W.stride(1) == 1
        self.ensure_workspace(T, d, V)
        logp = torch.empty(T, dtype=torch.float32, device=H.device)
        ent = torch.empty_like(logp)
        lse = torch.empty_like(logp)
        _check(self.lib.rl_token_logprobs(self.handle, _ptr(H), H.stride(0) if T else d, _ptr(W), W.stride(0),
                                          _ptr(tokens), _ptr(mask), T, d, V, _ptr(logp), _ptr(ent), _ptr(lse)),
               "rl_token_logprobs")
        return logp, ent, lse

    def rl_policy_loss_fwd_bwd(self, H, W, tokens, old_logp, ref_logp, adv, mask, eps_low, eps_high, beta,
                               ent_coef=0.0, token_weight=None, accumulate_dW=False, dW=None, want_aux=True,
                               dH=None, loss=None, agg_mode=0, sequence_level=False, seq_offsets=None,
                               dH_fp32=False, H_ref=None, W_ref=None, token_count=None):
        """H_ref [T, d_ref] and W_ref [V, d_ref] (bf16) switch the regulariser to the full-distribution
        KL(pi_theta || pi_ref) against softmax(W_ref h_ref); ref_logp is then unused."""
        self._bind_stream()
        T, d = H.shape
        V = W.shape[0]
        assert H.dtype == torch.bfloat16 and W.dtype == torch.bfloat16 and tokens.dtype == torch.int32
        assert H.stride(1) == 1 and W.stride(1) == 1
        kl_full = W_ref is not None
        if kl_full:
            assert H_ref is not None and H_ref.dtype == torch.bfloat16 and W_ref.dtype == torch.bfloat16
            assert H_ref.shape[0] == T and W_ref.shape[0] == V and H_ref.shape[1] == W_ref.shape[1]
            assert H_ref.stride(1) == 1 and W_ref.stride(1) == 1
        self.ensure_workspace(T, d, V, d_ref=W_ref.shape[1] if kl_full else 0)
        dev = W.device
        loss = torch.empty(1, dtype=torch.float32, device=dev) if loss is None else loss
        if dH is None:
            dH = torch.empty(T, d, dtype=torch.float32 if dH_fp32 else torch.bfloat16, device=dev)
        if dW is None:
            dW = torch.empty(V, d, dtype=torch.float32, device=dev)
        out = dict(loss=loss, dH=dH, dW=dW)
        plain = (ent_coef == 0.0 and token_weight is None and not accumulate_dW and not want_aux and agg_mode == 0
                 and not sequence_level and not dH_fp32 and not kl_full and token_count is None)
        args = [self.handle, _ptr(H), H.stride(0) if T else d, _ptr(W), W.stride(0), _ptr(tokens), _ptr(old_logp),
                _ptr(ref_logp), _ptr(adv), _ptr(mask), T, d, V, eps_low, eps_high, beta, _ptr(loss), _ptr(dH),
                _ptr(dW)]
        if plain:
            _check(self.lib.rl_policy_loss_fwd_bwd(*args), "rl_policy_loss_fwd_bwd")
            return out
        opts = rl_loss_opts()
        opts.struct_size = ctypes.sizeof(rl_loss_opts)
        opts.ent_coef = ent_coef
        opts.token_weight = token_weight.data_ptr() if token_weight is not None else None
        opts.accumulate_dW = int(accumulate_dW)
        opts.agg_mode = agg_mode
        opts.sequence_level = int(sequence_level)
        opts.dH_dtype = int(dH_fp32)
        if token_count is not None:
            assert token_count.dtype == torch.int64 and token_count.is_cuda and token_count.numel() == 1
            opts.token_count = token_count.data_ptr()
        if kl_full:
            opts.kl_full = 1
            opts.H_ref = H_ref.data_ptr() if T else None
            opts.ldH_ref = H_ref.stride(0) if T else W_ref.shape[1]
            opts.W_ref = W_ref.data_ptr()
            opts.ldW_ref = W_ref.stride(0)
            opts.d_ref = W_ref.shape[1]
        if seq_offsets is not None:
            assert seq_offsets.dtype == torch.int32 and seq_offsets.is_cuda
            opts.seq_offsets = seq_offsets.data_ptr()
            opts.n_seq = seq_offsets.numel() - 1
        if want_aux:
            out["logp"] = torch.empty(T, dtype=torch.float32, device=dev)
            out["entropy"] = torch.empty(T, dtype=torch.float32, device=dev)
            out["metrics"] = torch.empty(8, dtype=torch.float32, device=dev)
            opts.logp_out = out["logp"].data_ptr()
            opts.entropy_out = out["entropy"].data_ptr()
            opts.metrics_out = out["metrics"].data_ptr()
            if kl_full:
                out["kl"] = torch.empty(T, dtype=torch.float32, device=dev)
                opts.kl_out = out["kl"].data_ptr()
        _check(self.lib.rl_policy_loss_fwd_bwd_ex(*args, byref(opts)), "rl_policy_loss_fwd_bwd_ex")
        return out

    KL_ESTIMATES = {"k1": 0, "k3": 1, "given": 2}

    def rl_kl_shaped_returns(self, seq_value, logp, ref_logp, mask, seq_offsets, T, beta, gamma=1.0, kind="k3",
                             kl_tok=None, want_shaped=True, returns=None):
        """Token-level KL reward shaping: returns (shaped_reward [T] or None, returns [T])."""
        self._bind_stream()
        assert seq_value.dtype == torch.float32 and seq_offsets.dtype == torch.int32
        for x in (logp, ref_logp, kl_tok):
            assert x is None or (x.dtype == torch.float32 and x.is_contiguous() and x.numel() == T)
        dev = seq_value.device
        if returns is None:
            returns = torch.empty(T, dtype=torch.float32, device=dev)
        shaped = torch.empty(T, dtype=torch.float32, device=dev) if want_shaped else None
        _check(self.lib.rl_kl_shaped_returns(self.handle, _ptr(seq_value), _ptr(logp), _ptr(ref_logp), _ptr(kl_tok),
                                             _ptr(mask), _ptr(seq_offsets), seq_offsets.numel() - 1, T, beta, gamma,
                                             self.KL_ESTIMATES[kind], _ptr(shaped), _ptr(returns)),
               "rl_kl_shaped_returns")
        return shaped, returns

    def rl_token_loss(self, logp, entropy, old_logp, ref_logp, adv, mask, eps_low, eps_high, beta, ent_coef=0.0,
                      token_weight=None, token_count=None, want_grads=True, want_metrics=True, out=None):
        """The per-token loss arithmetic on its own, from log-probabilities (and entropies) the caller holds:
        returns dict(loss [1], dlogp [T], dentropy [T], metrics [8]); `out` may carry preallocated tensors."""
        self._bind_stream()
        T = logp.numel()
        for x in (logp, entropy, old_logp, ref_logp, adv, token_weight):
            assert x is None or (x.dtype == torch.float32 and x.is_contiguous() and x.numel() == T)
        assert mask is None or (mask.dtype == torch.uint8 and mask.numel() == T)
        assert token_count is None or token_count.dtype == torch.int64
        dev = logp.device
        out = dict(out or {})
        out.setdefault("loss", torch.empty(1, dtype=torch.float32, device=dev))
        if want_grads:
            out.setdefault("dlogp", torch.empty(T, dtype=torch.float32, device=dev))
            out.setdefault("dentropy", torch.empty(T, dtype=torch.float32, device=dev))
        if want_metrics:
            out.setdefault("metrics", torch.empty(8, dtype=torch.float32, device=dev))
        _check(self.lib.rl_token_loss(self.handle, _ptr(logp), _ptr(entropy), _ptr(old_logp), _ptr(ref_logp), _ptr(adv),
                                      _ptr(mask), T, eps_low, eps_high, beta, ent_coef, _ptr(token_weight),
                                      _ptr(token_count), _ptr(out["loss"]), _ptr(out.get("dlogp")),
                                      _ptr(out.get("dentropy")), _ptr(out.get("metrics"))), "rl_token_loss")
        return out

    def rl_mask_scan(self, mask, T=None, row_map=None, n_valid=None):
        """Row map of the valid rows: returns (row_map [T] int32, n_valid [1] int32), both on the device."""
        self._bind_stream()
        T = mask.numel() if T is None else T
        need = (T // 4096 + 3) * 4
        if self._ws is None or self._ws.numel() < need:
            self._ws = torch.empty(max(need, 1 << 20), dtype=torch.uint8, device=self.device)
        _check(self.lib.rl_set_workspace(self.handle, _ptr(self._ws), self._ws.numel()), "rl_set_workspace")
        if row_map is None:
            row_map = torch.empty(max(T, 1), dtype=torch.int32, device=self.device)
        if n_valid is None:
            n_valid = torch.empty(1, dtype=torch.int32, device=self.device)
        _check(self.lib.rl_mask_scan(self.handle, _ptr(mask), T, _ptr(row_map), _ptr(n_valid)), "rl_mask_scan")
        return row_map, n_valid

    def rl_token_logprobs_multi(self, Hs, Ws, tokens, mask=None, want_entropy=True):
        """Log-probabilities of the same tokens under several models (e.g. old policy and reference):
        lists of H [T, d_i] and W [V, d_i]; returns (list of logp, list of entropy or None)."""
        self._bind_stream()
        n = len(Hs)
        assert n == len(Ws) and n >= 1
        T, V = Hs[0].shape[0], Ws[0].shape[0]
        for H, W in zip(Hs, Ws):
            assert H.dtype == torch.bfloat16 and W.dtype == torch.bfloat16 and H.shape[0] == T and W.shape[0] == V
            assert H.stride(1) == 1 and W.stride(1) == 1 and H.shape[1] == W.shape[1]
        assert tokens.dtype == torch.int32
        self.ensure_workspace(T, max(W.shape[1] for W in Ws), V)
        dev = Ws[0].device
        logp = [torch.empty(T, dtype=torch.float32, device=dev) for _ in range(n)]
        ent = [torch.empty(T, dtype=torch.float32, device=dev) for _ in range(n)] if want_entropy else None
        arr_p = lambda ts: (c_void_p * n)(*[t.data_ptr() if t.numel() else None for t in ts])  # noqa: E731
        arr_i = lambda xs: (c_int64 * n)(*xs)  # noqa: E731
        _check(self.lib.rl_token_logprobs_multi(
            self.handle, n, arr_p(Hs), arr_i([H.stride(0) if T else H.shape[1] for H in Hs]), arr_p(Ws),
            arr_i([W.stride(0) for W in Ws]), arr_i([W.shape[1] for W in Ws]), _ptr(tokens), _ptr(mask), T, V,
            arr_p(logp), arr_p(ent) if ent is not None else None), "rl_token_logprobs_multi")
        return logp, ent

    # ------------------------------------------------------------------ vocabulary-parallel head
    def rl_shard_logit_stats(self, H, W_shard, tokens, mask, vocab_offset, V_total, stats=None):
        """Per-row (M, S, A, z_y) over this rank's rows of the head; stats [T, 4] fp32."""
        self._bind_stream()
        T, d = H.shape
        Vs = W_shard.shape[0]
        assert H.dtype == torch.bfloat16 and W_shard.dtype == torch.bfloat16 and tokens.dtype == torch.int32
        assert H.stride(1) == 1 and W_shard.stride(1) == 1
        self.ensure_workspace(T, d, Vs)
        if stats is None:
            stats = torch.empty(T, 4, dtype=torch.float32, device=H.device)
        assert stats.dtype == torch.float32 and stats.is_contiguous() and stats.numel() == 4 * T
        _check(self.lib.rl_shard_logit_stats(self.handle, _ptr(H), H.stride(0) if T else d, _ptr(W_shard),
                                             W_shard.stride(0), _ptr(tokens), _ptr(mask), T, d, Vs, vocab_offset,
                                             V_total, _ptr(stats)), "rl_shard_logit_stats")
        return stats

    def rl_merge_logit_stats(self, stats, mask=None):
        """stats [n_shards, T, 4] (all slices of the vocabulary) -> (logp, entropy, lse), each [T]."""
        self._bind_stream()
        assert stats.dtype == torch.float32 and stats.is_contiguous() and stats.dim() == 3 and stats.shape[2] == 4
        n_shards, T = stats.shape[0], stats.shape[1]
        logp = torch.empty(T, dtype=torch.float32, device=stats.device)
        ent = torch.empty_like(logp)
        lse = torch.empty_like(logp)
        _check(self.lib.rl_merge_logit_stats(self.handle, _ptr(stats), n_shards, _ptr(mask), T, _ptr(logp), _ptr(ent),
                                             _ptr(lse)), "rl_merge_logit_stats")
        return logp, ent, lse

    def rl_policy_loss_shard_bwd(self, H, W_shard, tokens, old_logp, ref_logp, adv, mask, vocab_offset, V_total,
                                 logp, entropy, lse, eps_low, eps_high, beta, ent_coef=0.0, token_weight=None,
                                 dH_fp32=True, accumulate_dW=False, dW=None, dH=None, agg_mode=0,
                                 sequence_level=False, seq_offsets=None):
        """This rank's share of the backward pass given the merged per-token statistics: returns
        dict(loss (whole vocabulary, same on every rank), dH (partial: sum over ranks), dW (its rows))."""
        self._bind_stream()
        T, d = H.shape
        Vs = W_shard.shape[0]
        assert H.dtype == torch.bfloat16 and W_shard.dtype == torch.bfloat16 and tokens.dtype == torch.int32
        assert H.stride(1) == 1 and W_shard.stride(1) == 1
        for x in (logp, entropy, lse):
            assert x.dtype == torch.float32 and x.is_contiguous() and x.numel() == T
        self.ensure_workspace(T, d, Vs)
        dev = W_shard.device
        loss = torch.empty(1, dtype=torch.float32, device=dev)
        if dH is None:
            dH = torch.empty(T, d, dtype=torch.float32 if dH_fp32 else torch.bfloat16, device=dev)
        if dW is None:
            dW = torch.empty(Vs, d, dtype=torch.float32, device=dev)
        opts = rl_loss_opts()
        opts.struct_size = ctypes.sizeof(rl_loss_opts)
        opts.ent_coef = ent_coef
        opts.token_weight = token_weight.data_ptr() if token_weight is not None else None
        opts.accumulate_dW = int(accumulate_dW)
        opts.agg_mode = agg_mode
        opts.sequence_level = int(sequence_level)
        opts.dH_dtype = int(dH.dtype == torch.float32)
        if seq_offsets is not None:
            opts.seq_offsets = seq_offsets.data_ptr()
            opts.n_seq = seq_offsets.numel() - 1
        _check(self.lib.rl_policy_loss_shard_bwd(
            self.handle, _ptr(H), H.stride(0) if T else d, _ptr(W_shard), W_shard.stride(0), _ptr(tokens),
            _ptr(old_logp), _ptr(ref_logp), _ptr(adv), _ptr(mask), T, d, Vs, vocab_offset, V_total, _ptr(logp),
            _ptr(entropy), _ptr(lse), eps_low, eps_high, beta, _ptr(loss), _ptr(dH), _ptr(dW), byref(opts)),
            "rl_policy_loss_shard_bwd")
        return dict(loss=loss, dH=dH, dW=dW)

    def selftest_wait_timeout(self, limit_ms=20):
        self._bind_stream()
        _check(self.lib.rl_selftest_wait_timeout(self.handle, limit_ms), "rl_selftest_wait_timeout")

    def selftest_cluster_exchange(self, mode, cluster_size, iters, nbytes=0, partner_xor=1):
        """Device time (ms) of `iters` rounds of the cluster exchange and the number of clusters that ran."""
        self._bind_stream()
        ms, ncl = c_float(), c_int()
        _check(self.lib.rl_selftest_cluster_exchange(self.handle, mode, cluster_size, iters, nbytes, partner_xor,
                                                     byref(ms), byref(ncl)), "rl_selftest_cluster_exchange")
        return ms.value, ncl.value

    def launch_count(self):
        n = c_int64()
        _check(self.lib.rl_launch_count(self.handle, byref(n)), "rl_launch_count")
        return n.value

    def set_profiling(self, on):
        _check(self.lib.rl_set_profiling(self.handle, int(on)), "rl_set_profiling")

    def profile_read(self):
        ms = (ctypes.c_double * 9)()
        n = (c_int64 * 9)()
        _check(self.lib.rl_profile_read(self.handle, ms, n), "rl_profile_read")
        return list(ms), list(n)

    def rl_policy_loss_fwd_bwd_host(self, H_host, W, tokens_host, old_host, ref_host, adv_host, mask_host,
                                    eps_low, eps_high, beta, ent_coef, dH, dW, rewards_host=None, group_size=0,
                                    seq_offsets_host=None):
        """Per-step inputs in (pinned) host memory; W, dH, dW on the device.  Returns (loss, metrics) floats."""
        self._bind_stream()
        T, d = H_host.shape
        V = W.shape[0]
        self.ensure_workspace(T, d, V, host=True)
        loss = (c_float * 1)()
        metrics = (c_float * 8)()
        _check(self.lib.rl_policy_loss_fwd_bwd_host(
            self.handle, _ptr(H_host), d, _ptr(W), W.stride(0), _ptr(tokens_host), _ptr(old_host), _ptr(ref_host),
            _ptr(adv_host), _ptr(rewards_host), rewards_host.numel() if rewards_host is not None else 0, group_size,
            _ptr(seq_offsets_host), _ptr(mask_host), T, d, V, eps_low, eps_high, beta, ent_coef,
            ctypes.cast(loss, c_void_p), ctypes.cast(metrics, c_void_p), _ptr(dH), _ptr(dW)),
            "rl_policy_loss_fwd_bwd_host")
        return loss[0], list(metrics)

    def rl_policy_loss_fwd_bwd_host_submit(self, slot, H_host, W, tokens_host, old_host, ref_host, adv_host, mask_host,
                                           eps_low, eps_high, beta, ent_coef, dH, dW, rewards_host=None, group_size=0,
                                           seq_offsets_host=None):
        """First half of a pipelined host-buffer step: enqueue copies and kernels, do not wait."""
        self._bind_stream()
        T, d = H_host.shape
        V = W.shape[0]
        need = c_size_t()
        _check(self.lib.rl_workspace_bytes_host_pipelined(self.handle, T, d, V, byref(need)),
               "rl_workspace_bytes_host_pipelined")
        if self._ws is None or self._ws.numel() < need.value:
            assert not any(self._slot_busy), "workspace must not be replaced while a step is in flight"
            self._ws = None
            self._ws = torch.empty(need.value, dtype=torch.uint8, device=self.device)
        _check(self.lib.rl_set_workspace(self.handle, _ptr(self._ws), self._ws.numel()), "rl_set_workspace")
        _check(self.lib.rl_policy_loss_fwd_bwd_host_submit(
            self.handle, slot, _ptr(H_host), d, _ptr(W), W.stride(0), _ptr(tokens_host), _ptr(old_host), _ptr(ref_host),
            _ptr(adv_host), _ptr(rewards_host), rewards_host.numel() if rewards_host is not None else 0, group_size,
            _ptr(seq_offsets_host), _ptr(mask_host), T, d, V, eps_low, eps_high, beta, ent_coef, _ptr(dH), _ptr(dW)),
            "rl_policy_loss_fwd_bwd_host_submit")
        self._slot_busy[slot] = True

    def rl_policy_loss_fwd_bwd_host_wait(self, slot):
        """Second half: block until the step submitted to `slot` is done; returns (loss, metrics)."""
        loss = (c_float * 1)()
        metrics = (c_float * 8)()
        _check(self.lib.rl_policy_loss_fwd_bwd_host_wait(self.handle, slot, ctypes.cast(loss, c_void_p),
                                                         ctypes.cast(metrics, c_void_p)),
               "rl_policy_loss_fwd_bwd_host_wait")
        self._slot_busy[slot] = False
        return loss[0], list(metrics)

    def rl_selftest_gemm(self, A, B, M, N, K, a_mn_major, b_mn_major, C=None, accumulate=False):
        self._bind_stream()
        if C is None:
            C = torch.empty(M, N, dtype=torch.float32, device=A.device)
        _check(self.lib.rl_selftest_gemm(self.handle, _ptr(A), _ptr(B), _ptr(C), M, N, K, int(a_mn_major),
                                         int(b_mn_major), int(accumulate)), "rl_selftest_gemm")
        return C


def debug_schedule(n_valid, rows_cap, k_len, n_tiles, n_range=1, n_fastest=0, m_group=0, stream_k=0, k_split_max=1,
                   cta_group=2, n_workers=74):
    """Work units of one tensor-core pass as the kernels would walk them (host only, needs no GPU):
    int32 array [n_units, 8] = worker, row tile, first / end column tile, output slice, first / end
    k-block, k-blocks per tile."""
    import numpy as np
    lib = load_library()
    n = c_int64()
    args = (n_valid, rows_cap, k_len, n_tiles, n_range, n_fastest, m_group, stream_k, k_split_max, cta_group, n_workers)
    _check(lib.rl_debug_schedule(*args, None, 0, byref(n)), "rl_debug_schedule")
    out = np.zeros((n.value, 8), dtype=np.int32)
    _check(lib.rl_debug_schedule(*args, out.ctypes.data_as(c_void_p), n.value, byref(n)), "rl_debug_schedule")
    return out


_default_ctx = {}


def default_context(device=0):
    if device not in _default_ctx:
        _default_ctx[device] = Context(device)
    return _default_ctx[device]


def rl_grpo_advantages(rewards, group_size, **kw):
    return default_context(rewards.device.index or 0).rl_grpo_advantages(rewards, group_size, **kw)


def rl_token_logprobs(H, W, tokens, mask=None):
    return default_context(H.device.index or 0).rl_token_logprobs(H, W, tokens, mask)


def rl_policy_loss_fwd_bwd(H, W, tokens, old_logp, ref_logp, adv, mask, eps_low, eps_high, beta, **kw):
    return default_context(W.device.index or 0).rl_policy_loss_fwd_bwd(
        H, W, tokens, old_logp, ref_logp, adv, mask, eps_low, eps_high, beta, **kw)


def rl_token_logprobs_static(H, W, tokens, mask, logp, entropy=None, lse=None, dev_status=None):
    """Allocation-free log-probabilities: no context, no workspace, outputs preallocated by the caller.

    For callers that cannot allocate device memory at call time (see include/rlhead.h).  Runs on
    the current device and the current torch stream; scratch is the library's fixed 16 MiB device
    array, so overlapping calls race and sizes beyond the limit raise RL_ERR_WORKSPACE.
    """
    lib = load_library()
    T, d = H.shape
    V = W.shape[0]
    assert H.dtype == torch.bfloat16 and W.dtype == torch.bfloat16 and tokens.dtype == torch.int32
    assert logp.dtype == torch.float32 and logp.numel() == T
    # the library works on the CURRENT device: make it the one the operands live on
    with torch.cuda.device(H.device):
        stream = c_void_p(torch.cuda.current_stream(H.device).cuda_stream)
        _check(lib.rl_token_logprobs_static(stream, _ptr(H), H.stride(0) if T else d, _ptr(W), W.stride(0),
                                            _ptr(tokens), _ptr(mask), T, d, V, _ptr(logp), _ptr(entropy), _ptr(lse),
                                            _ptr(dev_status)),
               "rl_token_logprobs_static")
    return logp
