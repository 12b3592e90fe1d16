"""ctypes binding of libecho_b200.so: argument marshalling only.

Every step of the rollout path runs in the library's CUDA kernels; torch is used here
for device memory and streams.  There is no CPU fallback: if the library is missing the
import of this module raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("ECHO_B200_LIB") or os.path.join(_HERE, "libecho_b200.so")   # override: another build of the library

ECHO_OK = 0
ERRORS = {
    -1: "ECHO_ERR_INVALID", -2: "ECHO_ERR_ARENA", -3: "ECHO_ERR_NO_POLICY", -4: "ECHO_ERR_VERSION",
    -5: "ECHO_ERR_BUSY", -6: "ECHO_ERR_CUDA", -7: "ECHO_ERR_DEVICE_CHECK", -8: "ECHO_ERR_TIMEOUT",
    -9: "ECHO_ERR_UNSUPPORTED",
}


class EchoError(RuntimeError):
    def __init__(self, code: int, detail: str = ""):
        self.code = code
        super().__init__(f"{ERRORS.get(code, code)} {detail}".strip())


class EchoConfig(C.Structure):
    _fields_ = [
        ("n_layers", C.c_int32), ("d_model", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
        ("head_dim", C.c_int32), ("d_ff", C.c_int32), ("vocab", C.c_int32),
        ("rms_eps", C.c_float), ("rope_theta", C.c_float), ("kv_page_size", C.c_int32),
        ("max_prompts", C.c_int32), ("max_G", C.c_int32), ("max_prompt_len", C.c_int32),
        ("max_new_tokens", C.c_int32), ("n_weight_buffers", C.c_int32), ("eos_id", C.c_int32),
        ("top_p", C.c_float), ("half_layers", C.c_int32), ("kv_pages", C.c_int32), ("queue_max_live", C.c_int32),
        ("queue_optimistic", C.c_int32),
    ]


class EchoWeights(C.Structure):
    _fields_ = [
        ("embed", C.c_void_p), ("lm_head", C.c_void_p), ("final_norm", C.c_void_p),
        ("wq", C.POINTER(C.c_void_p)), ("wk", C.POINTER(C.c_void_p)), ("wv", C.POINTER(C.c_void_p)),
        ("wo", C.POINTER(C.c_void_p)), ("w_gate", C.POINTER(C.c_void_p)), ("w_up", C.POINTER(C.c_void_p)),
        ("w_down", C.POINTER(C.c_void_p)), ("attn_norm", C.POINTER(C.c_void_p)),
        ("mlp_norm", C.POINTER(C.c_void_p)),
    ]


class EchoStats(C.Structure):
    _fields_ = [
        ("version_served", C.c_int64), ("tokens_generated", C.c_int64), ("kernels_launched", C.c_int64),
        ("decode_steps", C.c_int64), ("n_pages", C.c_int64), ("install_ms", C.c_float), ("prefill_ms", C.c_float),
        ("decode_ms", C.c_float), ("last_step_rows", C.c_float), ("queue_evictions", C.c_int64),
    ]


def _load() -> C.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2602_02192_b200.build` "
                          "(there is no fallback path)")
    lib = C.CDLL(LIB_PATH)
    vp, i32, u32, u64, i64, f32 = C.c_void_p, C.c_int32, C.c_uint32, C.c_uint64, C.c_int64, C.c_float
    lib.echo_arena_bytes.restype = C.c_size_t
    lib.echo_arena_bytes.argtypes = [C.POINTER(EchoConfig)]
    lib.echo_create.argtypes = [C.POINTER(EchoConfig), C.c_int, vp, C.c_size_t, vp, C.POINTER(vp)]
    lib.echo_destroy.argtypes = [vp]
    lib.echo_load_policy.argtypes = [vp, C.POINTER(EchoWeights), i64]
    lib.echo_wait_policy.argtypes = [vp]
    lib.echo_rollout.argtypes = [vp, vp, vp, i32, i32, i32, f32, u64, vp, vp, vp]
    lib.echo_rollout_forced.argtypes = [vp, vp, vp, i32, i32, i32, f32, u64, vp, vp, vp, vp]
    lib.echo_rollout_queue.argtypes = [vp, vp, vp, i32, i32, i32, f32, u64, vp, vp, vp, vp]
    lib.echo_rollout_queue.restype = C.c_int
    lib.echo_rollout_host.argtypes = [vp, vp, vp, i32, i32, i32, f32, u64, vp, vp, vp]
    lib.echo_score.argtypes = [vp, vp, vp, i32, i32, i32, f32, vp, vp, vp]
    lib.echo_score.restype = C.c_int
    lib.echo_turn_mask.argtypes = [vp, i32, i32, i32, i32, vp, vp]
    lib.echo_turn_mask.restype = C.c_int
    lib.echo_group_advantage.argtypes = [vp, i32, i32, f32, vp, vp]
    lib.echo_sync.argtypes = [vp]
    lib.echo_get_stats.argtypes = [vp, C.POINTER(EchoStats)]
    lib.echo_profile_config.argtypes = [vp, i32]
    lib.echo_profile_read.argtypes = [vp, vp, vp, i32, C.POINTER(i32)]
    lib.echo_debug_page_table.argtypes = [vp, vp, C.c_size_t, C.POINTER(i32), C.POINTER(i32)]
    lib.echo_plan_page_table.argtypes = [vp, i32, i32, i32, i32, vp, C.c_size_t, C.POINTER(i32), C.POINTER(i32)]
    lib.echo_plan_page_table.restype = C.c_int
    lib.echo_probe_read_bandwidth.argtypes = [vp, C.c_size_t, i32, vp, C.POINTER(f32), vp]
    lib.echo_probe_read_bandwidth.restype = C.c_int
    lib.echo_set_sequence_base.argtypes = [vp, u32]
    lib.echo_debug_capture.argtypes = [vp, i32, vp, vp, vp, vp]
    lib.echo_debug_wait_limit.argtypes = [u64, vp, C.POINTER(u64), vp]
    for name in ("echo_set_sequence_base", "echo_debug_capture", "echo_debug_wait_limit"):
        getattr(lib, name).restype = C.c_int
    lib.echo_debug_noise.argtypes = [u64, u32, u32, u32, u32, vp, vp, vp]
    lib.echo_sample.argtypes = [vp, i32, i32, i32, vp, u32, f32, u64, vp, vp, vp, vp]
    lib.echo_sample_top_p.argtypes = [vp, i32, i32, i32, vp, u32, f32, f32, u64, vp, vp, vp, vp, vp]
    lib.echo_sample_top_p.restype = C.c_int
    lib.echo_grpo_surrogate.argtypes = [vp, vp, vp, vp, vp, i32, i32, f32, f32, vp, vp]
    lib.echo_grpo_surrogate.restype = C.c_int
    lib.echo_grpo_objective.argtypes = [vp, vp, vp, vp, vp, vp, i32, i32, f32, f32, f32, vp, vp]
    lib.echo_grpo_objective.restype = C.c_int
    dbl = C.c_double
    lib.echo_mu_min.argtypes = [dbl, dbl, dbl, dbl, C.POINTER(dbl)]
    lib.echo_staleness_bound.argtypes = [i32, dbl, dbl, dbl, dbl, C.POINTER(i32)]
    lib.echo_greedy_provision.argtypes = [C.POINTER(dbl), C.POINTER(dbl), i32, dbl, C.POINTER(C.c_uint8),
                                          C.POINTER(i32), C.POINTER(dbl)]
    lib.echo_admissible.argtypes = [i64, i64, i64]
    lib.echo_peer_score.argtypes = [dbl, dbl, i32, i32, dbl, C.POINTER(dbl)]
    lib.echo_chain_assemble.argtypes = [C.POINTER(dbl), i32, dbl, dbl, C.POINTER(i32), C.POINTER(i32), C.POINTER(i32)]
    lib.echo_chain_arrival_time.argtypes = [dbl, dbl, dbl, i32, dbl, C.POINTER(dbl)]
    for name in ("echo_mu_min", "echo_staleness_bound", "echo_greedy_provision", "echo_admissible",
                 "echo_peer_score", "echo_chain_assemble", "echo_chain_arrival_time"):
        getattr(lib, name).restype = C.c_int
    lib.echo_gemm_bf16.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, vp, C.c_size_t, vp]
    lib.echo_decode_attention.argtypes = [vp, vp, i32, vp, i32, vp, vp, i32, i32, i32, i32, i32, vp, C.c_size_t, vp, i32, i32, vp]
    lib.echo_decode_attention.restype = C.c_int
    lib.echo_decode_attention_scratch_bytes.argtypes = [i32, i32, i32]
    lib.echo_decode_attention_scratch_bytes.restype = C.c_size_t
    lib.echo_gemm_bf16_noalloc.argtypes = [vp, vp, vp, i32, i32, i32, i32, vp]
    lib.echo_gemm_bf16_noalloc.restype = C.c_int
    lib.echo_gemm_bf16_noalloc_status.argtypes = [vp]
    lib.echo_gemm_bf16_noalloc_status.restype = C.c_int
    lib.echo_gemm_workspace_bytes.restype = C.c_size_t
    lib.echo_gemm_workspace_bytes.argtypes = [i32]
    lib.echo_tiled_weight_bytes.restype = C.c_size_t
    lib.echo_tiled_weight_bytes.argtypes = [i64, i64]
    lib.echo_retile_weights.restype = C.c_int
    lib.echo_retile_weights.argtypes = [vp, i64, i64, vp, C.c_size_t, vp]
    lib.echo_strerror.restype = C.c_char_p
    lib.echo_strerror.argtypes = [C.c_int]
    lib.echo_last_error.restype = C.c_char_p
    lib.echo_last_error.argtypes = [vp]
    for name in ("echo_create", "echo_destroy", "echo_load_policy", "echo_wait_policy", "echo_rollout",
                 "echo_rollout_forced", "echo_rollout_host", "echo_group_advantage", "echo_sync",
                 "echo_get_stats", "echo_profile_config", "echo_profile_read", "echo_debug_page_table", "echo_debug_noise", "echo_sample", "echo_gemm_bf16",
                 "echo_profile_config", "echo_profile_read"):
        getattr(lib, name).restype = C.c_int
    return lib


lib = _load()

EXPORTED = ["echo_arena_bytes", "echo_create", "echo_destroy", "echo_load_policy", "echo_wait_policy",
            "echo_rollout", "echo_rollout_forced", "echo_rollout_host", "echo_group_advantage", "echo_sync",
            "echo_get_stats", "echo_profile_config", "echo_profile_read", "echo_debug_page_table", "echo_debug_noise", "echo_sample", "echo_gemm_bf16",
            "echo_gemm_workspace_bytes", "echo_gemm_bf16_noalloc", "echo_decode_attention",
            "echo_decode_attention_scratch_bytes", "echo_plan_page_table", "echo_strerror", "echo_last_error",
            "echo_tiled_weight_bytes", "echo_retile_weights", "echo_sample_top_p", "echo_grpo_surrogate", "echo_grpo_objective", "echo_rollout_queue",
            "echo_mu_min", "echo_staleness_bound", "echo_greedy_provision", "echo_admissible",
            "echo_set_sequence_base", "echo_debug_capture", "echo_debug_wait_limit",
            "echo_gemm_bf16_noalloc_status", "echo_probe_read_bandwidth", "echo_peer_score", "echo_chain_assemble",
            "echo_chain_arrival_time", "echo_score", "echo_turn_mask"]


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return int(s.cuda_stream)


def _check(rc: int, ctx=None):
    if rc != ECHO_OK:
        detail = ""
        if ctx is not None and rc == -6:
            detail = lib.echo_last_error(ctx).decode()
        raise EchoError(rc, detail)


def make_config(shape, max_prompts: int, max_G: int, max_prompt_len: int, max_new_tokens: int,
                n_weight_buffers: int = 2, page_size: int = 16, eos_id: int = -1,
                top_p: float = 1.0, half_layers: int = 0, kv_pages: int = 0, queue_max_live: int = 0,
                queue_optimistic: int = 0) -> EchoConfig:
    """shape: any object with n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ff, vocab,
    rms_eps, rope_theta attributes."""
    return EchoConfig(shape.n_layers, shape.d_model, shape.n_q_heads, shape.n_kv_heads, shape.head_dim,
                      shape.d_ff, shape.vocab, shape.rms_eps, shape.rope_theta, page_size,
                      max_prompts, max_G, max_prompt_len, max_new_tokens, n_weight_buffers, eos_id, top_p,
                      min(int(half_layers), shape.n_layers), int(kv_pages), int(queue_max_live),
                      int(queue_optimistic))


def echo_arena_bytes(cfg: EchoConfig) -> int:
    return int(lib.echo_arena_bytes(C.byref(cfg)))


class Engine:
    """One context on one GPU.  Owns the arena tensor and a dedicated CUDA stream."""

    def __init__(self, cfg: EchoConfig, device: int = 0, stream: Optional[torch.cuda.Stream] = None):
        self.cfg = cfg
        self.device = torch.device("cuda", device)
        nbytes = echo_arena_bytes(cfg)
        if nbytes == 0:
            raise EchoError(-1, "configuration rejected")
        self.arena = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
        self.stream = stream if stream is not None else torch.cuda.Stream(device=self.device)
        self._ctx = C.c_void_p()
        self._keep = []          # weight tensors of installs that may still be running
        _check(lib.echo_create(C.byref(cfg), device, self.arena.data_ptr(), nbytes,
                               int(self.stream.cuda_stream), C.byref(self._ctx)))

    def close(self):
        if self._ctx:
            lib.echo_destroy(self._ctx)
            self._ctx = C.c_void_p()
            self._keep = []

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- policy ------------------------------------------------------------
    def echo_load_policy(self, weights: dict, version: int):
        """weights: name -> bf16 tensor (globals) or list of bf16 tensors (per layer); device or
        pinned host memory."""
        L = self.cfg.n_layers

        def arr(name):
            ts = weights[name]
            assert len(ts) == L
            for t in ts:
                assert t.dtype == torch.bfloat16 and t.is_contiguous()
            return (C.c_void_p * L)(*[t.data_ptr() for t in ts])

        for n in ("embed", "lm_head", "final_norm"):
            assert weights[n].dtype == torch.bfloat16 and weights[n].is_contiguous()
        arrays = {n: arr(n) for n in ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down", "attn_norm", "mlp_norm")}
        w = EchoWeights(weights["embed"].data_ptr(), weights["lm_head"].data_ptr(),
                        weights["final_norm"].data_ptr(),
                        *[C.cast(arrays[n], C.POINTER(C.c_void_p)) for n in
                          ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down", "attn_norm", "mlp_norm")])
        # source tensors written on torch's current stream must be complete before the copy reads them
        torch.cuda.current_stream(self.device).synchronize()
        _check(lib.echo_load_policy(self._ctx, C.byref(w), int(version)), self._ctx)
        self._keep.append(weights)
        self._keep = self._keep[-2:]

    def echo_wait_policy(self):
        _check(lib.echo_wait_policy(self._ctx), self._ctx)

    # -- rollouts ------------------------------------------------------------
    def echo_rollout(self, prompts: torch.Tensor, prompt_lens: Sequence[int], G: int, max_new_tokens: int,
                     temperature: float, seed: int, forced: Optional[torch.Tensor] = None,
                     out_tokens: Optional[torch.Tensor] = None, out_logprobs: Optional[torch.Tensor] = None):
        """prompts: int32 cuda tensor [P][cfg.max_prompt_len].  Returns (tokens int32 [P][G][T],
        logprobs fp32 [P][G][T] — both on the device, stream-ordered on self.stream — and versions
        int64 numpy [P][G])."""
        P = prompts.shape[0]
        assert prompts.dtype == torch.int32 and prompts.is_cuda and prompts.is_contiguous()
        assert prompts.shape[1] == self.cfg.max_prompt_len
        lens = np.ascontiguousarray(np.asarray(prompt_lens, dtype=np.int32))
        assert lens.shape == (P,)
        T = max_new_tokens
        if out_tokens is None:
            out_tokens = torch.empty((P, G, T), dtype=torch.int32, device=self.device)
        if out_logprobs is None:
            out_logprobs = torch.empty((P, G, T), dtype=torch.float32, device=self.device)
        versions = np.zeros((P, G), dtype=np.int64)
        # inputs produced on torch's current stream must be visible to the engine's stream
        self.stream.wait_stream(torch.cuda.current_stream(self.device))
        if forced is None:
            rc = lib.echo_rollout(self._ctx, prompts.data_ptr(), lens.ctypes.data, P, G, T, float(temperature),
                                  int(seed), out_tokens.data_ptr(), out_logprobs.data_ptr(), versions.ctypes.data)
        else:
            assert forced.dtype == torch.int32 and forced.is_cuda and forced.is_contiguous()
            assert tuple(forced.shape) == (P, G, T)
            rc = lib.echo_rollout_forced(self._ctx, prompts.data_ptr(), lens.ctypes.data, P, G, T,
                                         float(temperature), int(seed), forced.data_ptr(),
                                         out_tokens.data_ptr(), out_logprobs.data_ptr(), versions.ctypes.data)
        _check(rc, self._ctx)
        return out_tokens, out_logprobs, versions

    def echo_rollout_queue(self, prompts: torch.Tensor, prompt_lens: Sequence[int], G: int, max_new_tokens: int,
                           temperature: float, seed: int, forced: Optional[torch.Tensor] = None):
        """Rollout over a queue of prompts [n][cfg.max_prompt_len] (n may exceed cfg.max_prompts): freed
        slots are refilled from the queue.  Returns (tokens [n][G][T], logprobs [n][G][T], versions [n][G])."""
        n = prompts.shape[0]
        assert prompts.dtype == torch.int32 and prompts.is_cuda and prompts.is_contiguous()
        assert prompts.shape[1] == self.cfg.max_prompt_len
        lens = np.ascontiguousarray(np.asarray(prompt_lens, dtype=np.int32))
        assert lens.shape == (n,)
        T = max_new_tokens
        out_tokens = torch.empty((n, G, T), dtype=torch.int32, device=self.device)
        out_logprobs = torch.empty((n, G, T), dtype=torch.float32, device=self.device)
        versions = np.zeros((n, G), dtype=np.int64)
        if forced is not None:
            assert forced.dtype == torch.int32 and forced.is_cuda and forced.is_contiguous()
            assert tuple(forced.shape) == (n, G, T)
        self.stream.wait_stream(torch.cuda.current_stream(self.device))
        _check(lib.echo_rollout_queue(self._ctx, prompts.data_ptr(), lens.ctypes.data, n, G, T, float(temperature),
                                      int(seed), forced.data_ptr() if forced is not None else None,
                                      out_tokens.data_ptr(), out_logprobs.data_ptr(), versions.ctypes.data), self._ctx)
        return out_tokens, out_logprobs, versions

    def echo_score(self, prompts: torch.Tensor, prompt_lens: Sequence[int], tokens: torch.Tensor, temperature: float,
                   out_logprobs: Optional[torch.Tensor] = None):
        """Log-probabilities of given trajectories (int32 cuda [P][G][T]) in prefill-shaped passes.
        Returns (logprobs fp32 [P][G][T] on the device, versions)."""
        P, G, T = tokens.shape
        assert prompts.dtype == torch.int32 and prompts.is_cuda and prompts.is_contiguous()
        assert prompts.shape == (P, self.cfg.max_prompt_len)
        assert tokens.dtype == torch.int32 and tokens.is_cuda and tokens.is_contiguous()
        lens = np.ascontiguousarray(np.asarray(prompt_lens, dtype=np.int32))
        if out_logprobs is None:
            out_logprobs = torch.empty((P, G, T), dtype=torch.float32, device=self.device)
        versions = np.zeros((P, G), dtype=np.int64)
        self.stream.wait_stream(torch.cuda.current_stream(self.device))
        _check(lib.echo_score(self._ctx, prompts.data_ptr(), lens.ctypes.data, P, G, T, float(temperature),
                              tokens.data_ptr(), out_logprobs.data_ptr(), versions.ctypes.data), self._ctx)
        return out_logprobs, versions

    def echo_rollout_host(self, prompts: torch.Tensor, prompt_lens: Sequence[int], G: int, max_new_tokens: int,
                          temperature: float, seed: int, out_tokens: torch.Tensor, out_logprobs: torch.Tensor):
        """All buffers are host tensors (ideally pinned); returns versions.  Synchronous."""
        P = prompts.shape[0]
        assert not prompts.is_cuda and prompts.dtype == torch.int32 and prompts.is_contiguous()
        assert prompts.shape[1] == self.cfg.max_prompt_len
        assert not out_tokens.is_cuda and not out_logprobs.is_cuda
        lens = np.ascontiguousarray(np.asarray(prompt_lens, dtype=np.int32))
        versions = np.zeros((P, G), dtype=np.int64)
        _check(lib.echo_rollout_host(self._ctx, prompts.data_ptr(), lens.ctypes.data, P, G, max_new_tokens,
                                     float(temperature), int(seed), out_tokens.data_ptr(),
                                     out_logprobs.data_ptr(), versions.ctypes.data), self._ctx)
        return versions

    def echo_sync(self):
        _check(lib.echo_sync(self._ctx), self._ctx)

    def echo_get_stats(self) -> dict:
        st = EchoStats()
        _check(lib.echo_get_stats(self._ctx, C.byref(st)))
        return {k: getattr(st, k) for k, _ in EchoStats._fields_}

    def echo_profile_config(self, every_n_steps: int):
        _check(lib.echo_profile_config(self._ctx, int(every_n_steps)))

    def echo_profile_read(self):
        """(steps int32 [n], ms fp32 [n][4]) of the last rollout: attention, projections, sampler, step."""
        n = C.c_int32()
        _check(lib.echo_profile_read(self._ctx, None, None, 0, C.byref(n)), self._ctx)
        steps = np.zeros(n.value, dtype=np.int32)
        ms = np.zeros((n.value, 4), dtype=np.float32)
        if n.value:
            _check(lib.echo_profile_read(self._ctx, steps.ctypes.data, ms.ctypes.data, n.value, C.byref(n)),
                   self._ctx)
        return steps, ms

    def echo_set_sequence_base(self, base: int):
        _check(lib.echo_set_sequence_base(self._ctx, int(base)))

    def echo_debug_capture(self, layer: int, pre_in=None, pre_out=None, dec_in=None, dec_out=None):
        """fp32 cuda tensors (or None) that later rollouts fill with the residual stream around `layer`."""
        ptrs = []
        for t in (pre_in, pre_out, dec_in, dec_out):
            if t is not None:
                assert t.is_cuda and t.dtype == torch.float32 and t.is_contiguous()
            ptrs.append(t.data_ptr() if t is not None else None)
        self._capture_keep = (pre_in, pre_out, dec_in, dec_out)
        _check(lib.echo_debug_capture(self._ctx, int(layer), *ptrs))

    def echo_debug_page_table(self) -> np.ndarray:
        rows, width = C.c_int32(), C.c_int32()
        _check(lib.echo_debug_page_table(self._ctx, None, 0, C.byref(rows), C.byref(width)))
        out = np.zeros((rows.value, width.value), dtype=np.int32)
        if out.size:
            _check(lib.echo_debug_page_table(self._ctx, out.ctypes.data, out.size, C.byref(rows), C.byref(width)))
        return out


# -- context-free entry points --------------------------------------------------
def echo_group_advantage(rewards: torch.Tensor, eps: float = 1e-6, out: Optional[torch.Tensor] = None,
                         stream: Optional[torch.cuda.Stream] = None) -> torch.Tensor:
    assert rewards.is_cuda and rewards.dtype == torch.float32 and rewards.is_contiguous() and rewards.dim() == 2
    P, G = rewards.shape
    if out is None:
        out = torch.empty_like(rewards)
    with torch.cuda.device(rewards.device):
        _check(lib.echo_group_advantage(rewards.data_ptr(), P, G, float(eps), out.data_ptr(), _stream_ptr(stream)))
    return out


def echo_turn_mask(tokens: torch.Tensor, turn_start_id: int, shift_to_targets: bool = False) -> torch.Tensor:
    """uint8 [n][T] response mask of int32 token rows [n][T] (Appendix F, turn-aware masking)."""
    assert tokens.is_cuda and tokens.dtype == torch.int32 and tokens.is_contiguous() and tokens.dim() == 2
    n, T = tokens.shape
    out = torch.empty((n, T), dtype=torch.uint8, device=tokens.device)
    with torch.cuda.device(tokens.device):
        _check(lib.echo_turn_mask(tokens.data_ptr(), n, T, int(turn_start_id), 1 if shift_to_targets else 0,
                                  out.data_ptr(), _stream_ptr(None)))
    return out


def echo_grpo_objective(logp_new: torch.Tensor, logp_old: torch.Tensor, logp_sampler: torch.Tensor,
                        logp_ref: torch.Tensor, adv: torch.Tensor, mask: Optional[torch.Tensor], eps_clip: float,
                        C_trunc: float, beta: float) -> torch.Tensor:
    """The surrogate with the KL regulariser against a reference policy, one value per sequence."""
    n, T = logp_new.shape
    for x in (logp_new, logp_old, logp_sampler, logp_ref, adv):
        assert x.is_cuda and x.dtype == torch.float32 and x.is_contiguous()
    assert logp_old.shape == (n, T) and logp_sampler.shape == (n, T) and logp_ref.shape == (n, T) and adv.shape == (n,)
    if mask is not None:
        assert mask.is_cuda and mask.dtype == torch.uint8 and mask.is_contiguous() and mask.shape == (n, T)
    out = torch.empty(n, dtype=torch.float32, device=logp_new.device)
    with torch.cuda.device(logp_new.device):
        _check(lib.echo_grpo_objective(logp_new.data_ptr(), logp_old.data_ptr(), logp_sampler.data_ptr(),
                                       logp_ref.data_ptr(), adv.data_ptr(),
                                       mask.data_ptr() if mask is not None else None, n, T, float(eps_clip),
                                       float(C_trunc), float(beta), out.data_ptr(), _stream_ptr(None)))
    return out


def echo_grpo_surrogate(logp_new: torch.Tensor, logp_old: torch.Tensor, logp_sampler: torch.Tensor,
                        adv: torch.Tensor, mask: Optional[torch.Tensor], eps_clip: float, C_trunc: float) -> torch.Tensor:
    """Clipped surrogate with truncated importance sampling, one value per sequence ([n][T] inputs)."""
    n, T = logp_new.shape
    for x in (logp_new, logp_old, logp_sampler, adv):
        assert x.is_cuda and x.dtype == torch.float32 and x.is_contiguous()
    assert logp_old.shape == (n, T) and logp_sampler.shape == (n, T) and adv.shape == (n,)
    if mask is not None:
        assert mask.is_cuda and mask.dtype == torch.uint8 and mask.is_contiguous() and mask.shape == (n, T)
    out = torch.empty(n, dtype=torch.float32, device=logp_new.device)
    with torch.cuda.device(logp_new.device):
        _check(lib.echo_grpo_surrogate(logp_new.data_ptr(), logp_old.data_ptr(), logp_sampler.data_ptr(),
                                       adv.data_ptr(), mask.data_ptr() if mask is not None else None, n, T,
                                       float(eps_clip), float(C_trunc), out.data_ptr(), _stream_ptr(None)))
    return out


def echo_probe_read_bandwidth(n_bytes: int = 4 << 30, repeats: int = 10, device="cuda") -> float:
    """GB/s of a read-only pass over n_bytes of device memory (larger than L2 by default)."""
    buf = torch.empty(n_bytes // 16 * 16, dtype=torch.uint8, device=device)
    buf.zero_()
    sink = torch.zeros(1, dtype=torch.int32, device=device)
    ms = C.c_float(0.0)
    with torch.cuda.device(buf.device):
        torch.cuda.current_stream().synchronize()
        _check(lib.echo_probe_read_bandwidth(buf.data_ptr(), buf.numel(), int(repeats), sink.data_ptr(),
                                             C.byref(ms), _stream_ptr(None)))
    return buf.numel() / (ms.value * 1e-3) / 1e9


def echo_debug_wait_limit(limit_ns: int):
    """Runs the library's bounded wait on a barrier nobody signals; returns (return code, ns waited)."""
    waited = C.c_uint64(0)
    scratch = torch.zeros(2, dtype=torch.int64, device="cuda")
    rc = lib.echo_debug_wait_limit(int(limit_ns), scratch.data_ptr(), C.byref(waited), _stream_ptr(None))
    return rc, int(waited.value)


def echo_debug_noise(seed: int, s: int, j: int, v0: int, n: int, device="cuda"):
    words = torch.empty(n, dtype=torch.int32, device=device)
    uni = torch.empty(n, dtype=torch.float32, device=device)
    with torch.cuda.device(words.device):
        _check(lib.echo_debug_noise(int(seed), s, j, v0, n, words.data_ptr(), uni.data_ptr(), _stream_ptr(None)))
    return words, uni


def echo_sample(logits: torch.Tensor, rows: int, rows_per_logit_row: int, j: int, temperature: float, seed: int,
                seq_ids: Optional[torch.Tensor] = None, forced: Optional[torch.Tensor] = None):
    assert logits.is_cuda and logits.dtype == torch.float32 and logits.is_contiguous() and logits.dim() == 2
    V = logits.shape[1]
    tok = torch.empty(rows, dtype=torch.int32, device=logits.device)
    lp = torch.empty(rows, dtype=torch.float32, device=logits.device)
    with torch.cuda.device(logits.device):
        _check(lib.echo_sample(logits.data_ptr(), rows, V, rows_per_logit_row,
                               seq_ids.data_ptr() if seq_ids is not None else None, j, float(temperature),
                               int(seed), forced.data_ptr() if forced is not None else None,
                               tok.data_ptr(), lp.data_ptr(), _stream_ptr(None)))
    return tok, lp


def echo_sample_top_p(logits: torch.Tensor, rows: int, rows_per_logit_row: int, j: int, temperature: float,
                      top_p: float, seed: int, seq_ids: Optional[torch.Tensor] = None,
                      forced: Optional[torch.Tensor] = None):
    """echo_sample with nucleus truncation; returns (tokens, logprobs, cuts) where cuts[row] = (score key, id)
    of the last nucleus member of each logits row."""
    assert logits.is_cuda and logits.dtype == torch.float32 and logits.is_contiguous()
    V = logits.shape[-1]
    tok = torch.empty(rows, dtype=torch.int32, device=logits.device)
    lp = torch.empty(rows, dtype=torch.float32, device=logits.device)
    n_rows = (rows + rows_per_logit_row - 1) // rows_per_logit_row
    cuts = torch.zeros((n_rows, 2), dtype=torch.int64, device=logits.device).to(torch.int32).contiguous()
    with torch.cuda.device(logits.device):
        _check(lib.echo_sample_top_p(logits.data_ptr(), rows, V, rows_per_logit_row,
                                     seq_ids.data_ptr() if seq_ids is not None else None, j, float(temperature),
                                     float(top_p), int(seed), forced.data_ptr() if forced is not None else None,
                                     tok.data_ptr(), lp.data_ptr(), cuts.data_ptr(), _stream_ptr(None)))
    return tok, lp, cuts


def echo_gemm_bf16(X: torch.Tensor, W: torch.Tensor, impl: int = 0, epilogue: int = 0,
                   Y: Optional[torch.Tensor] = None) -> torch.Tensor:
    """epilogue 0: Y = X W^T (fp32); 1: Y += X W^T (fp32, Y given); 2: W = [Wg; Wu], Y = silu(X Wg^T) * (X Wu^T)
    (bf16).  impl >= 1000: W is given row-major and handed to the kernels in the block-tiled layout."""
    assert X.is_cuda and W.is_cuda and X.dtype == W.dtype and X.dtype in (torch.bfloat16, torch.float16)
    assert X.is_contiguous() and W.is_contiguous() and X.shape[1] == W.shape[1]
    M, K = X.shape
    N = W.shape[0] // 2 if epilogue == 2 else W.shape[0]
    half = X.dtype == torch.float16          # IEEE half operands (impl + 2000)
    if impl >= 1000:
        W = (torch.cat([echo_retile_weights(W[:N].contiguous()), echo_retile_weights(W[N:].contiguous())])
             if epilogue == 2 else echo_retile_weights(W))
    if Y is None:
        Y = torch.zeros((M, N), dtype=X.dtype if epilogue == 2 else torch.float32, device=X.device)
    with torch.cuda.device(X.device):
        nws = int(lib.echo_gemm_workspace_bytes(M)) if impl != 1 else 256
        ws = torch.empty(nws, dtype=torch.uint8, device=X.device)
        _check(lib.echo_gemm_bf16(X.data_ptr(), W.data_ptr(), Y.data_ptr(), M, N, K, epilogue,
                                  impl + (2000 if half else 0),
                                  ws.data_ptr(), nws, _stream_ptr(None)))
        torch.cuda.current_stream().synchronize()      # the workspace must outlive the kernel
    return Y


def echo_retile_weights(W: torch.Tensor) -> torch.Tensor:
    """Row-major bf16 matrix [rows][cols] -> the block-tiled layout (flat bf16 tensor) that echo_gemm_bf16
    reads with impl + 1000."""
    assert W.is_cuda and W.dtype in (torch.bfloat16, torch.float16) and W.is_contiguous() and W.dim() == 2
    rows, cols = W.shape
    n = int(lib.echo_tiled_weight_bytes(rows, cols))
    out = torch.empty(n // 2, dtype=W.dtype, device=W.device)
    with torch.cuda.device(W.device):
        _check(lib.echo_retile_weights(W.data_ptr(), rows, cols, out.data_ptr(), n, _stream_ptr(None)))
    return out


def echo_gemm_bf16_noalloc(X: torch.Tensor, W: torch.Tensor, Y: torch.Tensor, epilogue: int = 0) -> torch.Tensor:
    """Projection through the library's built-in scratch: this wrapper allocates nothing either, so
    the caller passes the output tensor (fp32 [M][N], or bf16 [M][N] for epilogue 2 with W = [Wg; Wu]).
    At most 32 rows; calls that may overlap on the GPU must not be issued concurrently."""
    assert X.is_cuda and W.is_cuda and Y.is_cuda and X.dtype == torch.bfloat16 and W.dtype == torch.bfloat16
    assert X.is_contiguous() and W.is_contiguous() and Y.is_contiguous() and X.shape[1] == W.shape[1]
    M, K = X.shape
    N = W.shape[0] // 2 if epilogue == 2 else W.shape[0]
    assert tuple(Y.shape) == (M, N) and Y.dtype == (torch.bfloat16 if epilogue == 2 else torch.float32)
    with torch.cuda.device(X.device):
        _check(lib.echo_gemm_bf16_noalloc(X.data_ptr(), W.data_ptr(), Y.data_ptr(), M, N, K, epilogue,
                                          _stream_ptr(None)))
    return Y


def echo_gemm_bf16_noalloc_status() -> int:
    """Waits for the current stream; how the last echo_gemm_bf16_noalloc on this device ended (0 = ok)."""
    return int(lib.echo_gemm_bf16_noalloc_status(_stream_ptr(None)))


def echo_decode_attention(q: torch.Tensor, kv_pool: torch.Tensor, page_table: torch.Tensor, row_pos: torch.Tensor,
                          full_pages: torch.Tensor, P: int, G: int, kernel_choice: int = 0) -> torch.Tensor:
    """q [B][Hq][hd]; kv_pool [n_pages][Hkv][2][16][hd], both bf16 or both float16; int32 device tensors
    for the tables."""
    assert q.dtype == kv_pool.dtype and q.dtype in (torch.bfloat16, torch.float16)
    B, Hq, hd = q.shape
    n_pages, Hkv = kv_pool.shape[0], kv_pool.shape[1]
    assert B == P * G and q.is_contiguous() and kv_pool.is_contiguous() and page_table.is_contiguous()
    assert page_table.dtype == torch.int32 and row_pos.dtype == torch.int32 and full_pages.dtype == torch.int32
    out = torch.empty_like(q)
    with torch.cuda.device(q.device):
        n = int(lib.echo_decode_attention_scratch_bytes(B, Hq, hd))
        scratch = torch.empty(n, dtype=torch.uint8, device=q.device)
        _check(lib.echo_decode_attention(q.data_ptr(), kv_pool.data_ptr(), n_pages, page_table.data_ptr(),
                                         page_table.shape[1], row_pos.data_ptr(), full_pages.data_ptr(), P, G, Hq,
                                         Hkv, hd, scratch.data_ptr(), n, out.data_ptr(),
                                         1 if q.dtype == torch.float16 else 0, int(kernel_choice), _stream_ptr(None)))
    return out


def echo_plan_page_table(prompt_lens, G: int, T: int, page_size: int = 16):
    """Host-only: (table int32 [P*G][width], prefill_table int32 [P][width], n_pages)."""
    lens = np.ascontiguousarray(np.asarray(prompt_lens, dtype=np.int32))
    P = len(lens)
    width, n_pages = C.c_int32(), C.c_int32()
    _check(lib.echo_plan_page_table(lens.ctypes.data, P, G, T, page_size, None, 0, C.byref(width), C.byref(n_pages)))
    out = np.zeros((P * G + P, width.value), dtype=np.int32)
    _check(lib.echo_plan_page_table(lens.ctypes.data, P, G, T, page_size, out.ctypes.data, out.size,
                                    C.byref(width), C.byref(n_pages)))
    return out[: P * G], out[P * G:], n_pages.value
