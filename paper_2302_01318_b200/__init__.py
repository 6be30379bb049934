"""Thin Python binding of libsps_b200.so (the C ABI of include/sps.h).

Argument marshalling only: torch supplies device memory and streams, every step of the path runs in
the library's CUDA kernels.  There is no CPU fallback: if the library is missing or there is no CUDA
device, calls raise.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

from . import build as _build

SPS_OK, SPS_EINVAL, SPS_ENOMEM, SPS_ECUDA, SPS_ERANGE, SPS_ESTATE, SPS_ETIMEOUT = 0, -1, -2, -3, -4, -5, -6
SPS_MAX_K = 15
FLAG_RESAMPLED, FLAG_BONUS, FLAG_FALLBACK = 1, 2, 4
CFG_NO_GRAPH = 1
CFG_TENSOR_PARALLEL = 2
LAYER_KEYS = ("attn_norm", "ffn_norm", "wq", "wk", "wv", "wo", "w_up", "w_down")
SCALED_KEYS = ("wq", "wk", "wv", "wo", "w_up", "w_down")   # matrices that carry row scales when weights are int8


class SpsError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__(f"sps error {code}: {msg}")
        self.code = code


class sps_model_cfg(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("d_model", C.c_int32), ("n_heads", C.c_int32), ("d_head", C.c_int32),
                ("d_ff", C.c_int32), ("vocab", C.c_int32), ("dtype", C.c_int32), ("rms_eps", C.c_float),
                ("rope_base", C.c_float), ("n_kv_heads", C.c_int32)]


class sps_cfg(C.Structure):
    _fields_ = [("target", sps_model_cfg), ("draft", sps_model_cfg), ("max_seq", C.c_int32), ("max_batch", C.c_int32),
                ("max_K", C.c_int32), ("device", C.c_int32), ("stream", C.c_void_p), ("flags", C.c_uint32)]


class sps_weights(C.Structure):
    _fields_ = [("tok_embed", C.c_void_p), ("unembed", C.c_void_p), ("final_norm", C.c_void_p)] + \
               [(k, C.POINTER(C.c_void_p)) for k in LAYER_KEYS] + [("unembed_scale", C.c_void_p)] + \
               [(k + "_scale", C.POINTER(C.c_void_p)) for k in SCALED_KEYS]


class sps_stats(C.Structure):
    _fields_ = [("loops", C.c_int32), ("draft_calls", C.c_int32), ("emitted", C.c_int32), ("accepted", C.c_int32),
                ("resampled", C.c_int32), ("bonus", C.c_int32), ("fallback", C.c_int32), ("overshoot", C.c_int32),
                ("hist_emitted", C.c_int32 * (SPS_MAX_K + 2)), ("ms_prefill", C.c_float), ("ms_decode", C.c_float),
                ("ms_draft", C.c_float), ("ms_verify", C.c_float), ("ms_accept", C.c_float), ("kernel_launches", C.c_int32)]

    def as_dict(self):
        d = {k: getattr(self, k) for k, _ in self._fields_ if k != "hist_emitted"}
        d["hist_emitted"] = list(self.hist_emitted)
        return d


_lib = None


def lib_path() -> str:
    return _build.LIB


def lib():
    """Load the CUDA library, building it first if the sources are newer.  Raises if that fails."""
    global _lib
    if _lib is None:
        path = _build.build()
        L = C.CDLL(path)
        vp, i32, u32, u64, f32, i64 = C.c_void_p, C.c_int32, C.c_uint32, C.c_uint64, C.c_float, C.c_int64
        L.sps_create.argtypes = [C.POINTER(sps_weights), C.POINTER(sps_weights), C.POINTER(sps_cfg), C.POINTER(vp)]
        L.sps_destroy.argtypes = [vp]
        L.sps_last_error.argtypes = [vp]
        L.sps_last_error.restype = C.c_char_p
        L.sps_generate.argtypes = [vp, vp, i32, i32, i32, f32, u64, vp, C.POINTER(sps_stats)]
        L.sps_generate_batch.argtypes = [vp, vp, i32, i32, i32, i32, f32, u64, vp, C.POINTER(sps_stats)]
        L.sps_reset.argtypes = [vp]
        L.sps_prefill.argtypes = [vp, vp, i32]
        L.sps_step.argtypes = [vp, i32, f32, u64, u32, vp, vp, vp]
        L.sps_last_logits.argtypes = [vp, i32, vp, vp, vp]
        L.sps_last_loop_trace.argtypes = [vp, vp, vp, vp, i32, vp]
        L.sps_set_forced_acceptance.argtypes = [vp, f32]
        L.sps_verify.argtypes = [vp, vp, i32, vp, C.POINTER(f32)]
        L.sps_score.argtypes = [vp, i32, vp, i32, vp, C.POINTER(f32)]
        L.sps_accept.argtypes = [vp, vp, vp, i32, i32, i32, f32, u64, u32, vp, vp, vp, vp]
        L.sps_sample.argtypes = [vp, i32, i32, f32, u64, u32, u32, vp, vp]
        L.sps_set_sampling.argtypes = [vp, i32, f32]
        L.sps_generate_adaptive.argtypes = [vp, vp, i32, i32, i32, i32, f32, u64, vp, C.POINTER(sps_stats)]
        L.sps_accept_filtered.argtypes = [vp, vp, vp, i32, i32, i32, f32, i32, f32, u64, u32, vp, vp, vp, vp]
        L.sps_sample_filtered.argtypes = [vp, i32, i32, f32, i32, f32, u64, u32, u32, vp, vp]
        L.sps_linear.argtypes = [vp, i32, vp, i32, i32, i32, vp, vp, vp, C.POINTER(f32)]
        L.sps_linear_scaled.argtypes = [vp, i32, vp, vp, i32, i32, i32, vp, vp, vp, C.POINTER(f32)]
        L.sps_linear_wide.argtypes = [vp, vp, i32, i32, i32, vp, vp, vp, C.POINTER(f32)]
        L.sps_linear_wide_workspace_bytes.argtypes = [i32, i32]
        L.sps_linear_wide_workspace_bytes.restype = i64
        L.sps_linear_workspace_bytes.argtypes = [i32, i32, i32, i32]
        L.sps_linear_workspace_bytes.restype = i64
        L.sps_philox.argtypes = [vp, vp, i32, vp, vp]
        L.sps_linear_static.argtypes = [vp, i32, vp, i32, i32, i32, vp, vp]
        L.sps_linear_static_max_floats.restype = i64
        L.sps_linear_static_floats_needed.argtypes = [i32, i32, i32, i32]
        L.sps_linear_static_floats_needed.restype = i64
        L.sps_prefill_batch.argtypes = [vp, vp, vp, i32, i32]
        L.sps_set_sequence_index0.argtypes = [vp, u32]
        L.sps_debug_set_wait.argtypes = [i64, i32]
        L.sps_tp_buffers.argtypes = [vp, C.POINTER(vp), C.POINTER(vp), C.POINTER(i64), C.POINTER(i64)]
        L.sps_tp_attach.argtypes = [vp, i32, i32, vp, vp]
        L.sps_tp_group_prefill.argtypes = [vp, i32, vp, i32]
        L.sps_tp_group_score.argtypes = [vp, i32, i32, vp, i32, vp, C.POINTER(f32)]
        L.sps_tp_group_generate.argtypes = [vp, i32, vp, i32, i32, i32, f32, u64, vp, C.POINTER(sps_stats)]
        _lib = L
    return _lib


def _check(rc, h=None):
    if rc != SPS_OK:
        msg = lib().sps_last_error(h)
        raise SpsError(rc, msg.decode() if msg else "")


def _np_ptr(a):
    return a.ctypes.data_as(C.c_void_p)


def _model_cfg(c: dict) -> sps_model_cfg:
    return sps_model_cfg(c["n_layers"], c["d_model"], c["n_heads"], c["d_head"], c["d_ff"], c["vocab"], c["dtype"],
                         c.get("rms_eps", 1e-5), c.get("rope_base", 10000.0), c.get("n_kv_heads", 0))


def _weights(w: dict, keep: list) -> sps_weights:
    sw = sps_weights()
    sw.tok_embed, sw.unembed, sw.final_norm = w["tok_embed"].data_ptr(), w["unembed"].data_ptr(), w["final_norm"].data_ptr()
    n = len(w["layers"])
    for k in LAYER_KEYS:
        arr = (C.c_void_p * max(n, 1))(*[lw[k].data_ptr() for lw in w["layers"]])
        keep.append(arr)
        setattr(sw, k, C.cast(arr, C.POINTER(C.c_void_p)))
    if "unembed_scale" in w:      # int8 weights (dtype 2): fp32 row scales beside every matrix
        sw.unembed_scale = w["unembed_scale"].data_ptr()
        for k in SCALED_KEYS:
            arr = (C.c_void_p * max(n, 1))(*[lw[k + "_scale"].data_ptr() for lw in w["layers"]])
            keep.append(arr)
            setattr(sw, k + "_scale", C.cast(arr, C.POINTER(C.c_void_p)))
    return sw


class Handle:
    """sps_create / sps_destroy and the calls that take a handle.  `target_w` / `draft_w` are dicts of
    CUDA torch tensors (tok_embed, unembed, final_norm, layers=[{attn_norm, ffn_norm, wq, wk, wv, wo,
    w_up, w_down}]); they must stay alive as long as the handle."""

    def __init__(self, target_cfg, target_w, draft_cfg=None, draft_w=None, max_seq=1024, max_batch=1, max_K=4,
                 device=0, stream=None, flags=0):
        self._keep = [target_w, draft_w]
        cfg = sps_cfg()
        cfg.target = _model_cfg(target_cfg)
        if draft_cfg is not None:
            cfg.draft = _model_cfg(draft_cfg)
        cfg.max_seq, cfg.max_batch, cfg.max_K, cfg.device = max_seq, max_batch, max_K, device
        cfg.stream = stream
        cfg.flags = flags
        tw = _weights(target_w, self._keep)
        dw = _weights(draft_w, self._keep) if draft_w is not None else None
        h = C.c_void_p()
        rc = lib().sps_create(C.byref(tw), C.byref(dw) if dw is not None else None, C.byref(cfg), C.byref(h))
        _check(rc, None)
        self._h = h
        self.vocab = target_cfg["vocab"]
        self.max_K = max_K
        self.B = 1          # sequences the last prefill set

    def close(self):
        if getattr(self, "_h", None):
            lib().sps_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def sps_generate(self, prompt, n_new, K, temperature, seed):
        p = np.ascontiguousarray(prompt, dtype=np.int32)
        out = np.zeros(n_new, dtype=np.int32)
        st = sps_stats()
        _check(lib().sps_generate(self._h, _np_ptr(p), p.shape[0], n_new, K, temperature, seed, _np_ptr(out), C.byref(st)),
               self._h)
        return out, st.as_dict()

    def sps_generate_adaptive(self, prompt, n_new, K_min, K_max, temperature, seed):
        p = np.ascontiguousarray(prompt, dtype=np.int32)
        out = np.zeros(n_new, dtype=np.int32)
        st = sps_stats()
        _check(lib().sps_generate_adaptive(self._h, _np_ptr(p), p.shape[0], n_new, K_min, K_max, temperature, seed, _np_ptr(out),
                                           C.byref(st)), self._h)
        return out, st.as_dict()

    def sps_generate_batch(self, prompts, n_new, K, temperature, seed):
        p = np.ascontiguousarray(prompts, dtype=np.int32)
        B, P = p.shape
        out = np.zeros((B, n_new), dtype=np.int32)
        st = (sps_stats * B)()
        _check(lib().sps_generate_batch(self._h, _np_ptr(p), B, P, n_new, K, temperature, seed, _np_ptr(out), st), self._h)
        return out, [s.as_dict() for s in st]

    def sps_set_sampling(self, top_k=0, top_p=1.0):
        _check(lib().sps_set_sampling(self._h, int(top_k), float(top_p)), self._h)

    def sps_set_forced_acceptance(self, alpha):
        """Measurement mode: accept every draft with probability alpha (0 = off)."""
        _check(lib().sps_set_forced_acceptance(self._h, float(alpha)), self._h)

    def sps_reset(self):
        _check(lib().sps_reset(self._h), self._h)
        self.B = 1

    def sps_prefill(self, toks):
        t = np.ascontiguousarray(toks, dtype=np.int32)
        _check(lib().sps_prefill(self._h, _np_ptr(t), t.shape[0]), self._h)
        self.B = 1

    def sps_prefill_batch(self, seqs):
        """seqs: list of B int sequences (their own lengths): the sequences so far of a batch."""
        lens = np.array([len(x) for x in seqs], dtype=np.int32)
        ld = int(lens.max())
        t = np.zeros((len(seqs), ld), dtype=np.int32)
        for b, x in enumerate(seqs):
            t[b, :len(x)] = x
        _check(lib().sps_prefill_batch(self._h, _np_ptr(t), _np_ptr(lens), len(seqs), ld), self._h)
        self.B = len(seqs)

    def tp_buffers(self):
        """(inbox pointer, flags pointer, inbox bytes, flags bytes) of a tensor-parallel rank's receive buffers."""
        inbox, flags, nb, nf = C.c_void_p(), C.c_void_p(), C.c_int64(0), C.c_int64(0)
        _check(lib().sps_tp_buffers(self._h, C.byref(inbox), C.byref(flags), C.byref(nb), C.byref(nf)), self._h)
        return inbox.value, flags.value, nb.value, nf.value

    def tp_attach(self, rank, world, peer_inbox, peer_flags):
        """peer_inbox / peer_flags: device addresses (ints) of every rank's buffers as this device sees them."""
        pi = (C.c_void_p * world)(*peer_inbox)
        pf = (C.c_void_p * world)(*peer_flags)
        _check(lib().sps_tp_attach(self._h, rank, world, pi, pf), self._h)

    def sps_set_sequence_index0(self, index0):
        """Sequence b of later generate / step calls uses Philox sequence index index0 + b."""
        _check(lib().sps_set_sequence_index0(self._h, int(index0)), self._h)

    def sps_step(self, K, temperature, seed, step):
        """One loop for every sequence of the last prefill.  Batch 1: (tokens [K+1], n_emitted, flags);
        batch B > 1: (tokens [B, K+1], n_emitted [B], flags [B])."""
        B = self.B
        out = np.full((B, K + 1), -1, dtype=np.int32)
        n = np.zeros(B, dtype=np.int32)
        fl = np.zeros(B, dtype=np.uint32)
        _check(lib().sps_step(self._h, K, temperature, seed, step, _np_ptr(out), _np_ptr(n), _np_ptr(fl)), self._h)
        if B == 1:
            return out[0], int(n[0]), int(fl[0])
        return out, n, fl

    def sps_last_loop_trace(self, cap=4096):
        """(loop_ms, loop_emitted, loop_K) of the last generation, one entry per loop."""
        ms, em, kk = np.zeros(cap, dtype=np.float32), np.zeros(cap, dtype=np.int32), np.zeros(cap, dtype=np.int32)
        n = C.c_int32(0)
        _check(lib().sps_last_loop_trace(self._h, _np_ptr(ms), _np_ptr(em), _np_ptr(kk), cap, C.byref(n)), self._h)
        m = min(n.value, cap)
        return ms[:m], em[:m], kk[:m]

    def sps_last_logits(self, K):
        """(q_logits, p_logits, drafts) of the last step: [K+1, V], [K, V], [K] for batch 1, with a leading B otherwise."""
        B = self.B
        q = np.zeros((B, K + 1, self.vocab), dtype=np.float32)
        p = np.zeros((B, K, self.vocab), dtype=np.float32)
        d = np.zeros((B, K), dtype=np.int32)
        _check(lib().sps_last_logits(self._h, K, _np_ptr(q), _np_ptr(p) if K else None, _np_ptr(d) if K else None), self._h)
        if B == 1:
            return q[0], p[0], d[0]
        return q, p, d

    def sps_verify(self, rows, K, out_logits):
        r = np.ascontiguousarray(rows, dtype=np.int32)
        ms = C.c_float(0)
        _check(lib().sps_verify(self._h, _np_ptr(r), K, out_logits.data_ptr(), C.byref(ms)), self._h)
        return ms.value

    def sps_score(self, which, rows, out_logits):
        r = np.ascontiguousarray(rows, dtype=np.int32)
        ms = C.c_float(0)
        _check(lib().sps_score(self._h, which, _np_ptr(r), r.shape[0], out_logits.data_ptr(), C.byref(ms)), self._h)
        return ms.value


def _stream_ptr(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    return stream


def sps_accept(q_logits, p_logits, draft_tokens, temperature, seed, step, out_n_accepted, out_tokens, out_flags,
               stream=None):
    """q_logits [B,K+1,V] fp32, p_logits [B,K,V] fp32, draft_tokens [B,K] int32: CUDA torch tensors;
    outputs CUDA int32 [B], int32 [B,K+1], int32-sized [B].  Enqueues one kernel on `stream`."""
    B, K1, V = q_logits.shape
    K = K1 - 1
    _check(lib().sps_accept(q_logits.data_ptr(), p_logits.data_ptr() if K else None,
                            draft_tokens.data_ptr() if K else None, B, K, V, temperature, seed, step,
                            _stream_ptr(stream), out_n_accepted.data_ptr(), out_tokens.data_ptr(), out_flags.data_ptr()))


def sps_accept_filtered(q_logits, p_logits, draft_tokens, temperature, top_k, top_p, seed, step, out_n_accepted, out_tokens,
                        out_flags, stream=None):
    """sps_accept with top-k / nucleus filtering of both distributions (temperature 0 = greedy)."""
    B, K1, V = q_logits.shape
    K = K1 - 1
    _check(lib().sps_accept_filtered(q_logits.data_ptr(), p_logits.data_ptr() if K else None,
                                     draft_tokens.data_ptr() if K else None, B, K, V, temperature, top_k, top_p, seed, step,
                                     _stream_ptr(stream), out_n_accepted.data_ptr(), out_tokens.data_ptr(),
                                     out_flags.data_ptr()))


def sps_sample_filtered(logits, temperature, top_k, top_p, seed, step, t, out_tokens, stream=None):
    B, V = logits.shape
    _check(lib().sps_sample_filtered(logits.data_ptr(), B, V, temperature, top_k, top_p, seed, step, t, _stream_ptr(stream),
                                     out_tokens.data_ptr()))


def sps_sample(logits, temperature, seed, step, t, out_tokens, stream=None):
    B, V = logits.shape
    _check(lib().sps_sample(logits.data_ptr(), B, V, temperature, seed, step, t, _stream_ptr(stream), out_tokens.data_ptr()))


def sps_linear_workspace_bytes(dtype, M, N, D):
    return int(lib().sps_linear_workspace_bytes(dtype, M, N, D))


def sps_linear(W, X, Y, workspace, stream=None, timed=False):
    """Y[M,N] = X[M,D] W[N,D]^T.  W CUDA fp32 or bf16, X/Y CUDA fp32, workspace CUDA uint8 (zeroed once)."""
    import torch
    dtype = 0 if W.dtype == torch.float32 else 1
    N, D = W.shape
    M = X.shape[0]
    ms = C.c_float(0)
    _check(lib().sps_linear(W.data_ptr(), dtype, X.data_ptr(), M, N, D, Y.data_ptr(), workspace.data_ptr(),
                            _stream_ptr(stream), C.byref(ms) if timed else None))
    return ms.value


def sps_linear_scaled(W, row_scale, X, Y, workspace, stream=None, timed=False):
    """Y[m,n] = row_scale[n] * sum_k X[m,k] W[n,k] with W CUDA int8 [N,D], row_scale CUDA fp32 [N]."""
    N, D = W.shape
    M = X.shape[0]
    ms = C.c_float(0)
    _check(lib().sps_linear_scaled(W.data_ptr(), 2, row_scale.data_ptr(), X.data_ptr(), M, N, D, Y.data_ptr(),
                                   workspace.data_ptr(), _stream_ptr(stream), C.byref(ms) if timed else None))
    return ms.value


def sps_linear_wide_workspace_bytes(N, D):
    return int(lib().sps_linear_wide_workspace_bytes(N, D))


def sps_linear_wide(W, X, Y, workspace, stream=None, timed=False):
    """Y[M,N] = X[M,D] W[N,D]^T for up to 128 rows (the prompt pass): W CUDA bf16, X/Y CUDA fp32."""
    N, D = W.shape
    M = X.shape[0]
    ms = C.c_float(0)
    _check(lib().sps_linear_wide(W.data_ptr(), X.data_ptr(), M, N, D, Y.data_ptr(), workspace.data_ptr(),
                                 _stream_ptr(stream), C.byref(ms) if timed else None))
    return ms.value


def sps_philox(ctr, key, out, stream=None):
    _check(lib().sps_philox(ctr.data_ptr(), key.data_ptr(), ctr.shape[0], _stream_ptr(stream), out.data_ptr()))


def sps_linear_static(W, X, Y, stream=None):
    """Y[M,N] = X[M,D] W[N,D]^T with the scratch held inside the library: for callers that cannot
    allocate device memory (see include/sps.h).  W CUDA fp32 or bf16, X/Y CUDA fp32."""
    import torch
    dtype = 0 if W.dtype == torch.float32 else 1
    N, D = W.shape
    _check(lib().sps_linear_static(W.data_ptr(), dtype, X.data_ptr(), X.shape[0], N, D, Y.data_ptr(), _stream_ptr(stream)))


def sps_linear_static_max_floats():
    return int(lib().sps_linear_static_max_floats())


def sps_linear_static_floats_needed(dtype, M, N, D):
    return int(lib().sps_linear_static_floats_needed(dtype, M, N, D))


def sps_debug_set_wait(limit_us=0, drop_stage=-1):
    """Test hook: bound of the kernels' waits in microseconds (0 = the default 2 s) and the stage the first CTA's copy
    producer leaves out (-1 = none)."""
    _check(lib().sps_debug_set_wait(int(limit_us), int(drop_stage)))
