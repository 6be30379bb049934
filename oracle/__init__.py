"""ORACLE -- test infrastructure only.

ctypes front end of ``sps_oracle.cpp``: a plain CPU statement of speculative
sampling (Algorithms 1 and 2, the modified rejection sampling scheme and
Theorem 1's quantities) and of the decoder both models are instances of.
Only the tests, the smoke check and the benchmark's CPU-baseline leg import
this package.  It imports nothing from the CUDA package and vice versa.

Arrays are numpy; bf16 tensors travel as ``uint16`` bit patterns.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sps_oracle.cpp")
_LIB = os.path.join(_HERE, "libsps_oracle.so")
_lib = None

FLAG_RESAMPLED = 1
FLAG_BONUS = 2
FLAG_FALLBACK = 4
FLAG_NEAR_ACCEPT = 256
FLAG_NEAR_CDF = 512
FLAG_NEAR_CUT = 1024


def build(force: bool = False) -> str:
    """Compile the oracle with the host compiler (no CUDA involved)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["g++", "-O2", "-std=c++17", "-pthread", "-shared", "-fPIC", "-o", _LIB, _SRC]
        subprocess.check_call(cmd)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        build()
        L = C.CDLL(_LIB)
        vp, i32, u32, u64, f64, i64 = C.c_void_p, C.c_int32, C.c_uint32, C.c_uint64, C.c_double, C.c_int64
        L.orc_philox4x32_10.argtypes = [vp, vp, vp]
        L.orc_uniforms.argtypes = [u64, u32, u32, u32, vp]
        L.orc_sample_row.argtypes = [vp, i32, f64, f64, vp]
        L.orc_sample_row.restype = i32
        L.orc_softmax.argtypes = [vp, i32, f64, vp]
        L.orc_accept_chain.argtypes = [vp, vp, vp, i32, i32, f64, u64, u32, u32, vp, vp, vp, vp]
        L.orc_accept_chain_wrong.argtypes = [vp, vp, vp, i32, i32, f64, u64, u32, u32, vp, vp]
        L.orc_table_model_create.argtypes = [vp, i32, i32, i32, i32]
        L.orc_table_model_create.restype = vp
        L.orc_tf_create.argtypes = [i32, i32, i32, i32, i32, i32, i32, f64, f64, i32]
        L.orc_tf_create.restype = vp
        L.orc_tf_set_globals.argtypes = [vp, vp, vp, vp]
        L.orc_tf_set_layer.argtypes = [vp, i32] + [vp] * 8
        L.orc_tf_begin_rows.argtypes = [vp, vp, vp, i32]
        L.orc_tf_layer.argtypes = [vp, i32] + [vp] * 8
        L.orc_tf_end.argtypes = [vp, vp, vp, vp, vp]
        L.orc_tf_hidden.argtypes = [vp, vp]
        L.orc_tf_kv.argtypes = [vp, i32, i32, vp, vp]
        L.orc_tf_set_kv_heads.argtypes = [vp, i32]
        L.orc_tf_set_kv_heads.restype = i32
        L.orc_model_forward.argtypes = [vp, vp, vp, i32, vp]
        L.orc_model_forward64.argtypes = [vp, vp, vp, i32, vp]
        L.orc_model_vocab.argtypes = [vp]
        L.orc_model_vocab.restype = i32
        L.orc_model_destroy.argtypes = [vp]
        L.orc_sps_create.argtypes = [vp, vp]
        L.orc_sps_create.restype = vp
        L.orc_sps_destroy.argtypes = [vp]
        L.orc_sps_reset.argtypes = [vp, vp, i32]
        L.orc_sps_len.argtypes = [vp]
        L.orc_sps_len.restype = i32
        L.orc_sps_tokens.argtypes = [vp, vp]
        L.orc_sps_last_logits.argtypes = [vp, vp, vp, vp]
        L.orc_sps_loop.argtypes = [vp, i32, f64, u64, u32, u32, vp, vp, vp, vp]
        L.orc_sps_loop.restype = i32
        L.orc_sps_generate.argtypes = [vp, vp, i32, i32, i32, f64, u64, u32, u32, vp, vp, vp, vp]
        L.orc_sps_generate.restype = i32
        L.orc_sps_trials.argtypes = [vp, vp, vp, i32, i32, i32, f64, u64, u32, i64, i32, vp, vp, vp, vp]
        L.orc_sps_trials_flagged.argtypes = [vp, vp, vp, i32, i32, i32, f64, u64, u32, i64, vp, vp, vp]
        L.orc_sps_trials_f.argtypes = [vp, vp, vp, i32, i32, i32, f64, i32, f64, u64, u32, i64, vp, vp, vp, vp]
        L.orc_sps_set_sampling.argtypes = [vp, i32, f64]
        L.orc_sample_row_f.argtypes = [vp, i32, f64, i32, f64, f64, vp]
        L.orc_sample_row_f.restype = i32
        L.orc_filtered.argtypes = [vp, i32, f64, i32, f64, vp, vp]
        L.orc_accept_chain_f.argtypes = [vp, vp, vp, i32, i32, f64, i32, f64, u64, u32, u32, vp, vp, vp, vp]
        L.orc_sps_generate_adaptive.argtypes = [vp, vp, i32, i32, i32, i32, f64, u64, u32, u32, vp, vp, vp, vp]
        L.orc_sps_generate_adaptive.restype = i32
        L.orc_sps_trials_adaptive.argtypes = [vp, vp, vp, i32, i32, i32, i32, f64, u64, u32, i64, vp, vp]
        L.orc_tf_set_cache_dtype.argtypes = [vp, i32]
        L.orc_num_threads.restype = i32
        L.orc_linear.argtypes = [vp, i32, vp, i32, i32, i32, vp]
        L.orc_set_threads.argtypes = [i32]
        L.orc_invcdf.argtypes = [vp, i32, f64, vp]
        L.orc_invcdf.restype = i32
        _lib = L
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def num_threads() -> int:
    return int(lib().orc_num_threads())


def set_threads(n: int) -> None:
    """Test hook: split large mat-vecs over n threads from now on (1 = none, 0 = the machine's count)."""
    lib().orc_set_threads(int(n))


def invcdf(weights, u: float):
    """Inverse-CDF draw in index order on unnormalised float64 weights: (token, near_tie)."""
    w = np.ascontiguousarray(weights, dtype=np.float64)
    nt = C.c_int(0)
    tok = lib().orc_invcdf(_p(w), w.shape[0], float(u), C.byref(nt))
    return int(tok), bool(nt.value)


def linear(W, X):
    """Y = X W^T in double.  W [N,D] float32 or uint16 (bf16 bits); X [M,D] float32."""
    W = np.ascontiguousarray(W)
    X = _f32(X)
    dtype = 0 if W.dtype == np.float32 else 1
    N, D = W.shape
    out = np.zeros((X.shape[0], N), dtype=np.float64)
    lib().orc_linear(_p(W), dtype, _p(X), X.shape[0], N, D, _p(out))
    return out


# --------------------------------------------------------------------------- RNG
def philox(ctr, key):
    c = np.asarray(ctr, dtype=np.uint32).copy()
    k = np.asarray(key, dtype=np.uint32).copy()
    out = np.zeros(4, dtype=np.uint32)
    lib().orc_philox4x32_10(_p(c), _p(k), _p(out))
    return out


def uniforms(seed: int, b: int, s: int, t: int):
    """(u_draft, u_acc, u_res) for sequence b, loop s, position t."""
    out = np.zeros(3, dtype=np.float64)
    lib().orc_uniforms(seed, b, s, t, _p(out))
    return out


# --------------------------------------------------------------------------- distributions
def softmax(logits, T: float = 1.0):
    lg = _f32(logits)
    out = np.zeros(lg.shape[-1], dtype=np.float64)
    lib().orc_softmax(_p(lg), lg.shape[-1], float(T), _p(out))
    return out


def filtered(logits, T: float = 1.0, top_k: int = 0, top_p: float = 1.0):
    """softmax(l / T) after top-k and nucleus filtering, renormalised; also whether the nucleus cut was a near tie."""
    lg = _f32(logits)
    out = np.zeros(lg.shape[-1], dtype=np.float64)
    nc = C.c_int(0)
    lib().orc_filtered(_p(lg), lg.shape[-1], float(T), int(top_k), float(top_p), _p(out), C.byref(nc))
    return out, bool(nc.value)


def sample_row(logits, T: float, u: float, top_k: int = 0, top_p: float = 1.0):
    lg = _f32(logits)
    nt = C.c_int(0)
    if top_k == 0 and top_p >= 1.0:
        tok = lib().orc_sample_row(_p(lg), lg.shape[-1], float(T), float(u), C.byref(nt))
    else:
        tok = lib().orc_sample_row_f(_p(lg), lg.shape[-1], float(T), int(top_k), float(top_p), float(u), C.byref(nt))
    return int(tok), bool(nt.value)


def accept_chain(q_logits, p_logits, drafts, T: float, seed: int, b: int, s: int, want_beta: bool = False,
                 wrong_rule: bool = False, top_k: int = 0, top_p: float = 1.0):
    """One loop's accept / resample / extra-token decision.  q_logits [K+1,V], p_logits [K,V]."""
    q = _f32(q_logits)
    K = q.shape[0] - 1
    V = q.shape[1]
    p = _f32(p_logits).reshape(K, V) if K > 0 else np.zeros((0, V), dtype=np.float32)
    d = _i32(drafts).reshape(K)
    out = np.full(K + 1, -1, dtype=np.int32)
    na = C.c_int32(0)
    fl = C.c_uint32(0)
    if wrong_rule:
        lib().orc_accept_chain_wrong(_p(q), _p(p), _p(d), K, V, float(T), seed, b, s, _p(out), C.byref(na))
        return {"n_accepted": int(na.value), "tokens": out}
    beta = np.zeros(max(K, 1), dtype=np.float64) if want_beta else None
    if top_k == 0 and top_p >= 1.0:
        lib().orc_accept_chain(_p(q), _p(p), _p(d), K, V, float(T), seed, b, s, _p(out), C.byref(na), C.byref(fl), _p(beta))
    else:
        lib().orc_accept_chain_f(_p(q), _p(p), _p(d), K, V, float(T), int(top_k), float(top_p), seed, b, s, _p(out),
                                 C.byref(na), C.byref(fl), _p(beta))
    res = {"n_accepted": int(na.value), "tokens": out, "flags": int(fl.value)}
    if want_beta:
        res["beta"] = beta[:K]
    return res


def accept_batch(q_logits, p_logits, drafts, T: float, seed: int, step: int, top_k: int = 0, top_p: float = 1.0):
    """accept_chain over a batch: q [B,K+1,V], p [B,K,V], drafts [B,K]; sequence index = row."""
    q = _f32(q_logits)
    B, K1, V = q.shape
    K = K1 - 1
    p = _f32(p_logits).reshape(B, K, V)
    d = _i32(drafts).reshape(B, K)
    n_acc = np.zeros(B, dtype=np.int32)
    toks = np.full((B, K + 1), -1, dtype=np.int32)
    flags = np.zeros(B, dtype=np.uint32)
    for b in range(B):
        r = accept_chain(q[b], p[b], d[b], T, seed, b, step, top_k=top_k, top_p=top_p)
        n_acc[b] = r["n_accepted"]
        toks[b] = r["tokens"]
        flags[b] = r["flags"]
    return n_acc, toks, flags


# --------------------------------------------------------------------------- models
class Model:
    def __init__(self, handle, keep=()):
        self._h = handle
        self._keep = list(keep)
        self.V = int(lib().orc_model_vocab(handle))

    def forward(self, tokens, positions, want_logits: bool = True):
        tok = _i32(tokens)
        pos = _i32(positions)
        M = tok.shape[0]
        if pos.shape[0] != M:
            raise ValueError("tokens and positions differ in length")
        out = np.zeros((M, self.V), dtype=np.float32) if want_logits else None
        lib().orc_model_forward(self._h, _p(tok), _p(pos), M, _p(out))
        return out

    def close(self):
        if self._h:
            lib().orc_model_destroy(self._h)
            self._h = None


class TableModel(Model):
    """Logits looked up from a table: context-free (depth 0, one row per position after pos0)
    or keyed on the last <= depth generated tokens."""

    def __init__(self, table, depth: int, pos0: int):
        t = _f32(table)
        h = lib().orc_table_model_create(_p(t), t.shape[0], t.shape[1], depth, pos0)
        super().__init__(h)


LAYER_KEYS = ("attn_norm", "ffn_norm", "wq", "wk", "wv", "wo", "w_up", "w_down")


class Transformer(Model):
    """cfg: dict(n_layers,d_model,n_heads,d_head,d_ff,vocab,dtype,rms_eps,rope_base[,n_kv_heads]);
    weights: dict(tok_embed, unembed, final_norm, layers=[dict(LAYER_KEYS)]) of numpy arrays,
    fp32 for dtype 0; uint16 bf16 bit patterns (norm gains stay fp32) for dtype 1."""

    def __init__(self, cfg: dict, weights: dict | None, max_seq: int, cache_dtype: int | None = None):
        self.cfg = dict(cfg)
        h = lib().orc_tf_create(cfg["n_layers"], cfg["d_model"], cfg["n_heads"], cfg["d_head"], cfg["d_ff"],
                                cfg["vocab"], cfg["dtype"], float(cfg.get("rms_eps", 1e-5)),
                                float(cfg.get("rope_base", 10000.0)), max_seq)
        if not h:
            raise ValueError("bad transformer config")
        super().__init__(h)
        if cfg.get("n_kv_heads", 0) not in (0, cfg["n_heads"]):      # multi-query / grouped-query attention
            if lib().orc_tf_set_kv_heads(h, int(cfg["n_kv_heads"])) != 0:
                raise ValueError("n_kv_heads must divide n_heads")
        if cache_dtype is not None:     # e.g. fp32 (dequantised) weights with a bf16 KV cache
            lib().orc_tf_set_cache_dtype(h, int(cache_dtype))
        if weights is not None:
            self.set_weights(weights)

    def _chk(self, a, gain=False):
        want = np.float32 if (gain or self.cfg["dtype"] == 0) else np.uint16
        a = np.ascontiguousarray(a)
        if a.dtype != want:
            raise TypeError(f"expected {want}, got {a.dtype}")
        self._keep.append(a)
        return a

    def set_weights(self, w: dict):
        te, ue, fn = self._chk(w["tok_embed"]), self._chk(w["unembed"]), self._chk(w["final_norm"], True)
        lib().orc_tf_set_globals(self._h, _p(te), _p(ue), _p(fn))
        for l, lw in enumerate(w["layers"]):
            arrs = [self._chk(lw[k], gain=k.endswith("norm")) for k in LAYER_KEYS]
            lib().orc_tf_set_layer(self._h, l, *[_p(a) for a in arrs])

    def forward64(self, tokens, positions):
        tok, pos = _i32(tokens), _i32(positions)
        if pos.shape[0] != tok.shape[0]:
            raise ValueError("tokens and positions differ in length")
        out = np.zeros((tok.shape[0], self.V), dtype=np.float64)
        lib().orc_model_forward64(self._h, _p(tok), _p(pos), tok.shape[0], _p(out))
        return out

    # layer-by-layer pass (a caller may hold one layer's weights at a time)
    def begin_rows(self, emb_rows, positions):
        e = self._chk(emb_rows)
        pos = _i32(positions)
        self._M = pos.shape[0]
        lib().orc_tf_begin_rows(self._h, _p(e), _p(pos), self._M)

    def layer(self, l: int, lw: dict):
        arrs = [self._chk(lw[k], gain=k.endswith("norm")) for k in LAYER_KEYS]
        lib().orc_tf_layer(self._h, l, *[_p(a) for a in arrs])
        del self._keep[-len(arrs):]

    def end(self, final_norm, unembed):
        fn, ue = self._chk(final_norm, True), self._chk(unembed)
        out = np.zeros((self._M, self.V), dtype=np.float64)
        lib().orc_tf_end(self._h, _p(fn), _p(ue), None, _p(out))
        return out

    def hidden(self):
        out = np.zeros((self._M, self.cfg["d_model"]), dtype=np.float64)
        lib().orc_tf_hidden(self._h, _p(out))
        return out

    def kv(self, l: int, position: int):
        d = (self.cfg.get("n_kv_heads", 0) or self.cfg["n_heads"]) * self.cfg["d_head"]
        k, v = np.zeros(d, dtype=np.float32), np.zeros(d, dtype=np.float32)
        lib().orc_tf_kv(self._h, l, position, _p(k), _p(v))
        return k, v


# --------------------------------------------------------------------------- loops
class Sps:
    """Algorithm 2 (K >= 1) / Algorithm 1 (K == 0) over two models."""

    def __init__(self, target: Model, draft: Model | None):
        self.target, self.draft = target, draft
        self.V = target.V
        self._h = lib().orc_sps_create(target._h, draft._h if draft is not None else None)

    def set_sampling(self, top_k: int = 0, top_p: float = 1.0):
        """top-k / nucleus filtering of both models' distributions (0 / 1.0 = off)."""
        lib().orc_sps_set_sampling(self._h, int(top_k), float(top_p))

    def reset(self, prompt):
        p = _i32(prompt)
        lib().orc_sps_reset(self._h, _p(p), p.shape[0])

    def tokens(self):
        n = lib().orc_sps_len(self._h)
        out = np.zeros(n, dtype=np.int32)
        lib().orc_sps_tokens(self._h, _p(out))
        return out

    def loop(self, K: int, T: float, seed: int, b: int, s: int):
        out = np.full(K + 1, -1, dtype=np.int32)
        na, fl, dnt = C.c_int32(0), C.c_uint32(0), C.c_uint32(0)
        e = lib().orc_sps_loop(self._h, K, float(T), seed, b, s, _p(out), C.byref(na), C.byref(fl), C.byref(dnt))
        return {"n_emitted": int(e), "n_accepted": int(na.value), "tokens": out, "flags": int(fl.value),
                "draft_near_tie": int(dnt.value)}

    def last_logits(self, K: int):
        q = np.zeros((K + 1, self.V), dtype=np.float32)
        p = np.zeros((K, self.V), dtype=np.float32)
        d = np.zeros(K, dtype=np.int32)
        lib().orc_sps_last_logits(self._h, _p(q), _p(p) if K else None, _p(d) if K else None)
        return q, p, d

    def generate(self, prompt, n_new: int, K: int, T: float, seed: int, b: int = 0, step0: int = 0):
        p = _i32(prompt)
        out = np.zeros(n_new, dtype=np.int32)
        loops = C.c_int32(0)
        hist = np.zeros(K + 2, dtype=np.int32)
        anyf = C.c_uint32(0)
        lib().orc_sps_generate(self._h, _p(p), p.shape[0], n_new, K, float(T), seed, b, step0, _p(out),
                               C.byref(loops), _p(hist), C.byref(anyf))
        return {"tokens": out, "loops": int(loops.value), "hist_emitted": hist, "flags": int(anyf.value)}

    def generate_adaptive(self, prompt, n_new: int, K_min: int, K_max: int, T: float, seed: int, b: int = 0, step0: int = 0):
        """Generation with the lookahead adapted from loop to loop (grow after a fully accepted loop, shrink after a
        first-draft rejection)."""
        p = _i32(prompt)
        out = np.zeros(n_new, dtype=np.int32)
        loops, drafts, anyf = C.c_int32(0), C.c_int32(0), C.c_uint32(0)
        lib().orc_sps_generate_adaptive(self._h, _p(p), p.shape[0], n_new, K_min, K_max, float(T), seed, b, step0, _p(out),
                                        C.byref(loops), C.byref(drafts), C.byref(anyf))
        return {"tokens": out, "loops": int(loops.value), "draft_calls": int(drafts.value), "flags": int(anyf.value)}

    def close(self):
        if self._h:
            lib().orc_sps_destroy(self._h)
            self._h = None


def trials(target: Model, draft: Model | None, prompt, n_new: int, K: int, T: float, seed: int, n_trials: int,
           b0: int = 0, wrong_rule: bool = False, top_k: int = 0, top_p: float = 1.0):
    """n_trials independent generations of n_new tokens (trial i uses sequence index b0+i)."""
    p = _i32(prompt)
    out = np.zeros((n_trials, n_new), dtype=np.int32)
    hist = np.zeros(K + 2, dtype=np.int64)
    first_acc = np.zeros(n_trials, dtype=np.int32)
    first_flags = np.zeros(n_trials, dtype=np.uint32)
    if top_k == 0 and top_p >= 1.0:
        lib().orc_sps_trials(target._h, draft._h if draft is not None else None, _p(p), p.shape[0], n_new, K, float(T),
                             seed, b0, n_trials, int(wrong_rule), _p(out), _p(hist), _p(first_acc), _p(first_flags))
    else:
        assert not wrong_rule
        lib().orc_sps_trials_f(target._h, draft._h if draft is not None else None, _p(p), p.shape[0], n_new, K, float(T),
                               int(top_k), float(top_p), seed, b0, n_trials, _p(out), _p(hist), _p(first_acc), _p(first_flags))
    return {"tokens": out, "hist_emitted": hist, "first_n_accepted": first_acc, "first_flags": first_flags}


def trials_flagged(target: Model, draft: Model | None, prompt, n_new: int, K: int, T: float, seed: int, n_trials: int,
                   b0: int = 0):
    """trials() that also returns, per trial, the flags of all its loops OR-ed together (near ties of draft draws
    included as FLAG_NEAR_CDF): the trials another implementation may legitimately decide differently."""
    p = _i32(prompt)
    out = np.zeros((n_trials, n_new), dtype=np.int32)
    hist = np.zeros(K + 2, dtype=np.int64)
    flags = np.zeros(n_trials, dtype=np.uint32)
    lib().orc_sps_trials_flagged(target._h, draft._h if draft is not None else None, _p(p), p.shape[0], n_new, K, float(T),
                                 seed, b0, n_trials, _p(out), _p(hist), _p(flags))
    return {"tokens": out, "hist_emitted": hist, "flags": flags}


def trials_adaptive(target: Model, draft: Model, prompt, n_new: int, K_min: int, K_max: int, T: float, seed: int,
                    n_trials: int, b0: int = 0):
    """n_trials independent adaptive-lookahead generations of n_new tokens."""
    p = _i32(prompt)
    out = np.zeros((n_trials, n_new), dtype=np.int32)
    tot = C.c_int64(0)
    lib().orc_sps_trials_adaptive(target._h, draft._h, _p(p), p.shape[0], n_new, K_min, K_max, float(T), seed, b0, n_trials,
                                  _p(out), C.byref(tot))
    return {"tokens": out, "draft_calls": int(tot.value)}
