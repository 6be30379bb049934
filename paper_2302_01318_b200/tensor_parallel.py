"""Tensor-parallel sharding of a model's weights (host logic) and a single-GPU emulation of a tensor-parallel group.

The paper serves its target and draft Megatron-style over several chips (section Conditional Scoring): the attention
and feed-forward blocks are split across the chips and each is followed by an all-reduce of (K + 1) x d_model numbers.
`shard_config` / `shard_weights` cut a model accordingly -- wq, wk, wv, w_up by output rows (whole heads, contiguous
blocks), wo, w_down by the matching input columns; embeddings, unembedding and norm gains stay whole -- and `Group`
drives `world` rank handles on ONE GPU through the library's group calls, which is how the sharded arithmetic and the
exchange kernels are checked without `world` GPUs.  No arithmetic of the method lives here: only slicing and argument
marshalling."""
from __future__ import annotations

import ctypes as C

import numpy as np

from . import CFG_TENSOR_PARALLEL, Handle, _check, lib, sps_stats

ROW_SHARDED = ("wq", "wk", "wv", "w_up")       # by output rows
COL_SHARDED = ("wo", "w_down")                 # by input columns


def shard_config(cfg: dict, world: int) -> dict:
    """The sps_model_cfg of one rank's shard: d_model stays, heads and feed-forward features are divided."""
    kv = cfg.get("n_kv_heads", 0) or cfg["n_heads"]
    if world < 1 or cfg["n_heads"] % world or kv % world or cfg["d_ff"] % world:
        raise ValueError("world must divide n_heads, n_kv_heads and d_ff")
    return dict(cfg, n_heads=cfg["n_heads"] // world, n_kv_heads=kv // world, d_ff=cfg["d_ff"] // world)


def _rows(t, rank, world):
    n = t.shape[0] // world
    return t[rank * n:(rank + 1) * n]


def _cols(t, rank, world):
    n = t.shape[1] // world
    return t[:, rank * n:(rank + 1) * n]


def shard_weights(cfg: dict, w: dict, rank: int, world: int) -> dict:
    """Rank `rank`'s shard of the weights `w` (torch tensors or numpy arrays, any device): contiguous copies of its
    rows / columns; whole tensors are shared, not copied.  int8 models: row scales follow their rows (the scales of
    wo / w_down belong to output rows, which are not split)."""
    shard_config(cfg, world)   # validates
    if not 0 <= rank < world:
        raise ValueError("rank outside 0..world-1")

    def own(t):
        return t.contiguous() if hasattr(t, "contiguous") else np.ascontiguousarray(t)
    out = {k: v for k, v in w.items() if k != "layers"}
    out["layers"] = []
    for lw in w["layers"]:
        s = {k: v for k, v in lw.items() if k.endswith("norm")}
        for k in ROW_SHARDED:
            s[k] = own(_rows(lw[k], rank, world))
            if k + "_scale" in lw:
                s[k + "_scale"] = own(_rows(lw[k + "_scale"], rank, world))
        for k in COL_SHARDED:
            s[k] = own(_cols(lw[k], rank, world))
            if k + "_scale" in lw:
                s[k + "_scale"] = lw[k + "_scale"]
        out["layers"].append(s)
    return out


class Group:
    """`world` rank handles of one tensor-parallel group on one GPU and one stream, attached to one another with plain
    device pointers (on `world` GPUs each process would hold one of them and attach IPC-mapped peer buffers).
    target_w / draft_w: the WHOLE models' weights on the device; they are sharded here."""

    def __init__(self, world, target_cfg, target_w, draft_cfg=None, draft_w=None, max_seq=256, max_K=4, device=0):
        import torch
        self.world = world
        self.stream = torch.cuda.Stream(device=device)
        self.ranks = []
        for r in range(world):
            tw = shard_weights(target_cfg, target_w, r, world)
            dw = shard_weights(draft_cfg, draft_w, r, world) if draft_w is not None else None
            self.ranks.append(Handle(shard_config(target_cfg, world), tw, shard_config(draft_cfg, world) if draft_cfg else None, dw,
                                     max_seq=max_seq, max_batch=1, max_K=max_K, device=device, stream=self.stream.cuda_stream,
                                     flags=CFG_TENSOR_PARALLEL))
        bufs = [h.tp_buffers() for h in self.ranks]
        for r, h in enumerate(self.ranks):
            h.tp_attach(r, world, [b[0] for b in bufs], [b[1] for b in bufs])
        self._arr = (C.c_void_p * world)(*[h._h for h in self.ranks])
        self.vocab = target_cfg["vocab"]

    def prefill(self, toks):
        t = np.ascontiguousarray(toks, dtype=np.int32)
        _check(lib().sps_tp_group_prefill(self._arr, self.world, t.ctypes.data_as(C.c_void_p), t.shape[0]), self.ranks[0]._h)

    def score(self, which, rows, out_logits):
        """out_logits: list of `world` CUDA float32 tensors [n_rows, vocab]; returns the device time in ms."""
        r = np.ascontiguousarray(rows, dtype=np.int32)
        outs = (C.c_void_p * self.world)(*[o.data_ptr() for o in out_logits])
        ms = C.c_float(0)
        _check(lib().sps_tp_group_score(self._arr, self.world, which, r.ctypes.data_as(C.c_void_p), r.shape[0], outs, C.byref(ms)),
               self.ranks[0]._h)
        return ms.value

    def generate(self, prompt, n_new, K, temperature, seed):
        """The whole speculative loop on the emulated group: (tokens, stats of rank 0)."""
        p = np.ascontiguousarray(prompt, dtype=np.int32)
        out = np.zeros(n_new, dtype=np.int32)
        st = sps_stats()
        _check(lib().sps_tp_group_generate(self._arr, self.world, p.ctypes.data_as(C.c_void_p), p.shape[0], n_new, K, temperature, seed,
                                           out.ctypes.data_as(C.c_void_p), C.byref(st)), self.ranks[0]._h)
        return out, st.as_dict()

    def close(self):
        for h in self.ranks:
            h.close()
        self.ranks = []
