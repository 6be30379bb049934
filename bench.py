#!/usr/bin/env python
"""Benchmark of the speculative-sampling hot path on B200.

One "step" = one whole generation through the library (`sps_generate`): prompt of P tokens, then
n_new tokens by speculative sampling with lookahead K at batch 1, i.e. every row of the hot path (K
draft steps, one K+1-row scoring pass, the fused accept / resample kernel, cache rollback, loop
control) run ~n_new/(tokens per loop) times.  Default workload: the 70B-shaped target with the 4B-shaped
draft (random-init bf16 weights generated on the device, shared (un)embedding), P = 128, n_new = 128,
K = 4, temperature 1 -- the configuration the headline metric is quoted on.

  value : tokens/s over the decode loops, timed with CUDA events on the library's stream (inputs resident)
  e2e   : tokens/s of the same calls by wall clock, prompt upload, prompt pass and result read-back included
  ar    : the same library's autoregressive decode (K = 0) on the same models

N > 1 (torchrun): independent replicas, one per GPU, no collective on the data path; the time is the
max over ranks.  `--impl reference` times the CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

import sps_synth  # noqa: E402

METRIC = "batch-1 tokens/s SpS vs AR decode; verify-pass HBM GB/s vs peak"
UNIT = "tokens/s"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            d = json.load(open(path))
            return float(d["hbm_gbs"]), "measured (MEASURED_PEAKS.json, device copy)"
        except Exception:
            pass
    return 6650.0, "fallback (earlier measurement on this pool)"


class ClockSampler:
    """nvidia-smi clocks and throttle reasons during the timed region"""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "200"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            self.th = threading.Thread(target=self._read, daemon=True)
            self.th.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons, pw = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1])); pw.append(float(f[2]))
            except ValueError:
                continue
            for nm, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(pw) if pw else None, "samples": len(sm), "reasons": sorted(reasons)}


def build_models(cfgname, device):
    c = sps_synth.CONFIGS[cfgname]
    wt = sps_synth.make_weights(c["target"], seed=0, tag="target", device=device)
    share = wt if cfgname.startswith("70b") else None
    wd = sps_synth.make_weights(c["draft"], seed=0, tag="draft", device=device, share_embed_from=share)
    return c, wt, wd


def kv_bytes_per_token(cfg):
    dkv = cfg.get("n_kv_heads", cfg["n_heads"]) * cfg["d_head"]
    return cfg["n_layers"] * 2 * dkv * (4 if cfg["dtype"] == 0 else 2)


# ----------------------------------------------------------------------------------------------- CPU oracle legs
class PinnedStage:
    """Reusable pinned host buffers for reading a layer's matrices back from the device (one per matrix name)."""

    def __init__(self):
        self.buf = {}

    def numpy(self, name, t):
        """`t` (device tensor, fp32 or bf16) as the numpy array the oracle reads; the array aliases a pinned buffer that
        the next call with the same name overwrites."""
        src = t.view(torch.int16) if t.dtype == torch.bfloat16 else t
        key = (name, src.dtype)
        if key not in self.buf or self.buf[key].numel() < src.numel():
            self.buf[key] = torch.empty(src.numel(), dtype=src.dtype, pin_memory=True)
        dst = self.buf[key][:src.numel()].view(src.shape)
        dst.copy_(src)
        a = dst.numpy()
        return a.view(np.uint16) if t.dtype == torch.bfloat16 else a


def oracle_full_pass(cfg, w_dev, tokens, stage):
    """One pass of the oracle over ALL layers of a device-resident model, the weights read back one layer at a time:
    rows `tokens` at positions 0 .. len - 1 with an empty cache.  Returns (logits float64 [rows, V], oracle seconds,
    read-back seconds).  An int8 model is the fp32 model of its dequantised matrices with a bf16 cache."""
    import oracle
    q8 = cfg["dtype"] == 2
    tok = torch.from_numpy(np.asarray(tokens, dtype=np.int64)).to(w_dev["tok_embed"].device)
    pos = np.arange(len(tokens), dtype=np.int32)
    emb = w_dev["tok_embed"][tok]
    m = oracle.Transformer(dict(cfg, dtype=0), None, len(tokens) + 1, cache_dtype=1) if q8 else oracle.Transformer(cfg, None, len(tokens) + 1)
    t_orc = t_copy = 0.0
    t0 = time.perf_counter()
    m.begin_rows(emb.float().cpu().numpy() if q8 else sps_synth.to_numpy(emb), pos)
    t_orc += time.perf_counter() - t0
    for l, lw in enumerate(w_dev["layers"]):
        t0 = time.perf_counter()
        if q8:
            one = layer_numpy(lw)
        else:
            one = {k: stage.numpy(k, v) for k, v in lw.items()}
        t1 = time.perf_counter()
        m.layer(l, one)
        t2 = time.perf_counter()
        t_copy += t1 - t0
        t_orc += t2 - t1
    t0 = time.perf_counter()
    un = unembed_numpy(w_dev) if q8 else stage.numpy("unembed", w_dev["unembed"])
    t1 = time.perf_counter()
    out = m.end(w_dev["final_norm"].cpu().numpy(), un)
    t_orc += time.perf_counter() - t1
    t_copy += t1 - t0
    m.close()
    return out, t_orc, t_copy


def cpu_baseline_full(h, c, wt, wd, K, tokens_per_loop, dev):
    """The oracle, as it stands, on ONE FULL scoring step of the bench's target (all layers, K + 1 rows) and one full
    draft step (all layers, one row), on the machine's host cores, with the very weights the GPU arm uses (read back
    layer by layer); the library scores the same rows so that the logit error is reported beside the time."""
    import oracle
    V = c["target"]["vocab"]
    rows = np.concatenate([sps_synth.make_prompt(0, 1, V), sps_synth.make_prompt(1, K, V)])      # x_0, then K draft tokens
    stage = PinnedStage()
    want, t_verify, t_copy = oracle_full_pass(c["target"], wt, rows, stage)
    h.sps_reset()
    h.sps_prefill(rows[:1])                      # a one-token sequence: nothing cached, the scoring rows sit at positions 0 .. K
    out = torch.zeros((K + 1, V), device=dev)
    h.sps_score(0, rows, out)
    err = float(np.abs(out.cpu().numpy().astype(np.float64) - want).max())
    _, t_draft, t_copy_d = oracle_full_pass(c["draft"], wd, rows[:1], stage) if K > 0 else (None, 0.0, 0.0)
    loop_s = t_verify + K * t_draft
    tl, dl = c["target"]["n_layers"], c["draft"]["n_layers"]
    return {"value": tokens_per_loop / loop_s, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": (f"one full scoring step of the oracle: {tl} of {tl} target layers + unembedding over {K + 1} rows "
                       f"(positions 0..{K}; the mat-vecs are >99.9% of its work at any context), {t_verify:.1f} s; one full draft step: "
                       f"{dl} of {dl} layers + unembedding over 1 row, {t_draft:.2f} s, counted {K} times; weights read back from the "
                       f"device layer by layer ({t_copy + t_copy_d:.1f} s, not counted); divided into the GPU arm's measured "
                       f"{tokens_per_loop:.3f} tokens per loop on the same models and seeds"),
            "seconds": {"verify_step": t_verify, "draft_step": t_draft, "loop": loop_s, "weight_readback": t_copy + t_copy_d},
            "logit_max_abs_err_vs_gpu": err, "logit_tolerance": 5e-2 if c["target"]["dtype"] >= 1 else 1e-3}


def oracle_loop_sample(c, K, models, seed, step):
    """One iteration of Algorithm 2 by the oracle on a depth-reduced pair (full widths and vocabulary), in pieces so that
    the draft steps and the scoring step are timed apart: K draft steps (one row each after the first), one scoring
    step over K + 1 rows, then the oracle's accept chain on its own logits.  Returns (draft seconds, scoring seconds,
    tokens emitted)."""
    import oracle
    ot, od, prefix = models
    n = len(prefix)
    V = c["target"]["vocab"]
    drafts, p_rows = [], []
    t0 = time.perf_counter()
    for t in range(K):
        tok = prefix[-1] if t == 0 else drafts[-1]
        lg = od.forward(np.array([tok], dtype=np.int32), np.array([n - 1 + t], dtype=np.int32))[0]
        d, _ = oracle.sample_row(lg, 1.0, oracle.uniforms(seed, 0, step, t)[0])
        drafts.append(d); p_rows.append(lg)
    t1 = time.perf_counter()
    rows = np.array([prefix[-1]] + drafts, dtype=np.int32)
    q = ot.forward(rows, np.arange(n - 1, n + K, dtype=np.int32))
    t2 = time.perf_counter()
    r = oracle.accept_chain(q, np.stack(p_rows) if K else np.zeros((0, V), np.float32), drafts, 1.0, seed, 0, step)
    return t1 - t0, t2 - t1, r["n_accepted"] + 1


def layer_numpy(lw):
    """One layer as the oracle reads it; an int8 layer as its dequantised fp32 matrices."""
    if "wq_scale" in lw:
        out = {k: lw[k].cpu().numpy() for k in ("attn_norm", "ffn_norm")}
        for k in sps_synth.LAYER_MATS:
            out[k] = (lw[k].float() * lw[k + "_scale"][:, None]).cpu().numpy()
        return out
    return {k: sps_synth.to_numpy(v) for k, v in lw.items()}


def unembed_numpy(w):
    if "unembed_scale" in w:
        return (w["unembed"].float() * w["unembed_scale"][:, None]).cpu().numpy()
    return sps_synth.to_numpy(w["unembed"])


DTYPE_NAME = {0: "fp32", 1: "bf16", 2: "int8-weight (row scales, fp16 activations, bf16 KV cache)"}


def run_reference(args):
    """--impl reference: the CPU oracle on the host cores (no GPU work).  Every step is one real iteration of
    Algorithm 2 by the oracle on a depth-reduced pair -- one target layer and one draft layer at the bench's full
    widths and vocabulary, random-init by the bench's recipe -- timed in its two phases; each phase is scaled to the
    full pair by the weight bytes a pass streams (the oracle's time is its mat-vecs'), and the tokens per loop are
    the oracle's own emitted counts.  Seconds per loop and the scale factors are in the line."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    cfgname = args.config
    c = sps_synth.CONFIGS[cfgname]
    K, P, n_new = args.K, c["prompt_len"], c["n_new"]
    tc, dc = c["target"], c["draft"]
    tc1, dc1 = dict(tc, n_layers=min(1, tc["n_layers"])), dict(dc, n_layers=min(1, dc["n_layers"]))
    one_t = sps_synth.make_weights(tc1, seed=0, tag="target", device="cpu")
    one_d = sps_synth.make_weights(dc1, seed=0, tag="draft", device="cpu", share_embed_from=one_t if cfgname.startswith("70b") else None)

    def orc(cfg1, w):
        if cfg1["dtype"] == 2:
            return oracle.Transformer(dict(cfg1, dtype=0), sps_synth.dequantized_numpy(w), 16 + K, cache_dtype=1)
        return oracle.Transformer(cfg1, sps_synth.weights_to_numpy(w), 16 + K)
    ot, od = orc(tc1, one_t), orc(dc1, one_d)
    prefix = [int(t) for t in sps_synth.make_prompt(0, 4, tc["vocab"])]
    pre = np.array(prefix[:-1], dtype=np.int32)
    ot.forward(pre, np.arange(len(pre)), want_logits=False)
    od.forward(pre, np.arange(len(pre)), want_logits=False)
    scale_t = sps_synth.weight_bytes(tc) / sps_synth.weight_bytes(tc1)
    scale_d = sps_synth.weight_bytes(dc) / sps_synth.weight_bytes(dc1)
    loop_s, emitted = [], []
    for i in range(args.warmup + args.steps):
        td, tv, e = oracle_loop_sample(c, K, (ot, od, prefix), seed=i, step=i)
        if i >= args.warmup:
            loop_s.append(td * scale_d + tv * scale_t)
            emitted.append(e)
    mean_loop, tpl = statistics.mean(loop_s), statistics.mean(emitted)
    value = tpl / mean_loop
    sample = (f"per step: one iteration of Algorithm 2 by the oracle on a depth-reduced pair (1 of {tc['n_layers']} target layers, 1 of "
              f"{dc['n_layers']} draft layers, full widths and vocabulary, context {len(prefix)}): {K} draft steps, one scoring step over "
              f"{K + 1} rows, accept chain; phase times scaled by streamed weight bytes (target x{scale_t:.1f}, draft x{scale_d:.1f}); "
              f"tokens per loop = the oracle's own mean emitted count ({tpl:.2f})")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * mean_loop * (n_new / tpl), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": workload_name(cfgname, K, P, n_new)},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample,
                             "seconds_per_loop": mean_loop, "tokens_per_loop": tpl},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def workload_name(cfgname, K, P, n_new):
    c = sps_synth.CONFIGS[cfgname]
    t, d = c["target"], c["draft"]
    return (f"{cfgname}: target L{t['n_layers']}/d{t['d_model']}/ff{t['d_ff']}/V{t['vocab']}, draft L{d['n_layers']}/"
            f"d{d['d_model']}/ff{d['d_ff']}, {DTYPE_NAME[t['dtype']]} random-init N(0,0.02) "
            f"(shared (un)embedding), prompt {P}, generate {n_new}, K={K}, T=1.0, batch 1")


# ----------------------------------------------------------------------------------------------- GPU arm
def run_ours(args):
    import paper_2302_01318_b200 as sps
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(dev))
    cfgname, K = args.config, args.K
    c, wt, wd = build_models(cfgname, dev)
    P, n_new, T = c["prompt_len"], c["n_new"], 1.0
    V = c["target"]["vocab"]
    max_seq = ((P + n_new + max(K, 8) + 63) // 64) * 64
    h = sps.Handle(c["target"], wt, c["draft"], wd, max_seq=max_seq, max_batch=1, max_K=max(K, 8), device=local)
    from paper_2302_01318_b200 import replicas
    # independent replicas: rank r generates the global sequences r, r + world, ... (no collective on the data path)
    seeds = replicas.shard_sequences((args.warmup + args.steps + 8) * world, rank, world)

    def gen(i, k, temp=None):
        prompt = sps_synth.make_prompt(seeds[i], P, V)
        t0 = time.perf_counter()
        out, st = h.sps_generate(prompt, n_new, k, T if temp is None else temp, seeds[i])
        return out, st, time.perf_counter() - t0

    def sps_generate_seeded(hh, seed_, k):
        return hh.sps_generate(sps_synth.make_prompt(seed_, P, V), n_new, k, T, seed_)[1]

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(args.warmup):
        gen(i, K)
    clk = ClockSampler(local)
    barrier()
    clk.start()
    stats, walls, loop_ms, loop_tok = [], [], [], []
    for i in range(args.steps):
        _, st, w = gen(args.warmup + i, K)
        stats.append(st); walls.append(w)
        ms, em, _ = h.sps_last_loop_trace()
        loop_ms.append(ms); loop_tok.append(em)
    barrier()
    clocks = clk.stop()
    dec_s, tokens = replicas.job_time_and_tokens(sum(s["ms_decode"] for s in stats) / 1e3, args.steps * n_new, dist, dev)
    wall_s, _ = replicas.job_time_and_tokens(sum(walls), 0, dist, dev)
    dec_ms = dec_s * 1e3
    value = tokens / (dec_ms / 1e3)
    e2e = tokens / wall_s
    loops = sum(s["loops"] for s in stats)
    emitted = sum(s["emitted"] for s in stats)
    accepted = sum(s["accepted"] for s in stats)
    hist = [sum(s["hist_emitted"][j] for s in stats) for j in range(K + 2)]
    ms_verify = sum(s["ms_verify"] for s in stats)
    ms_draft = sum(s["ms_draft"] for s in stats)
    ms_accept = sum(s["ms_accept"] for s in stats)
    peak, peak_src = measured_peaks()
    # algorithmic bytes: every weight of the model once per pass, plus the cached keys/values read
    ctx = P + n_new / 2.0
    vbytes = sps_synth.weight_bytes(c["target"]) + kv_bytes_per_token(c["target"]) * ctx
    dbytes = sps_synth.weight_bytes(c["draft"]) + kv_bytes_per_token(c["draft"]) * ctx
    v_gbs = vbytes * loops / (ms_verify / 1e3) / 1e9 if ms_verify > 0 else None
    d_gbs = dbytes * loops * K / (ms_draft / 1e3) / 1e9 if ms_draft > 0 and K > 0 else None
    n_lin_verify = 5 * c["target"]["n_layers"] + 1
    roofline = {"bound": "hbm", "kernel": ("lin_tc_kernel (tcgen05 weight-streaming linear layer)" if (c["target"]["dtype"] == 1 and K + 1 >= 5) else "lin_bf16_tma_kernel (weight-streaming linear layer)") + " averaged over the scoring pass",
                "achieved": v_gbs, "peak": peak, "unit": "GB/s", "frac": (v_gbs / peak) if v_gbs else None,
                "frac_of_8000_nominal": (v_gbs / 8000.0) if v_gbs else None, "peak_source": peak_src,
                "bytes_per_launch": vbytes / n_lin_verify, "avg_launch_us": 1e3 * ms_verify / loops / n_lin_verify if loops else None,
                # one ncu capture of this kernel on the 32000 x 8192 layer: dram read + write = 1.0088 x the algorithmic bytes of
                # that launch; traffic grows with the bytes of the matrix, so the ratio is applied to the average launch of a pass
                # (int8 weights: the capture of the 32768 x 8192 int8 layer gives 272.90 MB for 268.44 MB of weights, 1.0166 x)
                "traffic": args.traffic if args.traffic is not None else
                ({1: 1.0088, 2: 1.0166}.get(c["target"]["dtype"], 0) * vbytes / n_lin_verify or None)}
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": dec_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": {0: "f32", 1: "bf16", 2: "f16"}[c["target"]["dtype"]], "data": "synthetic",
            "config": {"workload": workload_name(cfgname, K, P, n_new), "l2": "weights streamed per pass exceed L2 by >1000x",
                       "parallelism": "replicas only" if world > 1 else "single GPU"},
            "clocks": clocks,
            "e2e": {"value": e2e, "unit": UNIT, "h2d_bytes_per_step": 4 * P + 24 + 16,
                    "d2h_bytes_per_step": int(loops / args.steps * 4 * (2 + K + 2))},
            "gpu_launches": sum(s["kernel_launches"] for s in stats),
            "roofline": roofline,
            "roofline_draft": {"bound": "hbm", "achieved": d_gbs, "peak": peak, "unit": "GB/s", "frac": (d_gbs / peak) if d_gbs else None},
            "loop": {"loops": loops, "tokens_per_loop": emitted / loops if loops else None,
                     "accept_rate": accepted / (loops * K) if loops and K else None, "hist_emitted": hist,
                     "ms_verify_per_loop": ms_verify / loops if loops else None,
                     "ms_draft_per_step": ms_draft / loops / K if loops and K else None,
                     "ms_accept_per_loop": ms_accept / loops if loops else None,
                     "ms_prefill": stats[-1]["ms_prefill"]},
            # the prompt pass: P - 1 rows through both models; bf16 models take it as tcgen05 GEMMs over 128-row chunks
            # (two bf16 halves per activation: 4 flops per weight and row), so the weights are read once per chunk
            "prefill": {"ms": stats[-1]["ms_prefill"], "rows": P - 1,
                        "tflops": (4.0 * (P - 1) * (sps_synth.weight_bytes(c["target"]) - c["target"]["vocab"] * c["target"]["d_model"] * 2
                                                   + sps_synth.weight_bytes(c["draft"]) - c["draft"]["vocab"] * c["draft"]["d_model"] * 2) / 2
                                   / (stats[-1]["ms_prefill"] / 1e3) / 1e12) if c["target"]["dtype"] == 1 and stats[-1]["ms_prefill"] > 0 else None}}
    # latency distribution over the timed loops: a loop delivers its tokens together, so a token's latency is its
    # loop's device time divided by the tokens that loop emitted (each token weighted once)
    lm, lt = np.concatenate(loop_ms), np.concatenate(loop_tok)
    per_tok = np.repeat(lm / lt, lt)
    pct = lambda a: {f"p{q}": float(np.percentile(a, q)) for q in (50, 90, 99)} | {"mean": float(a.mean()), "max": float(a.max())}
    line["latency"] = {"unit": "ms", "loop": pct(lm), "per_token": pct(per_tok), "loops": int(lm.size)}
    if rank == 0 and world == 1:
        # the same library's autoregressive decode on the same models
        ar_tps = None
        if args.ar_steps > 0:
            ar_stats = []
            gen(0, 0)
            for i in range(args.ar_steps):
                _, st, _ = gen(args.warmup + i, 0)
                ar_stats.append(st)
            ar_ms = sum(s["ms_decode"] for s in ar_stats)
            ar_tps = args.ar_steps * n_new / (ar_ms / 1e3)
            ar_gbs = sps_synth.weight_bytes(c["target"]) * args.ar_steps * n_new / (ar_ms / 1e3) / 1e9
            line["ar"] = {"value": ar_tps, "unit": UNIT, "ms_per_token": ar_ms / (args.ar_steps * n_new), "hbm_gbs": ar_gbs,
                          "frac": ar_gbs / peak}
            line["speedup_vs_ar"] = value / ar_tps
        if not args.no_cpu:
            line["cpu_baseline"] = cpu_baseline_full(h, c, wt, wd, K, emitted / loops if K > 0 else 1.0, dev)
    if rank == 0 and world == 1 and args.batch > 1 and c["target"]["dtype"] == 1:
        # the K / batch sweep's corner: `batch` sequences decoded together, batch x (K + 1) rows per scoring pass
        # (above 16 rows the linear layers run as tcgen05 GEMMs); aggregate tokens/s over the batch
        Bn = args.batch
        hb = sps.Handle(c["target"], wt, c["draft"], wd, max_seq=max_seq, max_batch=Bn, max_K=K, device=local)
        prompts = np.stack([sps_synth.make_prompt(1000 + b, P, V) for b in range(Bn)])
        hb.sps_generate_batch(prompts, n_new, K, T, 1)
        _, sb = hb.sps_generate_batch(prompts, n_new, K, T, 2)
        b_ms, b_loops = sb[0]["ms_decode"], max(s["loops"] for s in sb)
        line.setdefault("variants", {})[f"batch{Bn}_K{K}"] = {
            "value": Bn * n_new / (b_ms / 1e3), "unit": UNIT, "rows_per_pass": Bn * (K + 1), "loops": b_loops,
            "tokens_per_loop_per_sequence": sum(s["emitted"] for s in sb) / sum(s["loops"] for s in sb),
            "ms_verify_per_loop": sb[0]["ms_verify"] / b_loops, "ms_draft_per_step": sb[0]["ms_draft"] / (b_loops * max(K, 1)),
            "ms_prefill": sb[0]["ms_prefill"], "speedup_vs_batch1": Bn * n_new / (b_ms / 1e3) / value}
        hb.close()
    if rank == 0 and world == 1 and args.aligned_steps > 0 and c["target"]["dtype"] >= 1:
        # Same kernels, same shapes, but a pair whose draft agrees with its target about as often as the paper's
        # trained pair did: both bodies' output projections are damped in place (x gamma), so that the shared
        # (un)embedding dominates the logits.  A documented deviation from "all weights N(0, 0.02)", used only to
        # show tokens per loop in the paper's acceptance regime; kernel times do not depend on weight values.
        sfx = "_scale" if c["target"]["dtype"] == 2 else ""      # int8 matrices are damped through their row scales
        for w in (wt, wd):
            for lw in w["layers"]:
                lw["wo" + sfx].mul_(args.aligned_gamma)
                lw["w_down" + sfx].mul_(args.aligned_gamma)
        torch.cuda.synchronize()
        gen(0, K)
        al = [gen(args.warmup + i, K)[1] for i in range(args.aligned_steps)]
        al_ms = sum(s["ms_decode"] for s in al)
        al_loops = sum(s["loops"] for s in al)
        al_tps = args.aligned_steps * n_new / (al_ms / 1e3)
        line.setdefault("variants", {})
        line["variants"].update({"aligned": {"gamma": args.aligned_gamma, "value": al_tps, "unit": UNIT,
                                        "tokens_per_loop": sum(s["emitted"] for s in al) / al_loops,
                                        "accept_rate": sum(s["accepted"] for s in al) / (al_loops * K) if K else None,
                                        "speedup_vs_ar": al_tps / ar_tps if ar_tps else None}})
        # the decoding settings the paper's speed table uses, on the same pair: nucleus 0.8 and greedy
        # (top-k / nucleus / greedy filtering of both models ahead of the rejection scheme)
        for name, top_k, top_p, temp in (("aligned_nucleus_0.8", 0, 0.8, T), ("aligned_greedy", 0, 1.0, 0.0)):
            h.sps_set_sampling(top_k, top_p)
            gen(0, K, temp)
            fs = [gen(args.warmup + i, K, temp)[1] for i in range(args.aligned_steps)]
            f_ms, f_loops = sum(s["ms_decode"] for s in fs), sum(s["loops"] for s in fs)
            line["variants"][name] = {"value": args.aligned_steps * n_new / (f_ms / 1e3), "unit": UNIT,
                                      "tokens_per_loop": sum(s["emitted"] for s in fs) / f_loops,
                                      "accept_rate": sum(s["accepted"] for s in fs) / (f_loops * K) if K else None,
                                      "ms_draft_per_step": sum(s["ms_draft"] for s in fs) / (f_loops * max(K, 1)),
                                      "ms_accept_per_loop": sum(s["ms_accept"] for s in fs) / f_loops}
        h.sps_set_sampling(0, 1.0)
        # lookahead adapted from loop to loop between 1 and 6 (grow after a fully accepted loop, shrink after a
        # first-draft rejection)
        h.sps_generate_adaptive(sps_synth.make_prompt(seeds[0], P, V), n_new, 1, 6, T, seeds[0])
        ad = []
        for i in range(args.aligned_steps):
            ad.append(h.sps_generate_adaptive(sps_synth.make_prompt(seeds[args.warmup + i], P, V), n_new, 1, 6, T,
                                              seeds[args.warmup + i])[1])
        ad_ms, ad_loops = sum(s["ms_decode"] for s in ad), sum(s["loops"] for s in ad)
        line["variants"]["aligned_adaptive_K_1_6"] = {"value": args.aligned_steps * n_new / (ad_ms / 1e3), "unit": UNIT,
                                                      "tokens_per_loop": sum(s["emitted"] for s in ad) / ad_loops,
                                                      "mean_K": sum(s["draft_calls"] for s in ad) / ad_loops}
        # tokens per loop swept independently of the models: every draft accepted with a fixed probability (measurement
        # mode; the tokens follow no law, the kernels run as always)
        forced = []
        for alpha in (0.5, 0.7, 0.8, 0.9):
            h.sps_set_forced_acceptance(alpha)
            gen(0, K)
            st = gen(args.warmup, K)[1]
            forced.append({"alpha": alpha, "value": n_new / (st["ms_decode"] / 1e3), "tokens_per_loop": st["emitted"] / st["loops"],
                           "expected_tokens_per_loop": (1 - alpha ** (K + 1)) / (1 - alpha),
                           "speedup_vs_ar": n_new / (st["ms_decode"] / 1e3) / ar_tps if ar_tps else None})
        h.sps_set_forced_acceptance(0.0)
        line["variants"]["forced_acceptance"] = forced
        # lookahead sweep on the damped pair (the paper's K trade-off figure): one generation per K
        if args.k_sweep:
            # per K: `k_sweep_seeds` generations (different prompts and seeds); besides the rates, the time to n_new tokens
            # with its spread -- a longer lookahead makes the time per generation more variable (the K trade-off figure)
            sweep = []
            for k in (1, 2, 3, 4, 6, 8):
                gen(0, k)
                sts = [sps_generate_seeded(h, 3000 + j, k) for j in range(args.k_sweep_seeds)]
                t = np.array([s_["ms_decode"] for s_ in sts])
                loops_k = sum(s_["loops"] for s_ in sts)
                sweep.append({"K": k, "value": float(n_new * len(sts) / (t.sum() / 1e3)), "seeds": len(sts),
                              "tokens_per_loop": sum(s_["emitted"] for s_ in sts) / loops_k,
                              "accepted_per_loop": sum(s_["accepted"] for s_ in sts) / loops_k,
                              "ms_verify_per_loop": sum(s_["ms_verify"] for s_ in sts) / loops_k,
                              "ms_draft_per_step": sum(s_["ms_draft"] for s_ in sts) / (loops_k * k),
                              "time_to_n_new_ms": {"mean": float(t.mean()), "std": float(t.std()), "p90": float(np.percentile(t, 90)),
                                                   "min": float(t.min()), "max": float(t.max())}})
            line["variants"]["k_sweep"] = sweep
    h.close()
    if rank == 0 and world == 1 and args.mini_sweep and not args.sweep and c["target"]["dtype"] == 1 and cfgname.startswith("70b"):
        line["sweep_mini"] = mini_sweep(sps, c, wt, wd, local, peak)
    if rank == 0 and world == 1 and args.sweep and c["target"]["dtype"] == 1:
        line["sweep"] = sweep_bench(sps, c, wt, wd, local, peak)
        # the variants above damp both models' output projections in place, so that is the pair the sweep ran on
    if rank == 0 and world == 1 and ("sweep" in line or "sweep_mini" in line):
        line["sweep_models"] = "damped pair (acceptance in the paper's regime)" if args.aligned_steps > 0 else "random-init pair (natural acceptance)"
    if rank == 0 and world == 1 and args.mid_steps > 0 and cfgname != "mid":
        line.setdefault("variants", {})["mid"] = pair_variant(sps, "mid", local, peak, args.mid_steps)
    if rank == 0 and world == 1 and not args.no_sampler:
        line["sampler"] = sampler_bench(dev, peak)
    if rank == 0:
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def pair_variant(sps, cfgname, local, peak, steps):
    """Another pair of the workload table through the same calls (the mid-size bf16 pair: 24-layer d 2048 target,
    6-layer d 1024 draft, prompt 128, 256 new tokens, K = 4, batch 1): tokens/s of speculative and autoregressive
    decoding, the two passes' device times and their weight bytes over time against the measured HBM rate.  At this
    size a pass is ~120 launches of 8-33 MB each: what it shows is the fixed cost per layer, not the streaming rate."""
    dev = f"cuda:{local}"
    c, wt, wd = build_models(cfgname, dev)
    P, n_new, K, T, V = c["prompt_len"], c["n_new"], c["K"], c["T"], c["target"]["vocab"]
    h = sps.Handle(c["target"], wt, c["draft"], wd, max_seq=((P + n_new + K + 63) // 64) * 64, max_batch=1, max_K=K, device=local)

    def run(k, n):
        sts = []
        for i in range(n):
            sts.append(h.sps_generate(sps_synth.make_prompt(500 + i, P, V), n_new, k, T, 500 + i)[1])
        return sts
    run(K, 2); run(0, 1)
    st, ar = run(K, steps), run(0, max(1, steps // 2))
    h.close()
    loops = sum(x["loops"] for x in st)
    ms_dec, ms_v, ms_d = sum(x["ms_decode"] for x in st), sum(x["ms_verify"] for x in st), sum(x["ms_draft"] for x in st)
    tps = len(st) * n_new / (ms_dec / 1e3)
    ar_tps = len(ar) * n_new / (sum(x["ms_decode"] for x in ar) / 1e3)
    ctx = P + n_new / 2.0
    vb = sps_synth.weight_bytes(c["target"]) + kv_bytes_per_token(c["target"]) * ctx
    db = sps_synth.weight_bytes(c["draft"]) + kv_bytes_per_token(c["draft"]) * ctx
    v_gbs, d_gbs = vb * loops / (ms_v / 1e3) / 1e9, db * loops * K / (ms_d / 1e3) / 1e9
    return {"workload": workload_name(cfgname, K, P, n_new), "value": tps, "unit": UNIT, "ar": ar_tps, "speedup_vs_ar": tps / ar_tps,
            "tokens_per_loop": sum(x["emitted"] for x in st) / loops, "accept_rate": sum(x["accepted"] for x in st) / (loops * K),
            "ms_verify_per_loop": ms_v / loops, "ms_draft_per_step": ms_d / (loops * K), "ms_accept_per_loop": sum(x["ms_accept"] for x in st) / loops,
            "verify_gbs": v_gbs, "verify_frac": v_gbs / peak, "draft_gbs": d_gbs, "draft_frac": d_gbs / peak,
            "ar_frac": sps_synth.weight_bytes(c["target"]) * ar_tps / 1e9 / peak, "kernel_launches_per_loop": sum(x["kernel_launches"] for x in st) / loops}


def mini_sweep(sps, c, wt, wd, local, peak):
    """A compact cut of the K x batch sweep for the default line (the full one, `--sweep`, takes minutes): prompt 512,
    64 new tokens, temperature 1, K in {1, 2, 4, 8} at batch 1 and 8, against autoregressive decoding at that batch;
    per cell tokens/s over the batch, accepted drafts per target call and the scoring pass's time."""
    P, n_new, V, T = 512, 64, c["target"]["vocab"], 1.0
    out = []
    for Bn in (1, 8):
        hs = sps.Handle(c["target"], wt, c["draft"], wd, max_seq=((P + n_new + 8 + 63) // 64) * 64, max_batch=Bn, max_K=8, device=local)
        prompts = np.stack([sps_synth.make_prompt(2000 + b, P, V) for b in range(Bn)])
        ar = None
        for K in (0, 1, 2, 4, 8):
            hs.sps_generate_batch(prompts[:, :32], 8, K, T, 1)      # first use of (K, batch): eager run, then graph capture
            _, st = hs.sps_generate_batch(prompts, n_new, K, T, 7)
            ms, loops = st[0]["ms_decode"], max(s["loops"] for s in st)
            tps = Bn * n_new / (ms / 1e3)
            if K == 0:
                ar = tps
                continue
            ms_v = st[0]["ms_verify"] / loops
            out.append({"batch": Bn, "K": K, "value": tps, "ar": ar, "vs_ar": tps / ar,
                        "accepted_per_call": sum(s["accepted"] for s in st) / sum(s["loops"] for s in st),
                        "ms_verify": ms_v, "verify_frac": sps_synth.weight_bytes(c["target"]) / (ms_v / 1e3) / 1e9 / peak,
                        "ms_draft_per_step": st[0]["ms_draft"] / (loops * K)})
        hs.close()
    return out


def sweep_bench(sps, c, wt, wd, local, peak):
    """The K / batch sweep on the pair at its natural acceptance: K in {1, 2, 3, 4, 6, 8} x temperature {0.5, 1} x batch
    {1, 4, 8}, prompt 512, 256 new tokens; tokens/s over the batch, accepted drafts per target call, scoring-pass
    latency and its weight bytes over time, against the same library's autoregressive decode at that batch."""
    P, n_new, V = 512, 256, c["target"]["vocab"]
    out = []
    for Bn in (1, 4, 8):
        hs = sps.Handle(c["target"], wt, c["draft"], wd, max_seq=((P + n_new + 8 + 63) // 64) * 64, max_batch=Bn, max_K=8, device=local)
        prompts = np.stack([sps_synth.make_prompt(2000 + b, P, V) for b in range(Bn)])
        ar = {}
        for T in (0.5, 1.0):
            for K in (0, 1, 2, 3, 4, 6, 8):
                hs.sps_generate_batch(prompts[:, :32], 8, K, T, 1)      # first use of (K, batch): eager run, then graph capture
                _, st = hs.sps_generate_batch(prompts, n_new, K, T, 7)
                ms, loops = st[0]["ms_decode"], max(s["loops"] for s in st)
                tps = Bn * n_new / (ms / 1e3)
                if K == 0:
                    ar[T] = tps
                    continue
                ms_v = st[0]["ms_verify"] / loops
                out.append({"batch": Bn, "T": T, "K": K, "value": tps, "vs_ar": tps / ar[T],
                            "accepted_per_call": sum(s["accepted"] for s in st) / sum(s["loops"] for s in st),
                            "ms_verify": ms_v, "verify_gbs": sps_synth.weight_bytes(c["target"]) / (ms_v / 1e3) / 1e9,
                            "verify_frac": sps_synth.weight_bytes(c["target"]) / (ms_v / 1e3) / 1e9 / peak,
                            "ms_draft_per_step": st[0]["ms_draft"] / (loops * K), "ar": ar[T]})
        hs.close()
    return out


def sampler_bench(dev, peak_gbs):
    """The fused accept / resample / extra-token kernel alone (vocab 32000, K = 4, target logits N(0, 9), draft =
    target + N(0, 1)): device time per launch against the time its reads take at the measured HBM rate.  The bound used
    is the bytes the standalone call must read, V * (2K + 1) * 4 per sequence (K + 1 target rows, K draft rows: 1.15 MB
    at K = 4); the workload table's V * (K + 1) * 8 (1.28 MB) counts a draft row for the extra position too, which does
    not exist -- `bound_us_table` gives the time for that figure.  One CTA per sequence: at batch 1 the kernel is a latency chain on one SM, not a
    bandwidth problem, and its 1.15 MB of logits were just written by the two models (L2-resident, as here)."""
    import torch
    import paper_2302_01318_b200 as sps
    out = []
    K, V = 4, 32000
    for B in (1, 8, 64):
        ncopy = max(2, int(160e6 // (B * (2 * K + 1) * V * 4)) + 1) if B >= 8 else 2   # B >= 8: rotate past the L2
        bufs = []
        for i in range(ncopy):
            q, p, d = sps_synth.sampler_batch(B, K, V, seed=i, sigma=1.0)
            bufs.append([torch.from_numpy(x).to(dev) for x in (q, p, d)])
        na = torch.zeros(B, dtype=torch.int32, device=dev)
        tk = torch.zeros((B, K + 1), dtype=torch.int32, device=dev)
        fl = torch.zeros(B, dtype=torch.int32, device=dev)
        def run(i):
            q, p, d = bufs[i % ncopy]
            sps.sps_accept(q, p, d, 1.0, 7, i, na, tk, fl)
        for i in range(5):
            run(i)
        torch.cuda.synchronize()
        # the launches are replayed from a CUDA graph: a host that calls through Python cannot enqueue kernels of ~10 us
        # as fast as the GPU finishes them, and the figure wanted here is the kernel's, not the interpreter's
        n = 40
        side = torch.cuda.Stream()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                for i in range(n):
                    run(5 + i)
            g.replay()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            g.replay()
            e1.record()
            torch.cuda.synchronize()
        us = e0.elapsed_time(e1) * 1e3 / n
        nbytes = B * (2 * K + 1) * V * 4
        bound_us = nbytes / (peak_gbs * 1e9) * 1e6
        out.append({"B": B, "K": K, "V": V, "us": us, "read_bytes": nbytes, "bound_us": bound_us, "frac": bound_us / us,
                    "bound_us_table": B * (K + 1) * V * 8 / (peak_gbs * 1e9) * 1e6,
                    "mean_accepted": float(na.float().mean().item())})
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="70b", choices=list(sps_synth.CONFIGS))
    ap.add_argument("--K", type=int, default=4)
    ap.add_argument("--ar-steps", type=int, default=2)
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--aligned-steps", type=int, default=2)
    ap.add_argument("--aligned-gamma", type=float, default=1e-4)
    ap.add_argument("--batch", type=int, default=8, help="also decode this many sequences together (0 / 1 = skip)")
    ap.add_argument("--sweep", action="store_true", help="also run the K x temperature x batch sweep (prompt 512, 256 tokens; minutes)")
    ap.add_argument("--no-mini-sweep", dest="mini_sweep", action="store_false",
                    help="skip the compact K x batch sweep of the default line (prompt 512, 64 tokens, K in {1,2,4,8}, batch 1 and 8)")
    ap.add_argument("--k-sweep-seeds", type=int, default=8, help="generations per K in --k-sweep")
    ap.add_argument("--k-sweep", action="store_true", help="also run the damped pair at K = 1, 2, 3, 4, 6, 8")
    ap.add_argument("--no-sampler", action="store_true", help="skip the standalone accept-kernel timings")
    ap.add_argument("--mid-steps", type=int, default=3, help="generations of the mid-size pair reported under variants.mid (0 = skip)")
    ap.add_argument("--traffic", type=float, default=None,
                    help="ncu dram bytes per launch of the dominant kernel; default: bytes_per_launch x the ratio measured in profiles/")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
