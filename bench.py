"""Benchmark of the FAAR layer step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 2|3|4] [--impl ours|reference]

--config 2 (default): one job = the whole hot path for one linear layer of the down_proj-shaped workload
(W 2048x8192 BF16, calibration batch X 4096x8192 BF16): soft-quantisation set-up, K optimisation steps
(soft weights -> forward GEMM + MSE -> dW GEMM + dV + Round Loss + Adam update, beta annealed geometrically
over the K steps), then harden + pack.  `value` = K / (device time of that job), so the once-per-layer
kernels are inside the timed region.  With N > 1 every rank runs its own layer (layers are independent
problems: no data-path collective), value = N*K / max-over-ranks time.

--config 3 / 4: the seven linears of a Llama-3.2-1B- / Qwen3-1.7B-shaped decoder block, each optimised for K
steps on 4096-row minibatches of a synthetic calibration set (Stage-1 driver of the package); `value` =
K / (summed device time of the seven jobs) = block steps per second, with one line per linear under
`linears` (soft weights / forward / backward microseconds, TFLOP/s, fraction of the BF16 peak).

`--impl reference` times the CPU oracle (numpy, float64) on the host cores instead; each of its
steps is a row-sample of the same layer (the loss separates over output rows, so a sample of rows is
an exact sub-problem) and the rate is scaled by rows/sample.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

O, K, T = 2048, 8192, 4096
WORKLOAD = "Llama-3.2-1B-shaped down_proj: W 2048x8192 bf16 (0.02*N(0,1), 0.1% x10), X 4096x8192 bf16 " \
           "(Student-t(4), 16 channels x20), Adam lr 1e-2, beta 4->32 geometric"
BLOCK_WORKLOADS = {
    3: "Llama-3.2-1B-shaped decoder block, Stage 1 layer-wise: q/o 2048x2048, k/v 512x2048, gate/up 8192x2048, "
       "down 2048x8192, W bf16 0.02*N(0,1); calibration hidden states N(0,1) + 8 channels x30, RMS-normalised, "
       "4096-row minibatches; Adam lr 1e-2, beta 4->32 geometric",
    4: "Qwen3-1.7B-shaped decoder block, Stage 1 layer-wise: q/o 2048x2048, k/v 1024x2048, gate/up 6144x2048, "
       "down 2048x6144, W bf16 0.02*N(0,1); calibration hidden states N(0,1) + 8 channels x30, RMS-normalised, "
       "4096-row minibatches; Adam lr 1e-2, beta 4->32 geometric",
}
STAGE2_MODEL = dict(vocab=128256, hidden=2048, n_layers=16, n_heads=32, n_kv_heads=8, head_dim=64, ffn=8192)
STAGE2_BATCH, STAGE2_SEQ = 4, 2048
STAGE2_WORKLOAD = "Stage-2 full-model alignment step (Eq. 6) on a 16-layer Llama-3.2-1B-shaped model (hidden 2048, 32 heads / " \
                  "8 KV heads, head_dim 64, MLP 8192, vocab 128256, random-init bf16 0.02*N(0,1)), all 112 linears " \
                  "soft-quantised with their own V, batch 4 x 2048 token ids uniform over the vocabulary, loss = KL(logits) + " \
                  "MSE(last hidden state) + Round Loss, Adam lr 5e-4"
METRIC, UNIT = "faar_layer_steps_per_s", "steps/s"


def stage2_flops(m=STAGE2_MODEL, batch=STAGE2_BATCH, seq=STAGE2_SEQ):
    """Algorithmic flop of one alignment step (no recomputation counted): per quantised linear the frozen forward,
    the quantised forward, the input gradient and the dW GEMM (8 T O K); the LM head twice forward and once
    backward; causal attention forward in both models (2 products) and backward (4 products)."""
    T = batch * seq
    q, kv = m["n_heads"] * m["head_dim"], m["n_kv_heads"] * m["head_dim"]
    p_lin = m["n_layers"] * (2 * q * m["hidden"] + 2 * kv * m["hidden"] + 3 * m["ffn"] * m["hidden"])
    att_unit = 2.0 * batch * m["n_heads"] * seq * seq * m["head_dim"] / 2.0
    return 8.0 * T * p_lin + 3.0 * 2.0 * T * m["vocab"] * m["hidden"] + m["n_layers"] * 8.0 * att_unit
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
NOMINAL_BF16_TFLOPS = 2250.0

# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the GEMM kernels on the config-2
# layer, from one ncu capture each, with the SHA-256 (first 12 hex digits) of the kernel source at the time of
# the capture.  A kernel source that has changed since makes the figure stale: `traffic` is then null.
NCU_TRAFFIC = {
    "gemm_bwd": {"bytes": 458.2e6, "source_sha": "4f6f41dfef24"},
    "gemm_fwd": {"bytes": 156.3e6, "source_sha": "4f6f41dfef24"},
}
GEMM_SOURCE = os.path.join(ROOT, "paper_2603_22370_b200", "csrc", "faar_gemm.cu")


def ncu_traffic(kernel):
    """The recorded DRAM traffic of `kernel`, or None when the kernel source is no longer the captured one."""
    rec = NCU_TRAFFIC.get(kernel)
    if not rec or not os.path.exists(GEMM_SOURCE):
        return None
    with open(GEMM_SOURCE, "rb") as f:
        sha = hashlib.sha256(f.read()).hexdigest()[:12]
    return rec["bytes"] if sha == rec["source_sha"] else None


def tensor_fracs(tflops, pk):
    """Achieved BF16 rate against the three denominators: the measured burst rate (a kernel timed in a job
    short enough to stay at boost clocks), the measured sustained rate (a seconds-long job under the power
    cap) and the nominal dense peak."""
    return {"frac_burst": round(tflops / pk["bf16_tflops"], 4),
            "frac_sustained": round(tflops / pk["bf16_tflops_sustained"], 4),
            "frac_nominal": round(tflops / NOMINAL_BF16_TFLOPS, 4)}


def applicable_peak(job_ms, clocks):
    """Which measured BF16 peak a kernel timed inside this job is held against: the sustained one if the job
    ran for seconds or the clock record shows the power cap at work, else the burst one."""
    capped = bool(clocks) and "sw_power_cap" in (clocks.get("reasons") or [])
    if job_ms >= 1000.0 or capped:
        return "bf16_tflops_sustained", "frac_sustained", \
               "sustained (job of %.0f ms%s)" % (job_ms, ", sw_power_cap seen" if capped else "")
    return "bf16_tflops", "frac_burst", "burst (job of %.1f ms, no power cap in the clock record)" % job_ms


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {k: float(p[k]) for k in FALLBACK_PEAKS if k in p}, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def beta_at(t, steps, b0=4.0, b1=32.0):
    return b0 if steps <= 1 else b0 * (b1 / b0) ** (t / (steps - 1))


def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


# ------------------------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = "timestamp,index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active," \
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown," \
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap"

    def __init__(self, gpu_index: int):
        self.lines, self.windows, self.proc = [], [], None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(gpu_index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def window(self, t0, t1):
        self.windows.append((t0, t1))

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.1)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, smax, reasons, power = [], None, set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ts, line in self.lines:
            if not any(a - 0.05 <= ts <= b + 0.05 for a, b in self.windows):
                continue
            f = [x.strip() for x in line.split(",")]
            if len(f) < 10:
                continue
            try:
                sm.append(float(f[2]))
                smax = float(f[3])
                power.append(float(f[4]))
            except ValueError:
                continue
            for name, val in zip(names, f[6:10]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": smax, "reasons": sorted(reasons),
                "samples": len(sm), "power_w_max": max(power) if power else None}


# ------------------------------------------------------------------------------------------------
# the CPU oracle, timed (cpu_baseline leg and --impl reference)
# ------------------------------------------------------------------------------------------------
def oracle_rate(rows: int, steps: int, warmup: int, seed: int = 0, tokens: int = T, layer=(O, K, T), block_index=None):
    """Runs `warmup + steps` oracle steps on a sample of a layer (`rows` output rows, `tokens` tokens);
    returns (full-layer steps/s, seconds per sampled step, threads used).  A row sample is an exact
    sub-problem (the loss separates over rows); a token sample is a smaller calibration batch; the rate
    is scaled by the work ratio (O/rows) * (T/tokens).  layer = (O, K, T) of the full layer; block_index
    selects the decoder-block input recipe instead of the down_proj one."""
    import numpy as np

    from oracle import faar_oracle as fo
    from paper_2603_22370_b200 import inputs
    Of, Kf, Tf = layer
    if block_index is None:
        W, X = inputs.config2(seed, rows, Kf, tokens)
    else:
        W, X = inputs.block_linear(seed, block_index, rows, Kf, tokens)
    # the calibration batch is handed over in float64 once, so that a step's cost is the method's own
    # arithmetic on the sampled rows and scales with them
    X = X.astype(np.float64)
    Yref = inputs.to_bf16_f32(fo.layer_ref(X, W)).astype(np.float64)
    scales, sg, code, V = fo.softquant_init(W)
    m, u = np.zeros_like(V), np.zeros_like(V)
    total = warmup + steps
    t0 = None
    for i in range(total):
        if i == warmup:
            t0 = time.perf_counter()
        hp = fo.HParams(beta=beta_at(max(i - warmup, 0), steps), step=i + 1, lr=1e-2)
        V, m, u, _, _, _ = fo.layer_step(X, Yref, V, code, scales, sg, m, u, hp, "bf16")
    dt = (time.perf_counter() - t0) / steps
    fo.harden_pack(V, code, scales, sg)
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        threads = len(os.sched_getaffinity(0))
    return 1.0 / (dt * (Of / rows) * (Tf / tokens)), dt, threads


def block_linears(config: int):
    from paper_2603_22370_b200 import inputs
    return inputs.LLAMA32_1B_BLOCK if config == 3 else inputs.QWEN3_1P7B_BLOCK


def oracle_block_rate(config: int, rows: int, steps: int, warmup: int, tokens: int = T):
    """Block steps/s of the oracle: one sampled linear (k_proj's shape: K = 2048) timed, the block's seven
    linears scaled from it by their flop counts (4 T O K each).  Returns (rate, seconds per sampled step,
    threads, description of the sample)."""
    lin = block_linears(config)
    name, Ok, Kk = lin[1]
    rate_k, dt, threads = oracle_rate(min(rows, Ok), steps, warmup, tokens=tokens, layer=(Ok, Kk, T), block_index=1)
    flops_k = 4.0 * T * Ok * Kk
    flops_block = sum(4.0 * T * o * k for _, o, k in lin)
    sample = f"each step = {min(rows, Ok)} of {Ok} output rows of the {name} shape ({Ok}x{Kk}) on {tokens} of {T} tokens; " \
             f"scaled to the layer by rows and tokens, then to the block's seven linears by flop count (x{flops_block / flops_k:.1f})"
    return rate_k * flops_k / flops_block, dt, threads, sample


def run_reference(args):
    rank, _, world = dist_env()
    if rank != 0:
        return 0
    # size the sample (rows x tokens) so that warmup + steps finish in about two minutes
    budget = 120.0 / (args.steps + args.warmup)
    rows, tokens = 256, T
    block = args.config in (3, 4)

    def probe(r, tk, st, wu):
        if block:
            return oracle_block_rate(args.config, r, st, wu, tokens=tk)
        rate, dt, th = oracle_rate(r, st, wu, tokens=tk)
        return rate, dt, th, f"each step = {r} of {O} output rows (exact sub-problem: the loss separates over rows) on " \
                             f"{tk} of {T} tokens, K={K}; rate scaled by the work ratio {O}/{r} x {T}/{tk}"

    if args.config == 5:
        # each step of the run = the bounded sample of one alignment step (see oracle_stage2_rate)
        n = max(1, min(args.steps, 3))
        res = [oracle_stage2_rate() for _ in range(n)]
        rate, threads, sample = sum(r[0] for r in res) / n, res[0][2], res[0][3]
        line = {"impl": "reference", "metric": METRIC, "value": rate, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": 1e3 / rate, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": workload_config(5),
                "cpu_baseline": {"value": rate, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
                "e2e": {"value": rate, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}, "gpu_launches": 0}
        print(json.dumps(line))
        return 0
    while True:
        _, dt_probe, _, _ = probe(rows, tokens, 1, 1)
        if dt_probe <= budget or (rows <= 16 and tokens <= 128):
            break
        if rows > 16:
            rows //= 2
        else:
            tokens //= 2
    rate, dt, threads, sample = probe(rows, tokens, args.steps, args.warmup)
    line = {"impl": "reference", "metric": METRIC, "value": rate, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 / rate, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(args.config),
            "cpu_baseline": {"value": rate, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": rate, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))
    return 0


def workload_config(config: int):
    """The `config` object both arms print: the workload and its sizes, nothing else."""
    l2 = "no flush: one step touches about 410 MB (X, X^T, V, m, u, W_soft, Y_ref, dY^T, codes), more than the 126 MB L2"
    if config == 5:
        return {"workload": STAGE2_WORKLOAD, "batch": STAGE2_BATCH, "seq_len": STAGE2_SEQ, **STAGE2_MODEL,
                "l2": "no flush: one step touches tens of GB (weights, V and Adam moments of 973 M parameters, activations)",
                "timed_region": "K x (frozen forward, quantised forward, loss, backward with the update of all 112 V); "
                                "weights, V, Adam moments and the token batch resident in HBM"}
    if config == 2:
        return {"workload": WORKLOAD, "O": O, "K": K, "T": T, "l2": l2,
                "timed_region": "softquant_init + K x layer_step + harden_pack, inputs resident in HBM"}
    return {"workload": BLOCK_WORKLOADS[config], "T": T,
            "linears": {name: [o, k] for name, o, k in block_linears(config)},
            "l2": "no flush: every step takes the next 4096-row minibatch of a calibration set larger than the 126 MB L2 "
                  "(the k/v/q/o linears' per-step state alone is below it and is re-read from L2, as it would be in use)",
            "timed_region": "per linear: softquant_init + K x layer_step (minibatches round-robin) + harden_pack; "
                            "calibration set, its transposes and the frozen targets resident in HBM"}


# ------------------------------------------------------------------------------------------------
# our arm
# ------------------------------------------------------------------------------------------------
class Runtime:
    """Process-wide set-up shared by the layer and the block benchmark: one rank per GPU, the library built
    and loaded, a context on its own stream, the clock sampler, and the timing rule (barrier + synchronise on
    both sides, CUDA events on the launching stream, max over ranks)."""

    def __init__(self, args):
        import torch

        from paper_2603_22370_b200 import build as faar_build
        from paper_2603_22370_b200 import faar
        self.torch, self.faar = torch, faar
        self.rank, self.local_rank, self.world = dist_env()
        self.dist = None
        if self.world > 1:
            import torch.distributed as dist
            self.dist = dist
            torch.cuda.set_device(self.local_rank)
            dist.init_process_group("nccl", device_id=torch.device(f"cuda:{self.local_rank}"))
        self.dev = self.local_rank if self.world > 1 else 0
        torch.cuda.set_device(self.dev)
        self.device = f"cuda:{self.dev}"
        if self.rank == 0:
            faar_build.build()
        if self.world > 1:
            self.dist.barrier()
        faar.lib()                                     # raises if libfaar.so is missing: no fallback
        self.stream = torch.cuda.Stream(device=self.device)
        self.ctx = faar.Context(self.dev, self.stream)
        self.sampler = ClockSampler(self.dev) if self.rank == 0 else None

    def barrier(self):
        self.torch.cuda.synchronize()
        if self.world > 1:
            self.dist.barrier()
            self.torch.cuda.synchronize()

    def timed(self, fn):
        """device time (ms) of fn() on the stream, max over ranks, with a barrier + sync on both sides"""
        from paper_2603_22370_b200 import shard
        torch = self.torch
        self.barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        w0 = time.time()
        with torch.cuda.stream(self.stream):
            e0.record(self.stream)
            fn()
            e1.record(self.stream)
        self.stream.synchronize()
        self.barrier()
        w1 = time.time()
        _, ms = shard.job_rate(1.0, e0.elapsed_time(e1), self.device)     # max over ranks
        if self.sampler:
            self.sampler.window(w0, w1)
        return ms

    def finish(self):
        if self.world > 1:
            self.dist.destroy_process_group()


def run_block(args, rt):
    """--config 3 / 4: the seven linears of one decoder block through the package's Stage-1 driver."""
    import numpy as np

    from paper_2603_22370_b200 import inputs, stage1
    torch, faar, ctx, stream, device = rt.torch, rt.faar, rt.ctx, rt.stream, rt.device
    steps, warmup = args.steps, max(args.warmup, 3)
    lin = block_linears(args.config)
    n_tok = args.calib_tokens
    hid = 2048
    ffn = dict((n, o) for n, o, k in lin)["gate_proj"]
    rng_seed = 100 + rt.rank                                        # each rank its own block

    # ---- synthetic block: weights, hidden states (input of q, k, v, gate, up), o_proj's input
    with torch.cuda.stream(stream):
        Wd = {}
        for i, (name, o, k) in enumerate(lin):
            Wn, _ = inputs.block_linear(rng_seed, i, o, k, 8)
            Wd[name] = torch.from_numpy(Wn).to(device).to(torch.bfloat16)
        streams = inputs._streams(rng_seed + 1000, 2)
        H = torch.from_numpy(inputs.to_bf16_f32(inputs.hidden_states(streams[0], n_tok, hid))).to(device).to(torch.bfloat16)
        Ho = torch.from_numpy(inputs.to_bf16_f32(inputs.hidden_states(streams[1], n_tok, hid, rms_norm=False))).to(device).to(torch.bfloat16)
        A = stage1.mlp_activation(ctx, Wd["gate_proj"], Wd["up_proj"], H, T)
    stream.synchronize()
    Xin = {name: (A if name == "down_proj" else (Ho if name == "o_proj" else H)) for name, _, _ in lin}

    per_linear, total_ms, launches = {}, 0.0, 0
    e2e_ms, e2e_steps = 0.0, min(steps, 100)
    h2d_total = 0
    for name, o, k in lin:
        with torch.cuda.stream(stream):
            lay = stage1.StreamedLayer(ctx, Wd[name], Xin[name], T)

        def job(n):
            faar.softquant_init(ctx, lay.shape, lay.W, 0.0, lay.scales, lay.s_global, lay.code, lay.V, lay.ws)
            lay.m.zero_()
            lay.u.zero_()
            for t in range(n):
                lay.step(t, n, chain=args.chain)
            packed = torch.empty((o, k // 2), dtype=torch.uint8, device=device)
            faar.harden_pack(ctx, lay.shape, lay.V, lay.code, lay.scales, lay.s_global, packed, None, None, None)

        with torch.cuda.stream(stream):
            job(warmup)
        stream.synchronize()
        ms = rt.timed(lambda: job(steps))
        faar.check_status(ctx, lay.ws)

        def profiled():
            faar.profile_begin(ctx)
            job(steps)

        rt.timed(profiled)
        prof = faar.profile_end(ctx)
        bn, pairs = faar.last_gemm_config(ctx)
        us = {kname: 1e3 * v[1] / v[0] for kname, v in prof.items()}
        flops = 2.0 * T * o * k
        per_linear[name] = {"O": o, "K": k, "ms_per_step": round(ms / steps, 5),
                            "step_tflops": round(2 * flops * steps / (ms * 1e-3) / 1e12, 1),
                            "kernels_us": {kn: round(v, 2) for kn, v in us.items()},
                            "gemm_fwd_tflops": round(flops / (us["gemm_fwd"] * 1e-6) / 1e12, 1),
                            "gemm_bwd_tflops": round(flops / (us["gemm_bwd"] * 1e-6) / 1e12, 1),
                            "bwd_tile_n": bn, "bwd_cta_pairs": pairs, "job_ms": ms, "final_loss": lay.loss.tolist()}
        total_ms += ms
        launches += 2 + (1 + 2 * steps if args.chain else 3 * steps) + 1

        # end to end for this linear: every step's minibatch arrives from pinned host memory
        if not args.quick:
            Xh = lay.X[0].cpu().pin_memory()
            loss_h = torch.zeros(2, dtype=torch.float32).pin_memory()
            sets = [(torch.empty_like(lay.X[0]), torch.empty_like(lay.Xt[0]), torch.empty_like(lay.Yref[0])) for _ in range(2)]

            def e2e_job(n):
                faar.softquant_init(ctx, lay.shape, lay.W, 0.0, lay.scales, lay.s_global, lay.code, lay.V, lay.ws)
                lay.m.zero_()
                lay.u.zero_()
                for t in range(n):
                    hp = faar.make_hparams(beta=beta_at(t, n), step=t + 1)
                    Xd, Xtd, Yd = sets[t & 1]
                    faar.layer_step_host(ctx, lay.shape, hp, Xh, None, lay.W, Xd, Xtd, Yd, lay.V, lay.code, lay.scales,
                                         lay.s_global, lay.m, lay.u, lay.loss, loss_h, lay.ws)

            with torch.cuda.stream(stream):
                e2e_job(3)
            stream.synchronize()
            e2e_ms += rt.timed(lambda: e2e_job(e2e_steps))
            h2d_total += T * k * 2
            faar.check_status(ctx, lay.ws)
        del lay
        torch.cuda.empty_cache()

    clocks = rt.sampler.stop() if rt.sampler else None
    if rt.rank != 0:
        rt.finish()
        return 0
    pk, pk_kind = peaks()
    longest = max(v["job_ms"] for v in per_linear.values())
    peak_key, frac_key, peak_why = applicable_peak(longest, clocks)
    for v in per_linear.values():
        for g in ("gemm_fwd", "gemm_bwd"):
            v[g + "_frac"] = tensor_fracs(v[g + "_tflops"], pk)
        v["step_frac"] = tensor_fracs(v["step_tflops"], pk)
    value = rt.world * steps / (total_ms * 1e-3)
    block_flops = sum(4.0 * T * o * k for _, o, k in lin)
    # dominant kernel over the block: the launches of one GEMM kind that take the most time in a block step
    tot = {g: sum(v["kernels_us"][g] for v in per_linear.values()) for g in ("gemm_fwd", "gemm_bwd")}
    dominant = max(tot, key=tot.get)
    dom_tf = (block_flops / 2.0) / (tot[dominant] * 1e-6) / 1e12
    roofline = {"kernel": dominant + " (the seven linears' launches of one block step together)", "bound": "tensor",
                "achieved": round(dom_tf, 1), "peak": pk[peak_key], "unit": "TFLOP/s",
                "frac": tensor_fracs(dom_tf, pk)[frac_key], **tensor_fracs(dom_tf, pk), "traffic": None,
                "peak_source": f"{pk_kind} {peak_key}: {peak_why}",
                "timed": "per-kernel CUDA events on the launching stream, second pass of each linear's K-step job"}
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": steps, "warmup": warmup,
            "ms_per_step": total_ms / steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic", "config": workload_config(args.config),
            "calibration_tokens": n_tok, "chained_soft_weights": bool(args.chain), "clocks": clocks,
            "gpu_launches": launches, "roofline": roofline,
            "block_step_tflops": round(block_flops * steps / (total_ms * 1e-3) / 1e12, 1),
            "block_step_frac": tensor_fracs(block_flops * steps / (total_ms * 1e-3) / 1e12, pk),
            "linears": per_linear}
    if not args.quick:
        line["e2e"] = {"value": rt.world * e2e_steps / (e2e_ms * 1e-3), "unit": UNIT, "steps": e2e_steps,
                       "h2d_bytes_per_step": h2d_total, "d2h_bytes_per_step": 8 * len(lin),
                       "path": "faar_layer_step_host per linear: the minibatch copied in from pinned memory on a copy stream, "
                               "X^T and the frozen target rebuilt on the device, step, losses copied out"}
        cpu_rate, cpu_dt, cpu_threads, sample = oracle_block_rate(args.config, 128, 4, 1)
        line["cpu_baseline"] = {"value": cpu_rate, "unit": UNIT, "cores": cpu_threads, "kind": "oracle", "sample": sample}
    print(json.dumps(line))
    rt.finish()
    return 0


def oracle_stage2_rate(seq=128, warm=0):
    """Steps/s of the Stage-2 oracle (numpy, float64) for the full workload, from ONE alignment step on a bounded
    sample -- one decoder block of the sixteen, one sequence of `seq` tokens, the full vocabulary -- scaled by the
    algorithmic flop count.  Returns (rate, seconds of the sampled step, threads, description)."""
    import numpy as np

    from oracle import faar_oracle as fo
    from oracle import stage2_oracle as so
    from paper_2603_22370_b200 import inputs
    m = dict(STAGE2_MODEL, n_layers=1)
    cfg = so.ModelCfg(**m)
    rng = np.random.default_rng(0)
    params = {"embed": 0.02 * rng.standard_normal((cfg.vocab, cfg.hidden), dtype=np.float32),
              "lm_head": 0.02 * rng.standard_normal((cfg.vocab, cfg.hidden), dtype=np.float32),
              "final_norm": np.ones(cfg.hidden), "attn_norm.0": np.ones(cfg.hidden), "mlp_norm.0": np.ones(cfg.hidden)}
    W_fp, state = [{}], [{}]
    for name, (o, k) in cfg.linear_shapes().items():
        W = inputs.to_bf16_f32(inputs.weights(rng, o, k, 0.02))
        scales, sg, code, V = fo.softquant_init(W)
        W_fp[0][name], state[0][name] = W, (V, code, scales, sg)
    tokens = rng.integers(0, cfg.vocab, (1, seq))
    t0 = time.perf_counter()
    so.stage2_loss_and_grads(cfg, params, W_fp, state, tokens, beta=4.0)
    dt = time.perf_counter() - t0
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        threads = len(os.sched_getaffinity(0))
    ratio = stage2_flops() / stage2_flops(m, 1, seq)
    sample = f"one alignment step of the oracle on 1 of 16 decoder blocks and 1 x {seq} of {STAGE2_BATCH} x {STAGE2_SEQ} tokens " \
             f"(full vocabulary); time scaled by the flop ratio x{ratio:.0f}"
    return 1.0 / (dt * ratio), dt, threads, sample


def run_stage2(args, rt):
    """--config 5: full-model alignment steps through the package's Stage-2 driver."""
    from paper_2603_22370_b200 import stage2
    torch, faar, ctx, stream, device = rt.torch, rt.faar, rt.ctx, rt.stream, rt.device
    steps, warmup = args.steps, max(args.warmup, 3)
    m = dict(STAGE2_MODEL)
    if args.layers:
        m["n_layers"] = args.layers
    cfg = stage2.ModelConfig(**m)
    B, S = STAGE2_BATCH, STAGE2_SEQ
    gen = torch.Generator(device=device).manual_seed(1234 + rt.rank)

    def normal(*shape, sigma=0.02):
        return (sigma * torch.randn(shape, device=device, generator=gen, dtype=torch.float32)).to(torch.bfloat16)

    with torch.cuda.stream(stream):
        params = {"embed": normal(cfg.vocab, cfg.hidden, sigma=1.0), "lm_head": normal(cfg.vocab, cfg.hidden),
                  "final_norm": torch.ones(cfg.hidden, dtype=torch.float32, device=device)}
        weights = []
        for l in range(cfg.n_layers):
            params[f"attn_norm.{l}"] = torch.ones(cfg.hidden, dtype=torch.float32, device=device)
            params[f"mlp_norm.{l}"] = torch.ones(cfg.hidden, dtype=torch.float32, device=device)
            weights.append({n: normal(o, k) for n, (o, k) in cfg.linear_shapes().items()})
        model = stage2.Stage2Model(ctx, cfg, params, weights, B, S)
        tok_h = torch.randint(0, cfg.vocab, (B * S,), dtype=torch.int32).pin_memory()
        tok = tok_h.to(device, non_blocking=True)
    stream.synchronize()

    def job(n, t0=0):
        for t in range(n):
            model.step(tok, beta=beta_at(t0 + t, max(steps, 2)), lr=5e-4)

    with torch.cuda.stream(stream):
        job(warmup)
    stream.synchronize()
    faar.check_status(ctx, model.ws)
    ms_job = rt.timed(lambda: job(steps))
    faar.check_status(ctx, model.ws)
    faar.attention_status(ctx)                      # the attention kernels' bounded waits report separately
    loss_final = model.loss.cpu().tolist()

    def profiled():
        faar.profile_begin(ctx)
        job(1)

    rt.timed(profiled)
    prof = faar.profile_end(ctx)

    # end to end: the token batch comes from pinned host memory and the two loss values go back, every step
    loss_h = torch.zeros(2, dtype=torch.float32).pin_memory()

    def e2e_job(n):
        for t in range(n):
            tok.copy_(tok_h, non_blocking=True)
            model.step(tok, beta=beta_at(t, max(steps, 2)), lr=5e-4)
            loss_h.copy_(model.loss, non_blocking=True)
            stream.synchronize()

    ms_e2e = rt.timed(lambda: e2e_job(steps))
    clocks = rt.sampler.stop() if rt.sampler else None
    if rt.rank != 0:
        rt.finish()
        return 0
    pk, pk_kind = peaks()
    flop = stage2_flops(m)
    peak_key, frac_key, peak_why = applicable_peak(ms_job, clocks)
    value = rt.world * steps / (ms_job * 1e-3)
    tf = flop * steps / (ms_job * 1e-3) / 1e12
    kern = {k: {"launches": v[0], "total_ms": round(v[1], 3)} for k, v in prof.items()}
    step_ms = sum(v[1] for v in prof.values())
    for k in kern:
        kern[k]["share"] = round(prof[k][1] / step_ms, 4)
    gemm_ms = prof.get("gemm_ref", (0, 0.0))[1] + prof.get("gemm_bwd", (0, 0.0))[1]
    T = B * S
    q, kv = cfg.n_heads * cfg.head_dim, cfg.n_kv_heads * cfg.head_dim
    p_lin = cfg.n_layers * (2 * q * cfg.hidden + 2 * kv * cfg.hidden + 3 * cfg.ffn * cfg.hidden)
    gemm_flop = 8.0 * T * p_lin + 6.0 * T * cfg.vocab * cfg.hidden
    gemm_tf = gemm_flop / (gemm_ms * 1e-3) / 1e12 if gemm_ms else 0.0
    roofline = {"kernel": "the tensor-core GEMM launches of one step (forward products, input gradients, dW + update)",
                "bound": "tensor", "achieved": round(gemm_tf, 1), "peak": pk[peak_key], "unit": "TFLOP/s",
                "frac": tensor_fracs(gemm_tf, pk)[frac_key], **tensor_fracs(gemm_tf, pk), "traffic": None,
                "peak_source": f"{pk_kind} {peak_key}: {peak_why}",
                "timed": "per-kernel CUDA events on the launching stream, one profiled step after the timed job"}
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": steps, "warmup": warmup,
            "ms_per_step": ms_job / steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic", "config": workload_config(5) if not args.layers else
            dict(workload_config(5), n_layers=cfg.n_layers, note="reduced layer count (--layers)"),
            "clocks": clocks, "step_tflops": round(tf, 1), "step_frac": tensor_fracs(tf, pk),
            "e2e": {"value": rt.world * steps / (ms_e2e * 1e-3), "unit": UNIT, "steps": steps, "h2d_bytes_per_step": T * 4,
                    "d2h_bytes_per_step": 8, "path": "Stage2Model.step: token ids copied in from pinned memory, losses copied out and "
                                                     "the stream synchronised every step"},
            "gpu_launches": steps * sum(v[0] for v in prof.values()), "roofline": roofline, "kernels": kern,
            "final_loss": loss_final}
    if not args.quick:
        rate, dt, threads, sample = oracle_stage2_rate()
        line["cpu_baseline"] = {"value": rate, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample}
    print(json.dumps(line))
    rt.finish()
    return 0


def run_ours(args):
    import numpy as np
    import torch

    from paper_2603_22370_b200 import faar, inputs

    rt = Runtime(args)
    if args.config in (3, 4):
        return run_block(args, rt)
    if args.config == 5:
        return run_stage2(args, rt)
    rank, world, dev, device, dist = rt.rank, rt.world, rt.dev, rt.device, rt.dist
    n_gpus = args.gpus
    steps, warmup = args.steps, max(args.warmup, 3)
    stream, ctx = rt.stream, rt.ctx

    # ---- inputs, resident in HBM (each rank its own layer: seed = rank)
    Wn, Xn = inputs.config2(rank, O, K, T)
    W = torch.from_numpy(Wn).to(device).to(torch.bfloat16)
    X = torch.from_numpy(Xn).to(device).to(torch.bfloat16)
    del Wn
    shape = faar.make_shape(O, K, T, yref_transposed=1)      # target stored one row per output feature
    ws = torch.empty(faar.workspace_size(shape), dtype=torch.uint8, device=device)
    Xt = torch.empty((K, T), dtype=torch.bfloat16, device=device)
    Yref = torch.zeros((O, shape.ldy), dtype=torch.bfloat16, device=device)
    scales = torch.empty((O, K // 16), dtype=torch.uint8, device=device)
    code = torch.empty((O, K // 2), dtype=torch.uint8, device=device)
    s_global = torch.empty(1, dtype=torch.float32, device=device)
    V = torch.empty((O, K), dtype=torch.float32, device=device)
    m = torch.zeros((O, K), dtype=torch.float32, device=device)
    u = torch.zeros((O, K), dtype=torch.float32, device=device)
    loss = torch.zeros(2, dtype=torch.float32, device=device)
    packed = torch.empty((O, K // 2), dtype=torch.uint8, device=device)
    scales_out = torch.empty((O, K // 16), dtype=torch.uint8, device=device)
    torch.cuda.synchronize()

    with torch.cuda.stream(stream):
        faar.workspace_init(ctx, ws)
        faar.transpose_bf16(ctx, T, K, X, K, Xt, T)          # once per layer: K-major operand of the dW GEMM
        faar.layer_ref(ctx, shape, X, W, Yref, ws)           # frozen target (Procedure step 8)
    stream.synchronize()

    def chain_kw(t, n):
        """--chain: the backward pass of step t also builds step t+1's soft weights and step t+1 skips the
        soft-weights kernel (the same values bit for bit; two kernels per step instead of three)."""
        if not args.chain:
            return {}
        return dict(wsoft_ready=int(t > 0), beta_next=beta_at(t + 1, n) if t + 1 < n else 0.0)

    def job(n_steps, step0=0):
        """set-up, n_steps optimisation steps, harden + pack -- all enqueued on `stream`."""
        m.zero_()
        u.zero_()
        faar.softquant_init(ctx, shape, W, 0.0, scales, s_global, code, V, ws)
        for t in range(n_steps):
            hp = faar.make_hparams(beta=beta_at(t, n_steps), step=t + 1, **chain_kw(t, n_steps))
            faar.layer_step(ctx, shape, hp, X, Xt, Yref, V, code, scales, s_global, m, u, loss, ws)
        faar.harden_pack(ctx, shape, V, code, scales, s_global, packed, scales_out, None, None)

    sampler, barrier, timed = rt.sampler, rt.barrier, rt.timed

    # ---- warm-up, then the timed job
    with torch.cuda.stream(stream):
        job(warmup)
    stream.synchronize()
    ms_job = timed(lambda: job(steps))
    faar.check_status(ctx, ws)
    loss_final = loss.cpu().tolist()
    value = n_gpus * steps / (ms_job * 1e-3)
    # amax + init; soft weights + forward + backward per step (chained: one soft-weights launch in all); harden_pack
    gpu_launches = 2 + (1 + 2 * steps if args.chain else 3 * steps) + 1

    # ---- second pass of the same job with per-kernel CUDA events (library hooks, same stream)
    def profiled():
        faar.profile_begin(ctx)
        job(steps)

    timed(profiled)
    prof = faar.profile_end(ctx)

    # ---- the once-per-layer / HBM-bound kernels alone: back-to-back launches over rotated buffer sets
    # (3 sets x 150 MB > L2), one event pair around all of them, so launch overhead is amortised
    def elementwise_rates(rounds=10, sets=3):
        bufs = []
        for r in range(sets):
            bufs.append(dict(W=W.clone(), V=torch.rand((O, K), dtype=torch.float32, device=device), code=code.clone(),
                             scales=scales.clone(), packed=torch.empty_like(packed), so=torch.empty_like(scales_out),
                             wsoft=torch.empty((O, K), dtype=torch.bfloat16, device=device),
                             X=X.clone(), Xq=torch.empty_like(X), sx=torch.empty(1, dtype=torch.float32, device=device)))
        calls = {
            "softquant_init": lambda b: faar.softquant_init(ctx, shape, b["W"], 0.0, b["scales"], s_global, b["code"],
                                                            b["V"], ws),
            "soft_weights": lambda b: faar.softquant_eval(ctx, shape, b["V"], b["code"], b["scales"], s_global, 8.0,
                                                          None, None, b["wsoft"]),
            "harden_pack": lambda b: faar.harden_pack(ctx, shape, b["V"], b["code"], b["scales"], s_global, b["packed"],
                                                      b["so"], None, None),
        }
        calls["act_fakequant"] = lambda b: faar.act_fakequant(ctx, T, K, b["X"], K, 0.0, b["Xq"], K, b["sx"], None, None, ws)
        out = {}
        for name in ("soft_weights", "harden_pack", "act_fakequant", "softquant_init"):   # init last: it overwrites V
            fn = calls[name]
            with torch.cuda.stream(stream):
                for b in bufs:
                    fn(b)
            stream.synchronize()
            ms = timed(lambda: [fn(b) for _ in range(rounds) for b in bufs])
            out[name] = 1e3 * ms / (rounds * sets)
        return out

    ew_us = elementwise_rates()

    # ---- the layer's input gradient dX = dY W_soft (soft weights + transpose + GEMM in one call), alone
    def layer_dx_us(rounds=20):
        dY = torch.randn((T, O), dtype=torch.float32, device=device).to(torch.bfloat16)
        WsT = torch.empty((K, (O + 7) // 8 * 8), dtype=torch.bfloat16, device=device)
        dX = torch.empty((T, K), dtype=torch.bfloat16, device=device)
        plain = faar.make_shape(O, K, T)                       # dY is [T, O] here
        fn = lambda: faar.layer_dx(ctx, plain, 8.0, dY, V, code, scales, s_global, WsT, dX, ws)
        with torch.cuda.stream(stream):
            for _ in range(3):
                fn()
        stream.synchronize()
        return 1e3 * timed(lambda: [fn() for _ in range(rounds)]) / rounds

    dx_us = layer_dx_us()

    # ---- the deployable operands through the library's own NVFP4 GEMM: X_q W_final^T, alone
    def nvfp4_gemm_us(rounds=20):
        pw = torch.empty((O, K // 2), dtype=torch.uint8, device=device)
        sw = torch.empty((O, K // 16), dtype=torch.uint8, device=device)
        faar.harden_pack(ctx, shape, V, code, scales, s_global, pw, sw, None, None)
        Xq = torch.empty_like(X)
        sx = torch.empty(1, dtype=torch.float32, device=device)
        px = torch.empty((T, K // 2), dtype=torch.uint8, device=device)
        scx = torch.empty((T, K // 16), dtype=torch.uint8, device=device)
        faar.act_fakequant(ctx, T, K, X, K, 0.0, Xq, K, sx, px, scx, ws)
        tw = torch.empty(-(-O // 128) * -(-(K // 16) // 4) * 512, dtype=torch.uint8, device=device)
        tx = torch.empty(-(-T // 128) * -(-(K // 16) // 4) * 512, dtype=torch.uint8, device=device)
        faar.swizzle_scales(ctx, O, K // 16, sw, tw)
        faar.swizzle_scales(ctx, T, K // 16, scx, tx)
        Y = torch.empty((T, O), dtype=torch.bfloat16, device=device)
        fn = lambda: faar.nvfp4_gemm(ctx, T, O, K, px, tx, sx, pw, tw, s_global, Y, O, ws)
        with torch.cuda.stream(stream):
            for _ in range(3):
                fn()
        stream.synchronize()
        return 1e3 * timed(lambda: [fn() for _ in range(rounds)]) / rounds

    fp4_us = nvfp4_gemm_us()

    # ---- Eq. 6's alignment loss alone: 4096 tokens x 128 256 logits (3.2 GB moved per call, far above L2)
    AL_T, AL_V, AL_D = args.align_tokens, 128256, 2048

    def align_loss_us(rounds=5):
        g = torch.Generator(device=device).manual_seed(1)
        zf = (torch.randn((AL_T, AL_V), device=device, generator=g) * 3).to(torch.bfloat16)
        zq = (zf.float() + 0.3 * torch.randn((AL_T, AL_V), device=device, generator=g)).to(torch.bfloat16)
        hf = torch.randn((AL_T, AL_D), device=device, generator=g).to(torch.bfloat16)
        hq = (hf.float() + 0.05 * torch.randn((AL_T, AL_D), device=device, generator=g)).to(torch.bfloat16)
        dz, dh = torch.empty_like(zq), torch.empty_like(hq)
        l2 = torch.zeros(2, dtype=torch.float32, device=device)
        aws = torch.empty(faar.align_loss_workspace_size(AL_T, AL_V), dtype=torch.uint8, device=device)
        faar.workspace_init(ctx, aws)
        fn = lambda: faar.align_loss(ctx, AL_T, AL_V, AL_D, zf, zq, AL_V, hf, hq, AL_D, 1.0, 1.0, dz, dh, l2, aws)
        with torch.cuda.stream(stream):
            for _ in range(3):
                fn()
        stream.synchronize()
        us = 1e3 * timed(lambda: [fn() for _ in range(rounds)]) / rounds
        faar.check_status(ctx, aws)
        return us

    al_us = align_loss_us()

    if args.quick:
        if rank == 0:
            print(json.dumps({"quick": True, "steps": steps, "ms_per_step": ms_job / steps,
                              "kernels_avg_us": {k: round(1e3 * v[1] / v[0], 2) for k, v in prof.items()},
                              "elementwise_alone_us": {k: round(v, 2) for k, v in ew_us.items()},
                              "layer_dx_us": round(dx_us, 2), "nvfp4_gemm_us": round(fp4_us, 2),
                              "align_loss_us": round(al_us, 2)}))
        if sampler:
            sampler.stop()
        if world > 1:
            dist.destroy_process_group()
        return 0

    # ---- end to end: the calibration batch comes from pinned host memory every step; its frozen target is
    # formed on the device from the copied batch (Procedure step 8) rather than shipped
    Xh = torch.from_numpy(Xn).to(torch.bfloat16).pin_memory()
    loss_h = torch.zeros(2, dtype=torch.float32).pin_memory()
    # two staging sets, used alternately: the copy of batch t+1 overlaps step t
    stage_sets = [(torch.empty_like(X), torch.empty_like(Xt), torch.empty_like(Yref)) for _ in range(2)]
    e2e_steps = min(steps, 200)
    h2d_bytes = T * K * 2
    e2e_path = "faar_layer_step_host: pinned X copied in on a copy stream (two staging sets, the copy of batch t+1 " \
               "overlaps step t), X^T and the frozen target Y_ref = X W^T rebuilt on the device, step, losses copied out"

    def e2e_job(n):
        m.zero_()
        u.zero_()
        faar.softquant_init(ctx, shape, W, 0.0, scales, s_global, code, V, ws)
        for t in range(n):
            hp = faar.make_hparams(beta=beta_at(t, n), step=t + 1, **chain_kw(t, n))
            X_dev, Xt_dev, Y_dev = stage_sets[t & 1]
            faar.layer_step_host(ctx, shape, hp, Xh, None, W, X_dev, Xt_dev, Y_dev, V, code, scales, s_global, m, u,
                                 loss, loss_h, ws)
        faar.harden_pack(ctx, shape, V, code, scales, s_global, packed, scales_out, None, None)

    with torch.cuda.stream(stream):
        e2e_job(3)
    stream.synchronize()
    ms_e2e = timed(lambda: e2e_job(e2e_steps))
    e2e_value = n_gpus * e2e_steps / (ms_e2e * 1e-3)
    faar.check_status(ctx, ws)

    # ---- the same end to end with quantised activations (the X_q of Eq. 5): the batch travels as the packed NVFP4
    # codes and block scales the library's own quantiser produced (4.5 bits per value) plus its frozen target
    with torch.cuda.stream(stream):
        Xq_units = torch.empty_like(X)
        sx = torch.empty(1, dtype=torch.float32, device=device)
        px = torch.empty((T, K // 2), dtype=torch.uint8, device=device)
        scx = torch.empty((T, K // 16), dtype=torch.uint8, device=device)
        faar.act_fakequant(ctx, T, K, X, K, 0.0, Xq_units, K, sx, px, scx, ws)
    stream.synchronize()
    act_scale = float(sx.item())
    px_h, scx_h, yref_h = px.cpu().pin_memory(), scx.cpu().pin_memory(), Yref.cpu().pin_memory()
    pk_sets = [(torch.empty_like(px), torch.empty_like(scx), torch.empty_like(X), torch.empty_like(Yref)) for _ in range(2)]
    pk_bytes = px_h.numel() + scx_h.numel() + yref_h.numel() * 2
    del Xq_units

    def e2e_packed_job(n):
        m.zero_()
        u.zero_()
        faar.softquant_init(ctx, shape, W, 0.0, scales, s_global, code, V, ws)
        for t in range(n):
            hp = faar.make_hparams(beta=beta_at(t, n), step=t + 1, act_scale=act_scale)
            pd, sd, xd, yd = pk_sets[t & 1]
            faar.layer_step_host_nvfp4(ctx, shape, hp, px_h, scx_h, yref_h, pd, sd, xd, yd, V, code, scales, s_global, m, u,
                                       loss, loss_h, ws)
        faar.harden_pack(ctx, shape, V, code, scales, s_global, packed, scales_out, None, None)

    with torch.cuda.stream(stream):
        e2e_packed_job(3)
    stream.synchronize()
    ms_e2e_pk = timed(lambda: e2e_packed_job(e2e_steps))
    faar.check_status(ctx, ws)
    clocks = sampler.stop() if sampler else None

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return 0

    # ---- rooflines
    pk, pk_kind = peaks()
    n_w = O * K
    flops = 2.0 * T * O * K
    peak_key, frac_key, peak_why = applicable_peak(ms_job, clocks)

    def avg_us(name):
        return 1e3 * prof[name][1] / prof[name][0] if name in prof else None

    kernels = {}
    for name, bound, work in [
        ("gemm_fwd", "tensor", flops), ("gemm_bwd", "tensor", flops),
        ("soft_weights", "hbm", 6.5625 * n_w),              # V 4 + code .5 + scale 1/16 read, BF16 operand 2 written
        ("softquant_init", "hbm", 6.5625 * n_w),            # W 2 read; V 4 + code .5 + scale 1/16 written
        ("harden_pack", "hbm", 5.125 * n_w),                # V 4 + code .5 + scale 1/16 read; .5 + 1/16 written
        ("act_fakequant", "hbm", 4.0 * T * K),              # X 2 read, X_q units 2 written (+2 for the amax pass)
    ]:
        if bound == "tensor":
            us = avg_us(name)
            ach = work / (us * 1e-6) / 1e12
            kernels[name] = {"avg_us": round(us, 2), "bound": bound, "achieved": round(ach, 1), "peak": pk[peak_key],
                             "unit": "TFLOP/s", "frac": tensor_fracs(ach, pk)[frac_key], **tensor_fracs(ach, pk),
                             "timed": "CUDA events around each launch inside the K-step job"}
        else:
            # HBM-bound kernels: timed alone, launches back to back over rotated buffers (cold L2)
            us = ew_us[name]
            ach = work / (us * 1e-6) / 1e9
            kernels[name] = {"avg_us": round(us, 2), "bound": bound, "achieved": round(ach, 1), "peak": pk["hbm_gbs"],
                             "unit": "GB/s", "frac": round(ach / pk["hbm_gbs"], 4),
                             "timed": "30 back-to-back launches over 3 rotated buffer sets, one event pair"}
    dx_tf = flops / (dx_us * 1e-6) / 1e12
    kernels["layer_dx"] = {"avg_us": round(dx_us, 2), "bound": "tensor", "achieved": round(dx_tf, 1),
                           "peak": pk["bf16_tflops"], "unit": "TFLOP/s", "frac": tensor_fracs(dx_tf, pk)["frac_burst"],
                           **tensor_fracs(dx_tf, pk),
                           "timed": "20 back-to-back calls (soft weights, transpose and GEMM each), one event pair",
                           "note": "input gradient dX = dY W_soft, not part of a Stage-1 step"}
    fp4_tf = flops / (fp4_us * 1e-6) / 1e12
    kernels["nvfp4_gemm"] = {"avg_us": round(fp4_us, 2), "bound": "tensor", "achieved": round(fp4_tf, 1),
                             "peak": 4.0 * pk["bf16_tflops"], "unit": "TFLOP/s", "frac": round(fp4_tf / (4.0 * pk["bf16_tflops"]), 4),
                             "frac_nominal": round(fp4_tf / 9000.0, 4),
                             "peak_note": "measured BF16 burst rate x 4 (the nominal FP4 : BF16 ratio)",
                             "timed": "20 back-to-back calls, one event pair",
                             "note": "X_q W_final^T on the packed NVFP4 operands (block-scaled FP4 tensor-core path); a check "
                                     "of the deployable output, not part of a Stage-1 step"}
    al_bytes = 3.0 * AL_T * AL_V * 2 + 3.0 * AL_T * AL_D * 2          # both logit / hidden tensors read, one gradient written
    kernels["align_loss"] = {"avg_us": round(al_us, 2), "bound": "hbm", "achieved": round(al_bytes / (al_us * 1e-6) / 1e9, 1),
                             "peak": pk["hbm_gbs"], "unit": "GB/s",
                             "frac": round(al_bytes / (al_us * 1e-6) / 1e9 / pk["hbm_gbs"], 4),
                             "timed": f"5 back-to-back calls on {AL_T} tokens x 128256 logits (+ 2048 hidden), one event pair",
                             "note": "Eq. 6's KL and last-hidden terms with gradients; not part of a Stage-1 step"}
    kernels["softquant_init"]["note"] = "amax pass + bracket pass together; the amax pass re-reads W (+2 B/weight, not counted)"
    for name in prof:
        kernels.setdefault(name, {})["in_job_avg_us"] = round(avg_us(name), 2)
        kernels[name]["launches"] = prof[name][0]
    dominant = max(("gemm_fwd", "gemm_bwd"), key=lambda k: prof[k][1])
    d = kernels[dominant]
    roofline = {"kernel": dominant, "bound": "tensor", "achieved": d["achieved"], "peak": d["peak"],
                "unit": "TFLOP/s", "frac": d["frac"], "frac_burst": d["frac_burst"],
                "frac_sustained": d["frac_sustained"], "frac_nominal": d["frac_nominal"],
                "traffic": ncu_traffic(dominant),
                "peak_source": f"{pk_kind} {peak_key}: {peak_why}",
                "timed": "per-kernel CUDA events on the launching stream, second pass of the same K-step job"}

    # ---- CPU oracle beside it (bounded sample)
    cpu_rows, cpu_steps = 256, 8
    cpu_rate, cpu_dt, cpu_threads = oracle_rate(cpu_rows, cpu_steps, 1)
    cpu_baseline = {"value": cpu_rate, "unit": UNIT, "cores": cpu_threads, "kind": "oracle",
                    "sample": f"{cpu_steps} steps on the first {cpu_rows} of {O} output rows (exact sub-problem: the "
                              f"loss separates over rows), all {T} tokens; rate scaled by {O}/{cpu_rows}"}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": n_gpus, "steps": steps, "warmup": warmup,
            "ms_per_step": ms_job / steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic", "config": workload_config(2),
            "chained_soft_weights": bool(args.chain),
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": UNIT, "steps": e2e_steps,
                    "h2d_bytes_per_step": h2d_bytes, "d2h_bytes_per_step": 8,
                    "path": e2e_path},
            "e2e_nvfp4_activations": {"value": n_gpus * e2e_steps / (ms_e2e_pk * 1e-3), "unit": UNIT, "steps": e2e_steps,
                                      "h2d_bytes_per_step": pk_bytes, "d2h_bytes_per_step": 8,
                                      "path": "faar_layer_step_host_nvfp4: quantised activations (Eq. 5's X_q) as packed NVFP4 "
                                              "codes + block scales and the frozen target copied in from pinned memory, "
                                              "expanded on the device, step, losses copied out; a different workload from "
                                              "`e2e` (which steps on the unquantised BF16 batch)"},
            "gpu_launches": gpu_launches, "roofline": roofline, "cpu_baseline": cpu_baseline,
            "kernels": kernels, "final_loss": loss_final,
            "step_tflops": round(2 * flops * steps / (ms_job * 1e-3) / 1e12, 1)}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=2, choices=[2, 3, 4, 5],
                    help="2: the down_proj-shaped layer (the headline); 3 / 4: the seven linears of a Llama-3.2-1B- / "
                         "Qwen3-1.7B-shaped decoder block")
    ap.add_argument("--layers", type=int, default=0,
                    help="--config 5 only: decoder blocks of the model (0 = the workload's 16); smaller for profiler captures")
    ap.add_argument("--calib-tokens", type=int, default=65536,
                    help="rows of the synthetic calibration set of --config 3 / 4 (4096-row minibatches, round-robin)")
    ap.add_argument("--align-tokens", type=int, default=4096,
                    help="tokens of the alignment-loss timing (128256 logits each); smaller for profiler captures")
    ap.add_argument("--chain", action="store_true",
                    help="build each step's soft weights inside the previous step's backward kernel (same values; the "
                         "job is faster, the backward kernel slower, so its roofline line is not comparable)")
    ap.add_argument("--quick", action="store_true",
                    help="timed job and per-kernel pass only (no end-to-end pass, no CPU oracle leg); for profilers")
    args = ap.parse_args()
    return run_reference(args) if args.impl == "reference" else run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
