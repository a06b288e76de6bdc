#!/usr/bin/env python
"""Throughput of the integer-only RoBERTa-Base encoder (I-BERT) on B200.

One *step* = one forward pass of the whole 12-layer integer-only encoder (5 kernels per
layer, all inside libibert_b200) over one batch of synthetic int8 activations.
Prints ONE JSON line (rank 0).  ``--impl reference`` times the CPU oracle instead.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--config 2|3|4] [--batch B] [--sustain SECONDS] [--scales analytic|calibrated]
                    [--workload layers|model] [--pow2-scores] [--graph] [--only KERNEL]

With --gpus N > 1 and no WORLD_SIZE in the environment it starts the N ranks itself.
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
from pathlib import Path

ROOT = Path(__file__).resolve().parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))

METRIC = "tokens/s int-only RoBERTa-Base on 1 B200; % INT8 TC peak, % HBM for i-ops"
UNIT = "tokens/s"
DEFAULT_BATCH = {2: 128, 3: 32, 4: 64}


SPEC_INT8_TOPS = 4500.0          # nominal dense INT8 rate of one B200
SPEC_SM_MHZ = 1965.0


def _table_rows(path: Path) -> list[list[str]]:
    """Cells of every `| a | b | ... |` row of a markdown file (header and ruler rows included)."""
    if not path.exists():
        return []
    rows = []
    for line in path.read_text().splitlines():
        line = line.strip()
        if line.startswith("|") and line.endswith("|"):
            rows.append([c.strip().strip("`") for c in line[1:-1].split("|")])
    return rows


def ncu_figures() -> dict:
    """{(kernel class, config, batch): {"dram_bytes", "warp_instructions", "alu", "fma"}} from
    profiles/ncu_figures.md -- the per-launch figures of the committed ncu captures (DRAM bytes, warp
    instructions in all / on the ALU pipe / on the multiply-add pipe), written by the same step that
    writes the per-kernel summaries, so that this file and they cannot drift."""
    out = {}
    for r in _table_rows(ROOT / "profiles" / "ncu_figures.md"):
        if len(r) < 7:
            continue
        try:
            out[(r[0], int(r[1]), int(r[2]))] = {"dram_bytes": float(r[3]), "warp_instructions": float(r[4]),
                                                 "alu": float(r[5]), "fma": float(r[6])}
        except ValueError:
            continue                      # header / ruler rows
    return out


def probe_peaks() -> dict:
    """Figures of the issue-rate probes (profiles/issue_probes.md): {"int32_lane_ops_per_clk_sm": ...,
    "i8_mma_tops": ...}; empty when the summary is absent."""
    out = {}
    for r in _table_rows(ROOT / "profiles" / "issue_probes.md"):
        if len(r) >= 2 and r[0] in ("int32_lane_ops_per_clk_sm", "alu_pipe_lane_ops_per_clk_sm", "i8_mma_tops"):
            try:
                out[r[0]] = float(r[1])
            except ValueError:
                pass
    return out


# --------------------------------------------------------------------------- helpers
def measured_peaks() -> tuple[dict, str]:
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        d = json.loads(p.read_text())
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"])}, "measured"
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap,power.draw")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) >= 6:
                self.rows.append(parts)

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        mhz, mx, reasons, watts = [], None, set(), []
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for r in self.rows:
            try:
                mhz.append(float(r[0]))
                mx = float(r[1])
            except ValueError:
                continue
            for n, v in zip(names, r[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
            if len(r) > 6:
                try:
                    watts.append(float(r[6]))
                except ValueError:
                    pass
        return {"sm_mhz": statistics.median(mhz) if mhz else None, "sm_max_mhz": mx,
                "reasons": sorted(reasons), "samples": len(mhz),
                "power_w_median": statistics.median(watts) if watts else None,
                "power_w_max": max(watts) if watts else None}


def algorithmic_work(H: int, F: int, L: int, heads: int, T: int) -> dict:
    """Per-launch algorithmic ops / bytes of each kernel class of one layer on T tokens."""
    w = {}
    w["gemm_qkv"] = {"ops": 2.0 * T * 3 * H * H, "bytes": T * H + 3 * H * H + T * 3 * H}
    w["attention"] = {"ops": 2.0 * T * L * 64 * 2 * heads, "bytes": T * 3 * H + T * H}
    w["gemm_out"] = {"ops": 2.0 * T * H * H, "bytes": T * H + H * H + 4 * T * H}
    w["layernorm"] = {"ops": 0.0, "bytes": 4 * T * H + T * H + T * H}
    w["gemm_ffn1_gelu"] = {"ops": 2.0 * T * F * H, "bytes": T * H + F * H + T * F}
    w["gemm_ffn2"] = {"ops": 2.0 * T * F * H, "bytes": T * F + F * H + 4 * T * H}
    # linear + residual + LayerNorm in one kernel: operands, int8 residual in, int8 out
    w["gemm_out_ln"] = {"ops": 2.0 * T * H * H, "bytes": T * H + H * H + T * H + T * H}
    w["gemm_ffn2_ln"] = {"ops": 2.0 * T * F * H, "bytes": T * F + F * H + T * H + T * H}
    return w


# --------------------------------------------------------------------------- reference arm
def oracle_on_sample(n_seq: int, L: int, x=None, params=None, model=None):
    """The CPU oracle on the first n_seq sequences of the very batch the GPU processes (sequences
    are independent, so its result must equal the GPU's rows for those sequences).
    Returns (result array, seconds, layers)."""
    import oracle
    oracle.lib()
    if model is not None:
        e, hd = model["emb"], model["head"]
        ids, lens = model["ids"][:n_seq * L], model["lens"][:n_seq]
        t0 = time.perf_counter()
        h = oracle.embedding(ids, L, e["word"], e["S_word"], e["pos"], e["S_pos"], e["gamma"], e["beta"], e["S_out"])
        for p in model["layers"]:
            h = oracle.encoder_layer(p, h, n_seq, L, lens=lens).out
        out = oracle.classifier(h, n_seq, L, model["layers"][-1]["S_out"], hd["w"], hd["S_w"], hd["bias"])
        return out, time.perf_counter() - t0, len(model["layers"])
    t0 = time.perf_counter()
    h = x[:n_seq * L]
    for p in params:
        h = oracle.encoder_layer(p, h, n_seq, L).out
    return h, time.perf_counter() - t0, len(params)


def run_reference(args):
    """The reference arm: the CPU oracle, as it stands, on a bounded sample of the workload.
    Under a multi-rank launch rank 0 alone computes; the ranks only meet at a gloo barrier."""
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("gloo", rank=rank, world_size=world)
        dist.barrier()
        dist.destroy_process_group()
    if rank != 0:
        return
    import oracle
    from paper_2101_01321_b200 import synth
    cfg = synth.CONFIGS[args.config]
    if args.seq_len:
        import dataclasses
        cfg = dataclasses.replace(cfg, L=args.seq_len)
    batch = args.batch or DEFAULT_BATCH[args.config]
    n_seq = 2
    full_model = args.workload == "model"
    oracle.lib()
    if full_model:
        m = synth.make_full_model(args.config, n_seq, L=cfg.L, scales=args.scales)
        params = m["layers"]

        def step():
            return oracle_on_sample(n_seq, cfg.L, model=m)[0]
    else:
        x, params = synth.make_model(args.config, n_seq, L=cfg.L, scales=args.scales)

        def step():
            return oracle_on_sample(n_seq, cfg.L, x=x, params=params)[0]

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = time.perf_counter() - t0
    tokens = n_seq * cfg.L * args.steps
    value = tokens / dt
    sample = (f"each step = first {n_seq} sequences ({n_seq * cfg.L} tokens) of the batch through "
              f"{'the embedding, ' if full_model else ''}all {len(params)} layers"
              f"{' and the classifier' if full_model else ''} with the CPU oracle")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int8",
        "data": "synthetic", "config": workload_config(cfg, batch, args.gpus, full_model,
                                                       float(m["lens"].mean()) / cfg.L if full_model else 1.0,
                                                       scales=args.scales),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def workload_config(cfg, batch, n_gpus, full_model=False, valid_frac=1.0, use_graph=False, pow2=False,
                    scales="analytic", packed=False):
    layout = (f"packed batch (no padding; the sentence-length mix fills {100 * valid_frac:.0f} % of B x L)" if packed else
              f"key-padding mask ({100 * valid_frac:.0f} % of the positions valid)")
    what = (f"token ids -> INT8 embedding + LayerNorm -> {cfg.layers} integer-only encoder layers, {layout} "
            f"-> first-token classifier"
            if full_model else f"{cfg.layers}-layer integer-only encoder")
    scale_note = {"analytic": "closed-form static scales (int8 sites clip at 4-5 sigma, Q16 sites at 8 sigma)",
                  "calibrated": "static scales from each site's max|x| on the first sequences of the seeded input "
                                "(written by tests/golden/make_calibrated_scales.py with the CPU oracle)"}[scales]
    return {"workload": f"config {cfg.config_id}: {what}, H={cfg.H}, "
                        f"heads={cfg.heads}, FFN={cfg.F}, L={cfg.L}, B={batch} per GPU",
            "batch_per_gpu": batch, "global_batch": batch * n_gpus, "parallelism": f"dp{n_gpus} (batch shards, no collective)",
            "l2": "flushed between timed steps (512 MiB write); per-step activation traffic also exceeds L2",
            "launch": "CUDA graph replay" if use_graph else "one C-ABI call per layer",
            "activation_scales": scale_note,
            "score_scales": "raised to ln2 / 2^k" if pow2 else "as the activation scales give them"}


# --------------------------------------------------------------------------- our arm
def run_ours(args):
    import numpy as np
    import torch

    from paper_2101_01321_b200 import binding, build, dp, synth

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    dist = None
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (no CPU path)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    build.build()

    cfg = synth.CONFIGS[args.config]
    if args.seq_len:
        import dataclasses
        cfg = dataclasses.replace(cfg, L=args.seq_len)
    batch = args.batch or DEFAULT_BATCH[args.config]
    T = batch * cfg.L
    # weak scaling: rank r owns sequences [r*batch, (r+1)*batch) of the global batch
    first, last = dp.shard_range(batch * world, world, rank)
    assert last - first == batch
    stream = torch.cuda.Stream(device=dev)
    ctx = binding.Context(local_rank, stream)
    if args.fusion:
        ctx.ibert_set_fusion(args.fusion)
    bufs = [torch.empty((T, cfg.H), dtype=torch.int8, device=dev) for _ in range(2)]
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
    full_model = args.workload == "model"
    if not full_model:
        # the headline workload: the encoder layers on full-length sequences, int8 activations in and out
        x_np, params = synth.make_model(args.config, batch, shard=rank, pow2_scores=args.pow2_scores, L=cfg.L,
                                          scales=args.scales)
        layers = [ctx.ibert_layer_create(p) for p in params]
        x_dev = torch.from_numpy(x_np).to(dev)
        x_pin = torch.from_numpy(x_np).pin_memory()
        out_pin = torch.empty((T, cfg.H), dtype=torch.int8).pin_memory()
        x_stage = torch.empty((T, cfg.H), dtype=torch.int8, device=dev)
        valid_tokens = T

        graphs = {}

        def forward(src, eager=False, final_out=None):
            if args.graph and not eager:
                # one captured graph per (input buffer, output buffer)
                dst = final_out if final_out is not None else bufs[(len(layers) - 1) & 1]
                key = (src.data_ptr(), dst.data_ptr())
                g = graphs.get(key)
                if g is None:
                    g = graphs[key] = binding.Graph(ctx, layers, src, batch, cfg.L, dst)
                return g.launch()
            h = src
            for i, ly in enumerate(layers):
                last = i == len(layers) - 1
                h, _ = ctx.ibert_encoder_layer(ly, h, batch, cfg.L,
                                               out=final_out if (last and final_out is not None) else bufs[i & 1])
            return h
    else:
        # the model around the layers on a padded batch: token ids in, INT8 embedding + LayerNorm,
        # the layers with a key-padding mask, first-token classifier, INT32 logits out
        m = synth.make_full_model(args.config, batch, shard=rank, L=cfg.L, scales=args.scales)
        layers = [ctx.ibert_layer_create(p) for p in m["layers"]]
        e, hd = m["emb"], m["head"]
        word_d, pos_d = torch.from_numpy(e["word"]).to(dev), torch.from_numpy(e["pos"]).to(dev)
        hw_d, hb_d = torch.from_numpy(hd["w"]).to(dev), torch.from_numpy(hd["bias"]).to(dev)
        lens_d = torch.from_numpy(m["lens"]).to(dev)
        valid_tokens = int(m["lens"].sum())
        ids_np = m["ids"]
        if args.packed:
            # the same sequences without their padding: valid rows in sequence order + first-row offsets
            keep = np.concatenate([np.arange(b * cfg.L, b * cfg.L + n) for b, n in enumerate(m["lens"])])
            ids_np = np.ascontiguousarray(m["ids"][keep])
            cu_d = torch.from_numpy(np.concatenate([[0], np.cumsum(m["lens"])]).astype(np.int32)).to(dev)
            bufs = [torch.empty((valid_tokens, cfg.H), dtype=torch.int8, device=dev) for _ in range(2)]
        x_dev = torch.from_numpy(ids_np).to(dev)
        x_pin = torch.from_numpy(ids_np).pin_memory()
        x_stage = torch.empty_like(x_dev)
        logits = torch.empty((batch, synth.N_LABELS), dtype=torch.int32, device=dev)
        out_pin = torch.empty((batch, synth.N_LABELS), dtype=torch.int32).pin_memory()
        emb_out = torch.empty((x_dev.numel(), cfg.H), dtype=torch.int8, device=dev)
        S_last = m["layers"][-1]["S_out"]

        def forward(src, eager=False, final_out=None):
            dst = final_out if final_out is not None else logits
            if args.packed:
                h, _ = ctx.ibert_embedding_packed_i8(src, cu_d, cfg.L, word_d, e["S_word"], pos_d, e["S_pos"], e["gamma"],
                                                     e["beta"], e["S_out"], out=emb_out)
                for i, ly in enumerate(layers):
                    h, _ = ctx.ibert_encoder_layer_packed(ly, h, cu_d, cfg.L, out=bufs[i & 1])
                return ctx.ibert_classifier_packed_i8(h, cu_d, S_last, hw_d, hd["S_w"], hb_d, out=dst)[0]
            h, _ = ctx.ibert_embedding_i8(src, cfg.L, word_d, e["S_word"], pos_d, e["S_pos"], e["gamma"], e["beta"],
                                          e["S_out"], out=emb_out)
            for i, ly in enumerate(layers):
                h, _ = ctx.ibert_encoder_layer_masked(ly, h, batch, cfg.L, lens_d, out=bufs[i & 1])
            out, _ = ctx.ibert_classifier_i8(h, batch, cfg.L, S_last, hw_d, hd["S_w"], hb_d, out=dst)
            return out

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize(dev)

    def timed_steps(n, e2e=False):
        """Per-step CUDA events on the launching stream; L2 flushed (untimed) between steps."""
        times = []
        with torch.cuda.stream(stream):
            for _ in range(n):
                flush.fill_(1)
                e0 = torch.cuda.Event(enable_timing=True)
                e1 = torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                if e2e:
                    x_stage.copy_(x_pin, non_blocking=True)
                    h = forward(x_stage)
                    out_pin.copy_(h, non_blocking=True)
                else:
                    forward(x_dev)
                e1.record(stream)
                times.append((e0, e1))
        stream.synchronize()
        return [a.elapsed_time(b) for a, b in times]

    def timed_e2e(n):
        """n steps from host buffers: every step's input goes pinned host -> device and its result
        device -> pinned host inside the timed region; the copies run on side streams over two
        buffer sets so that step i+1's upload and step i-1's download overlap step i's kernels.
        Returns the total milliseconds between the first upload and the last download."""
        s_up, s_down = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
        stage = [torch.empty_like(x_stage) for _ in range(2)]
        outs = [torch.empty_like(out_pin, device=dev) for _ in range(2)]
        pins = [torch.empty_like(out_pin).pin_memory() for _ in range(2)]
        ev_up = [torch.cuda.Event() for _ in range(2)]
        ev_run = [torch.cuda.Event() for _ in range(2)]
        ev_down = [torch.cuda.Event() for _ in range(2)]
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        stream.synchronize()
        e0.record(stream)
        s_up.wait_event(e0)
        for i in range(n):
            b = i & 1
            with torch.cuda.stream(s_up):
                if i >= 2:
                    s_up.wait_event(ev_run[b])             # step i-2 has consumed this staging buffer
                stage[b].copy_(x_pin, non_blocking=True)
                ev_up[b].record(s_up)
            with torch.cuda.stream(stream):
                stream.wait_event(ev_up[b])
                if i >= 2:
                    stream.wait_event(ev_down[b])          # step i-2's result has left this output buffer
                forward(stage[b], final_out=outs[b])
                ev_run[b].record(stream)
            with torch.cuda.stream(s_down):
                s_down.wait_event(ev_run[b])
                pins[b].copy_(outs[b], non_blocking=True)
                ev_down[b].record(s_down)
        for b in range(2):
            stream.wait_event(ev_down[b])
        e1.record(stream)
        stream.synchronize()
        return e0.elapsed_time(e1)

    with torch.cuda.stream(stream):
        for _ in range(max(args.warmup, 3)):
            forward(x_dev)
    stream.synchronize()
    ctx.check()

    sampler = ClockSampler(local_rank)
    barrier()
    sampler.start()
    t_steps = timed_steps(args.steps)
    barrier()
    clocks = sampler.stop()
    ctx.check()
    total_ms = sum(t_steps)

    timed_e2e(3)
    barrier()
    total_e2e_ms = timed_e2e(args.steps)
    barrier()

    # per-kernel device time of the same steps (separate pass: event pairs around every launch)
    with torch.cuda.stream(stream):
        ctx.ibert_profile_begin()
        prof_steps = min(args.steps, 5)
        for _ in range(prof_steps):
            flush.fill_(1)
            forward(x_dev, eager=True)          # event pairs cannot be recorded into a graph replay
        prof = ctx.ibert_profile_end()
    ctx.check()

    # sustained leg: steps back to back (no L2 flush, no gaps) for at least --sustain seconds, clocks
    # and power sampled meanwhile -- what a serving loop would see once the power cap settles
    sustained = None
    if args.sustain > 0:
        est = max(total_ms / args.steps, 1e-3)
        chunk = max(1, int(250.0 / est))                    # ~0.25 s of work per host synchronization
        sus_sampler = ClockSampler(local_rank)
        barrier()
        sus_sampler.start()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n_sus = 0
        t_host = time.perf_counter()
        with torch.cuda.stream(stream):
            e0.record(stream)
            while time.perf_counter() - t_host < args.sustain or n_sus == 0:
                for _ in range(chunk):
                    forward(x_dev)
                n_sus += chunk
                stream.synchronize()
            e1.record(stream)
        stream.synchronize()
        sus_clocks = sus_sampler.stop()
        ctx.check()
        sus_ms = e0.elapsed_time(e1)
        sus_ms = dp.max_over_ranks([sus_ms], device=dev)[0]
        ms_step = sus_ms / n_sus
        mhz = sus_clocks.get("sm_mhz")
        n_computed = valid_tokens if (full_model and args.packed) else T
        sustained = {"value": n_computed * n_sus * world / (sus_ms / 1e3), "unit": UNIT, "steps": n_sus,
                     "seconds": sus_ms / 1e3, "ms_per_step": ms_step, "clocks": sus_clocks,
                     "ms_per_step_at_max_clock": (ms_step * mhz / SPEC_SM_MHZ) if mhz else None,
                     "how": "steps enqueued back to back without L2 flushes, one host synchronization every "
                            f"{chunk} steps; ms_per_step_at_max_clock = ms_per_step x median SM MHz / {SPEC_SM_MHZ:.0f}"}
    barrier()

    total_ms, total_e2e_ms = dp.max_over_ranks([total_ms, total_e2e_ms], device=dev)

    if rank == 0:
        peaks, peak_kind = measured_peaks()
        probes = probe_peaks()
        figures = ncu_figures()
        n_sms = torch.cuda.get_device_properties(dev).multi_processor_count
        sm_mhz_max = clocks.get("sm_max_mhz") or SPEC_SM_MHZ
        # padded batches: every position is computed and counted; packed batches: only real tokens exist
        computed = valid_tokens if (full_model and args.packed) else T
        work = algorithmic_work(cfg.H, cfg.F, cfg.L, cfg.heads, computed)
        # Peaks.  A kernel timed by an event pair inside a step of a few milliseconds runs at burst
        # clocks, so the tensor peak is 2 x the BURST bf16 cuBLAS rate (int8 : bf16 dense = 2 nominal).
        int8_peak = 2.0 * peaks["bf16_tflops"]
        # integer issue: 128 lane-operations per clock and SM over both integer pipes, 64 on the ALU pipe
        # alone (shifts, min / max, selects, permutes: the pipe the epilogues and i-softmax saturate first)
        issue_lanes = probes.get("int32_lane_ops_per_clk_sm", 128.0)
        alu_lanes = probes.get("alu_pipe_lane_ops_per_clk_sm", 64.0)
        issue_peak = issue_lanes * n_sms * sm_mhz_max * 1e6 / 1e12          # T lane-operations / s
        alu_peak = alu_lanes * n_sms * sm_mhz_max * 1e6 / 1e12
        alu_source = (f"{alu_lanes:.0f} lane-operations per clock and SM on the ALU pipe x SMs x max SM clock "
                      f"({'measured by the issue probe, profiles/issue_probes.md' if probes else 'unit count; probe summary absent'})")
        kern = {}
        prof_total = sum(v[0] for v in prof.values())
        for k, (ms, n) in prof.items():
            if n == 0:
                continue
            per = ms / n
            w = work.get(k, {"ops": 0.0, "bytes": 0.0})
            tops = w["ops"] / per / 1e9 if w["ops"] else None
            gbs = w["bytes"] / per / 1e6
            kern[k] = {"launches_per_step": n // prof_steps, "ms_per_launch": per, "share": ms / prof_total,
                       "tops": tops, "gbs": gbs,
                       "frac_tensor": (tops / int8_peak) if tops and k != "attention" else None,
                       "frac_hbm": gbs / peaks["hbm_gbs"]}
            fig = figures.get((k, args.config, batch))
            if fig:
                kern[k]["ncu_dram_bytes"] = fig["dram_bytes"]
                kern[k]["frac_alu_pipe"] = fig["alu"] * 32.0 / (per * 1e-3) / (alu_peak * 1e12)
                kern[k]["frac_int32_issue"] = (fig["alu"] + fig["fma"]) * 32.0 / (per * 1e-3) / (issue_peak * 1e12)
        top = max(kern, key=lambda k: kern[k]["share"])
        fig = figures.get((top, args.config, batch))
        if top == "attention":
            # i-softmax dominates: lane-operations on the ALU pipe per launch (ncu count when a capture of
            # this workload is committed, else 11 per score element, the count of the config-2 capture)
            lane_ops = fig["alu"] * 32.0 if fig else 11.0 * computed * cfg.L * cfg.heads
            ach = lane_ops / (kern[top]["ms_per_launch"] * 1e-3) / 1e12
            roof = {"kernel": top, "bound": "alu", "achieved": ach, "peak": alu_peak,
                    "unit": "Tinstr/s (int32 lane-ops on the ALU pipe)", "frac": ach / alu_peak, "peak_source": alu_source,
                    "algorithmic": lane_ops,
                    "algorithmic_source": "ncu ALU-pipe instructions of the committed capture x 32" if fig else
                                          "11 ALU-pipe lane-ops per score element (no ncu capture of this workload committed)"}
        elif work[top]["ops"]:
            roof = {"kernel": top, "bound": "tensor", "achieved": kern[top]["tops"], "peak": int8_peak,
                    "unit": "TOP/s", "frac": kern[top]["tops"] / int8_peak,
                    "peak_source": f"2 x {peak_kind} BURST bf16 cuBLAS rate (int8 dense = 2 x bf16 nominal); the "
                                   "kernel is event-timed inside a millisecond-scale step",
                    "frac_vs_spec": kern[top]["tops"] / SPEC_INT8_TOPS,
                    "frac_vs_sustained_peak": kern[top]["tops"] / (2.0 * peaks["bf16_tflops_sustained"]),
                    "algorithmic": work[top]["ops"]}
            if probes.get("i8_mma_tops"):
                roof["frac_vs_mma_issue_probe"] = kern[top]["tops"] / probes["i8_mma_tops"]
        else:
            roof = {"kernel": top, "bound": "hbm", "achieved": kern[top]["gbs"], "peak": peaks["hbm_gbs"],
                    "unit": "GB/s", "frac": kern[top]["gbs"] / peaks["hbm_gbs"],
                    "peak_source": f"{peak_kind} copy bandwidth", "algorithmic": work[top]["bytes"]}
        roof["ms_per_launch"] = kern[top]["ms_per_launch"]
        if fig and top != "attention":
            lane_ops = fig["alu"] * 32.0
            roof["integer_datapath"] = {"alu_lane_ops_per_launch": lane_ops, "peak_lane_ops_per_s": alu_peak * 1e12,
                                        "frac": lane_ops / (kern[top]["ms_per_launch"] * 1e-3) / (alu_peak * 1e12),
                                        "peak_source": alu_source,
                                        "note": "the epilogue's work on the ALU pipe (ncu count of the committed capture) "
                                                "against that pipe's issue rate: the bound this kernel actually runs into"}
        roof["traffic"] = fig["dram_bytes"] if fig else None
        roof["traffic_unit"] = ("bytes per launch (ncu dram__bytes_read.sum + dram__bytes_write.sum, "
                                "profiles/ncu_figures.md)")
        tokens = computed * args.steps * world
        value = tokens / (total_ms / 1e3)
        e2e_value = tokens / (total_e2e_ms / 1e3)

        # CPU baseline: the oracle on the first sequences of the same batch -- timed, and compared with
        # the rows the GPU produced for those sequences
        # (single-GPU runs only: with more ranks the others would sit in the teardown meanwhile)
        cpu = parity = None
        if world == 1:
            n_seq = min(8, batch)
            with torch.cuda.stream(stream):
                got_dev = forward(x_dev, eager=True)
            stream.synchronize()
            ctx.check()
            if full_model:
                want, dt_s, n_layers = oracle_on_sample(n_seq, cfg.L, model=m)
                got = got_dev[:n_seq].cpu().numpy()
            else:
                want, dt_s, n_layers = oracle_on_sample(n_seq, cfg.L, x=x_np, params=params)
                got = got_dev[:n_seq * cfg.L].cpu().numpy()
            tok_s = n_seq * cfg.L
            import oracle
            cpu = {"value": tok_s / dt_s, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                   "sample": f"first {n_seq} sequences ({tok_s} tokens) of the GPU's batch through "
                             f"{'embedding, ' if full_model else ''}all {n_layers} layers"
                             f"{' and the classifier' if full_model else ''}, {dt_s:.1f} s"}
            parity = {"tokens": tok_s, "values": int(want.size),
                      "mismatches": int((got.reshape(-1) != np.asarray(want).reshape(-1)).sum()) if got.size == want.size else -1,
                      "against": "CPU oracle on the same int8 inputs and parameters, element by element"}

        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": total_ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
            "config": workload_config(cfg, batch, world, full_model, valid_tokens / T,
                                      args.graph and not full_model, args.pow2_scores and not full_model, args.scales,
                                      full_model and args.packed),
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": x_pin.numel() * x_pin.element_size(),
                    "d2h_bytes_per_step": out_pin.numel() * out_pin.element_size(),
                    "ms_per_step": total_e2e_ms / args.steps,
                    "how": "pinned host -> device upload and device -> pinned host download of every step inside "
                           "the timed region, on side streams over two buffer sets (overlapping the neighbouring "
                           "steps' kernels); no L2 flush: each step's input arrives from host memory"},
            "gpu_launches": sum(v["launches_per_step"] for v in kern.values()) * args.steps,
            "roofline": roof,
            "sustained": sustained,
            "valid_tokens_per_s": valid_tokens * args.steps * world / (total_ms / 1e3),
            "parity": parity,
            "kernels": kern,
            "cpu_baseline": cpu,
        }
        print(json.dumps(line))
    if not full_model:
        for g in graphs.values():
            g.close()
    for ly in layers:
        ly.close()
    ctx.close()
    if dist is not None:
        dist.destroy_process_group()


def run_only(args):
    """Runs ONE kernel class alone through its C-ABI entry point at the workload's shape
    (for ncu captures and per-kernel timing).  Prints a small JSON line."""
    import numpy as np
    import torch

    from paper_2101_01321_b200 import binding, build, synth

    build.build()
    cfg = synth.CONFIGS[args.config]
    if args.seq_len:
        import dataclasses
        cfg = dataclasses.replace(cfg, L=args.seq_len)
    batch = args.batch or DEFAULT_BATCH[args.config]
    T, H, F, L = batch * cfg.L, cfg.H, cfg.F, cfg.L
    dev = torch.device("cuda", 0)
    stream = torch.cuda.Stream(device=dev)
    ctx = binding.Context(0, stream)
    g = torch.Generator(device="cpu").manual_seed(synth.SEED_BASE)

    def i8(*shape):
        return torch.randint(-127, 128, shape, generator=g, dtype=torch.int8).to(dev)

    p = synth.static_activation_scales(H, F, L, 0.035)
    rng = np.random.default_rng(synth.SEED_BASE)
    k = args.only
    alg_bytes = None
    if k == "layer":
        # one encoder layer through the call the step makes: its five kernels in the forms the layer
        # chooses (internal layouts included), for captures that select a kernel by name and launch index
        x_np, params = synth.make_model(args.config, batch, scales=args.scales)
        layer = ctx.ibert_layer_create(params[0])
        x = torch.from_numpy(x_np).to(dev)
        out = torch.empty_like(x)
        fn = lambda: ctx.ibert_encoder_layer(layer, x, batch, L, out=out)
    elif k in ("gemm_out_ln", "gemm_ffn2_ln"):
        N, K = (H, H) if k == "gemm_out_ln" else (H, F)
        x, w, res = i8(T, K), i8(N, K), i8(T, N)
        bias = torch.randint(-1000, 1000, (N,), generator=g, dtype=torch.int32).to(dev)
        S_w = rng.uniform(5e-4, 7e-4, N)
        S_x = 0.03
        S_acc = S_x * 6e-4 * 127 * 127 * np.sqrt(K)
        gamma, beta = 1.0 + 0.1 * rng.standard_normal(N), 0.1 * rng.standard_normal(N)
        out = torch.empty((T, N), dtype=torch.int8, device=dev)
        fn = lambda: ctx.ibert_linear_layernorm_i8(x, S_x, w, S_w, bias, 8 * S_acc / 32767, res, S_acc / 127,
                                                   gamma, beta, 4.5 / 127, out=out)
    elif k.startswith("gemm"):
        N, K = {"gemm_qkv": (3 * H, H), "gemm_out": (H, H), "gemm_ffn1_gelu": (F, H), "gemm_ffn1_hgelu": (F, H),
                "gemm_ffn2": (H, F)}[k]
        x, w = i8(T, K), i8(N, K)
        bias = torch.randint(-1000, 1000, (N,), generator=g, dtype=torch.int32).to(dev)
        S_w = rng.uniform(5e-4, 7e-4, N)
        S_x = 0.03
        S_acc = S_x * 6e-4 * 127 * 127 * np.sqrt(K)           # ~ one standard deviation of the product
        if k == "gemm_ffn1_gelu":
            out = torch.empty((T, N), dtype=torch.int8, device=dev)
            fn = lambda: ctx.ibert_linear_gelu_i8(x, S_x, w, S_w, bias, 8 * S_acc / 32767, 4 * S_acc / 127, out=out)
        elif k == "gemm_ffn1_hgelu":
            out = torch.empty((T, N), dtype=torch.int8, device=dev)
            fn = lambda: ctx.ibert_linear_hgelu_i8(x, S_x, w, S_w, bias, 8 * S_acc / 32767, 4 * S_acc / 127, out=out)
        elif k == "gemm_qkv":
            out = torch.empty((T, N), dtype=torch.int8, device=dev)
            fn = lambda: ctx.ibert_linear_i8(x, S_x, w, S_w, bias, 0, 4 * S_acc / 127, out=out)
        else:
            out = torch.empty((T, N), dtype=torch.int32, device=dev)
            fn = lambda: ctx.ibert_linear_i8(x, S_x, w, S_w, bias, 1, 8 * S_acc / 32767, out=out)
    elif k == "attention":
        qkv = torch.clamp(torch.randn((T, 3 * H), generator=g) * 32, -127, 127).to(torch.int8).to(dev)
        out = torch.empty((T, H), dtype=torch.int8, device=dev)
        fn = lambda: ctx.ibert_attention_i8(qkv, batch, L, H, cfg.heads, p["S_q"], p["S_k"], p["S_v"], p["S_ctx"], 255, out=out)
    elif k in ("layernorm", "layernorm_i16"):
        q, S, r, S_r, gamma, beta, S_out = synth.layernorm_inputs(T, H, 1.0)
        qd, rd = torch.from_numpy(q.astype(np.int16) if k == "layernorm_i16" else q).to(dev), torch.from_numpy(r).to(dev)
        out = torch.empty((T, H), dtype=torch.int8, device=dev)
        fn = lambda: ctx.ibert_layernorm_i(qd, S, rd, S_r, gamma, beta, S_out, out=out)
        alg_bytes = T * H * ((2 if k == "layernorm_i16" else 4) + 1 + 1)
    elif k in ("gelu", "hgelu", "gelu_lut"):
        q, S, S_out = synth.gelu_inputs(1 << 24, 1.0)
        qd = torch.from_numpy(q).to(dev)
        out = torch.empty(q.shape, dtype=torch.int8, device=dev)
        alg_bytes = q.size * 5
        fn = {"gelu": lambda: ctx.ibert_gelu_i(qd, S, S_out, out=out),
              "hgelu": lambda: ctx.ibert_hgelu_i(qd, S, S_out, out=out),
              "gelu_lut": lambda: ctx.ibert_gelu_lut_i(qd, S, S_out, out=out)}[k]
    elif k in ("softmax", "softmax_lut"):
        rows = batch * cfg.heads * L
        q, S = synth.softmax_inputs(rows, L, 1.0)
        qd = torch.from_numpy(q).to(dev)
        out = torch.empty(q.shape, dtype=torch.uint8, device=dev)
        alg_bytes = q.size * 5
        fn = (lambda: ctx.ibert_softmax_i(qd, S, 255, out=out)) if k == "softmax" else \
             (lambda: ctx.ibert_softmax_lut_i(qd, S, 255, out=out))
    else:
        raise SystemExit(f"unknown kernel class {k}")
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
    times = []
    with torch.cuda.stream(stream):
        for _ in range(max(args.warmup, 1)):
            fn()
        for _ in range(args.steps):
            flush.fill_(1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            fn()
            e1.record(stream)
            times.append((e0, e1))
    stream.synchronize()
    ctx.check()
    ms = [a.elapsed_time(b) for a, b in times]
    line = {"only": k, "tokens": T, "ms_median": statistics.median(ms), "ms_min": min(ms), "launches": args.steps}
    if alg_bytes:
        peaks, peak_kind = measured_peaks()
        gbs = alg_bytes / statistics.median(ms) / 1e6
        line["roofline"] = {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                            "frac": gbs / peaks["hbm_gbs"], "algorithmic": alg_bytes,
                            "peak_source": f"{peak_kind} copy bandwidth; the time includes the event pair (about 5 us)"}
    print(json.dumps(line))
    ctx.close()


def spawn_ranks(n: int, argv: list[str]) -> int:
    """`bench.py --gpus N` started as a plain process: re-launches itself as N ranks (one per GPU)
    through torch.distributed.run on this node and returns that launcher's exit code."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), str(Path(__file__).resolve()), *argv]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--config", type=int, default=2, choices=[2, 3, 4])
    ap.add_argument("--batch", type=int, default=0)
    ap.add_argument("--seq-len", type=int, default=0, help="override the config's sequence length (latency grids)")
    ap.add_argument("--pow2-scores", action="store_true",
                    help="layers workload: query scales raised so that every score scale is ln2 / 2^k "
                         "(i-exp quotient by shift and mask)")
    ap.add_argument("--fusion", type=int, default=0, choices=[0, 1, 2],
                    help="linear + LayerNorm: 0 by problem size (default), 1 cluster kernel whenever supported, 2 never")
    ap.add_argument("--graph", action="store_true",
                    help="layers workload: replay the forward pass from a captured CUDA graph (ibert_encoder_graph_*)")
    ap.add_argument("--workload", choices=["layers", "model"], default="layers",
                    help="layers: the encoder layers on full-length sequences (headline); model: token ids -> "
                         "embedding -> layers with a key-padding mask on a sentence-length mix -> classifier")
    ap.add_argument("--packed", action="store_true",
                    help="model workload: the same sentence-length mix stored without padding (cu_seqlens); "
                         "tokens/s then counts real tokens only")
    ap.add_argument("--only", default="", help="run one kernel class alone (profiling aid)")
    ap.add_argument("--sustain", type=float, default=3.0,
                    help="seconds of back-to-back steps for the sustained-clock leg (0 = skip)")
    ap.add_argument("--scales", choices=["analytic", "calibrated"], default="calibrated",
                    help="static activation scales: closed-form from the input distributions, or the blob "
                         "calibrated with the CPU oracle (tests/golden/calibrated_scales.json)")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and not args.only:
        raise SystemExit(spawn_ranks(args.gpus, sys.argv[1:]))
    if args.only:
        run_only(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
