#!/usr/bin/env python
"""Benchmark of the fused dictionary-decode + GEMV path (one JSON line on stdout).

A step is one pass over every linear layer of one LLaMA-3.2-3B decode step at batch 1: 197 products in
ONE persistent launch (tq_fused_gemv_stack), replayed as a CUDA graph.  Weights are seeded synthetic
Student-t values, quantized per row to int8, dictionary-coded with one table for the whole model and
tiled on the GPU, resident in HBM before the timed region starts.  `value` is the effective bandwidth
on algorithmic bytes (tokens and raw words of the layout + tile index + row scales + x + y) per second.
Extra keys time the same model at 8 and 32 vectors, launched as a decoder must launch it (layers that
feed one another in separate launches), the 1B stack, tq_decompress of the whole set and the prefill
product at 2048 tokens; `e2e` is the same step through the host-buffer call (x from pinned host memory, y back
to it, every step: as one call and as a few calls on two streams); `cpu_baseline` is the CPU oracle on the host's cores.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--model 3b|1b] [--batch B] [--layers L]
  python bench.py --impl reference ...     # the CPU oracle on a bounded sample of the workload
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

from inputs import synth  # noqa: E402

METRIC = "fused_decode_gemv_effective_bandwidth"
UNIT = "GB/s"


def log(*a):
    print(*a, file=sys.stderr, flush=True)


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            j = json.load(f)
        return float(j["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.lines: list[str] = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def wait_first(self, timeout=5.0):
        t0 = time.time()
        while not self.lines and time.time() - t0 < timeout and self.proc is not None:
            time.sleep(0.02)

    def stop(self, t_start=0.0, t_end=float("inf")):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for ts, ln in self.lines:
            if ts < t_start or ts > t_end:
                continue
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel from the ncu capture
# summarised under profiles/ (None: not captured for that launch shape, or kernel changed since).
# tiles_stack: 219.7 MB read + 6.8 MB written for 207.7 MB of algorithmic bytes on a 14-matrix stack (2 decoder
# layers), i.e. 1.090 x; traffic grows with the bytes streamed, so the 3B launch (3.36 GB) is scaled by that ratio.
L2_BYTES = 126 << 20
E2E_GROUPS = 4  # host-buffer calls per step of the pipelined end-to-end leg
TRAFFIC_RATIO = {"tiles_stack": 1.090}
TRAFFIC = {}
# the arithmetic each layout's product kernel computes in
DTYPE = {"tiles": "s8 x s8 -> s32 (int8 levels x four base-256 digits of block-fixed-point bf16 activations, "
                  "exact integer tensor-core sums, fp64 epilogue)",
         "planes": "int8 weights x bf16 activations, fp32 accumulate",
         "stream": "int8 weights x bf16 activations, fp32 accumulate"}


def build_model(tq, shapes, batch, device, threads=0, table_entries=None, layout=1, quantizer="rows", bits=8):
    """Generate, quantize, build the table and encode (host), upload.  quantizer "rows": per-row
    symmetric int8 on the GPU (the workload definition); "paper": Listing 1, one scale and zero point
    per tensor, unsigned levels (host).  Returns (matrices, xs, ys, table, ...)."""
    t0 = time.time()
    if threads:
        tq.tq_set_num_threads(threads)
    q_host, scales, zeros = [], [], []
    q_dev, s_dev = [], []  # levels and scales kept on the device for the device-side encoder (tiles layout)
    on_device = layout == 2 and quantizer == "rows"
    for i, (name, rows, cols) in enumerate(shapes):
        w = synth.weight(rows, cols, synth.matrix_seed(i), device=device)
        if quantizer == "paper":
            q, s, z = tq.tq_quantize_tensor_bits(w.cpu().numpy(), bits)
            q_host.append(q.reshape(rows, cols))
            scales.append(np.full(rows, s, dtype=np.float32))
            zeros.append(np.full(rows, z, dtype=np.float32))
        else:
            q, s = tq.tq_quantize_rows_device(w)
            q_host.append(q.cpu().numpy())
            scales.append(s.cpu().numpy())
            zeros.append(None)
            if on_device:
                q_dev.append(q)
                s_dev.append(s)
        del w, q, s
    t1 = time.time()
    if table_entries is not None:
        hd = tq.tq_dict_from_entries(table_entries)
    elif on_device:  # windows counted on the GPU, candidates ranked on the host: the same table
        hd = tq.tq_build_dictionary_device([q.view(-1) for q in q_dev])
    else:
        hd = tq.tq_build_dictionary(q_host)
    t2 = time.time()
    dd = tq.tq_dict_upload(hd, device=device)
    mats = []
    for i, (name, rows, cols) in enumerate(shapes):
        if on_device:  # Listing 3 and the tiling on the GPU, no host stream
            mats.append(tq.tq_upload_device(dd, q_dev[i], s_dev[i]))
            q_dev[i] = s_dev[i] = None
            continue
        stream, h, m = tq.tq_encode(hd, q_host[i])
        mats.append(tq.tq_upload(dd, stream, rows, cols, scales[i], zeros[i], levels_signed=(quantizer != "paper"),
                                 layout=layout))
        del stream
    t3 = time.time()
    # all x in one arena and all y in another (16-byte aligned pieces), so that the end-to-end
    # path moves each with one copy
    xoff, yoff, xo, yo = [], [], 0, 0
    for (_, rows, cols) in shapes:
        xoff.append(xo)
        yoff.append(yo)
        xo += -(-batch * cols // 8) * 8
        yo += -(-batch * rows // 4) * 4
    x_arena = torch.zeros(xo, dtype=torch.bfloat16, device=device)
    y_arena = torch.zeros(yo, dtype=torch.float32, device=device)
    xs, ys = [], []
    for i, (_, rows, cols) in enumerate(shapes):
        x = x_arena[xoff[i]: xoff[i] + batch * cols].view(batch, cols)
        x.copy_(synth.activations(batch, cols, 7000 + i, device=device))
        xs.append(x)
        ys.append(y_arena[yoff[i]: yoff[i] + batch * rows].view(batch, rows))
    stats = {"gen_quant_s": t1 - t0, "table_s": t2 - t1, "encode_upload_s": t3 - t2, "K": hd.K}
    return mats, xs, ys, hd, q_host, scales, stats, x_arena, y_arena, dd


def algorithmic_bytes(info, batch):
    """Bytes the method has to move for one call: the tokens and raw words of the layout in use
    (for tiles: with the table limited to what shared memory holds), its index, the row scale, x
    and y.  Padding is not counted."""
    if info.layout == 0:   # paper stream: 2 bytes per code, 10 per escaped group
        tokens = info.stream_bytes
    else:                  # planes / tiles: one 2-byte token per group + one 4-byte word per raw group
        tokens = 2 * (info.n_hits + info.n_miss) + 4 * info.n_raw_words
    if info.layout == 2:   # tiles: a 4-byte raw-stream index per tile of 16 rows x 128 columns
        index = 4 * (-(-info.rows // 16) * -(-info.cols // 128) + 1)
    else:
        index = 8 * info.rows
    return tokens + index + 4 * info.rows + 2 * batch * info.cols + 4 * batch * info.rows


def oracle_sample_run(hd_entries, q_host, scales, shapes, batch, sample_idx, reps=1, workers=1, decode_only=False):
    """The CPU oracle on a bounded sample: Listing 4 decode + fp64 layer product per matrix.
    Streams are produced beforehand by the oracle's own encoder (untimed).  The oracle itself is
    single-threaded plain C; with workers > 1 the matrices of the sample are dealt to that many
    Python threads (the ctypes calls release the interpreter lock), each running the unchanged
    oracle on its share.  Returns (algorithmic bytes of the sample, [wall seconds per repetition],
    [wall seconds of the decode alone per repetition])."""
    from concurrent.futures import ThreadPoolExecutor
    from oracle import oracle
    od = oracle.Dictionary.from_entries(hd_entries)
    workers = max(1, min(workers, len(sample_idx)))
    order = sorted(sample_idx, key=lambda i: -shapes[i][1] * shapes[i][2])
    shares = [[] for _ in range(workers)]
    load = [0] * workers
    for i in order:  # largest first, each to the least loaded worker
        w = load.index(min(load))
        shares[w].append(i)
        load[w] += shapes[i][1] * shapes[i][2]
    pool = ThreadPoolExecutor(workers)

    def encode_share(share):
        return {i: od.encode(q_host[i]) for i in share}
    enc = {}
    for part in pool.map(encode_share, shares):
        enc.update(part)
    xs = {i: synth.activations(batch, shapes[i][2], 7000 + i).double().numpy() for i in sample_idx}
    total = sum(2 * (enc[i][1] + 5 * enc[i][2]) + shapes[i][1] * 12 + 2 * batch * shapes[i][2] + 4 * batch * shapes[i][1]
                for i in sample_idx)

    def run_share(args):
        share, with_product = args
        for i in share:
            _, rows, cols = shapes[i]
            codes = od.decode(enc[i][0], rows * cols).reshape(rows, cols).view(np.int8)
            if with_product:
                oracle.layer_forward(codes, scales[i], xs[i])
    times, dec_times = [], []
    for r in range(reps):
        t0 = time.perf_counter()
        list(pool.map(run_share, [(sh, True) for sh in shares]))
        times.append(time.perf_counter() - t0)
        if decode_only:
            t0 = time.perf_counter()
            list(pool.map(run_share, [(sh, False) for sh in shares]))
            dec_times.append(time.perf_counter() - t0)
    pool.shutdown()
    return total, times, dec_times


def time_stack(tq, stack, stream, reps, warmup=3):
    """ms per tq_fused_gemv_stack call, replayed as a CUDA graph, CUDA events on the launching stream."""
    with torch.cuda.stream(stream):
        tq.tq_fused_gemv_stack(stack)  # kernel attributes are set outside the capture
        stream.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            tq.tq_fused_gemv_stack(stack)
        for _ in range(warmup):
            g.replay()
        stream.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(reps):
            g.replay()
        e1.record(stream)
        stream.synchronize()
    return e0.elapsed_time(e1) / reps


def batch_operands(shapes, batch, device):
    xs = [synth.activations(batch, cols, 7000 + i, device=device) for i, (_, rows, cols) in enumerate(shapes)]
    ys = [torch.zeros((batch, rows), dtype=torch.float32, device=device) for _, rows, cols in shapes]
    return xs, ys


def time_extras(tq, mats, infos, shapes, args, device, stream, extra):
    """Standalone tq_decompress of the whole weight set and the prefill product (tq_fused_gemm) at
    M tokens, timed with CUDA events on the launching stream (3 warm-ups, inputs far larger than L2)."""
    out = {}
    n_weights = sum(i.rows * i.cols for i in infos)
    max_elems = max(i.rows * i.cols for i in infos)
    buf = torch.empty(max_elems, dtype=torch.uint8, device=device)

    if args.layout == "tiles" and not args.per_layer:  # one persistent launch, every matrix to its own buffer
        del buf
        big = torch.empty(n_weights, dtype=torch.uint8, device=device)
        outs, o = [], 0
        for i in infos:
            outs.append(big[o: o + i.rows * i.cols])
            o += i.rows * i.cols
        dstack = tq.tq_stack_create(mats)

        def run_dec():
            tq.tq_decompress_stack(dstack, outs)
    else:
        def run_dec():
            for m in mats:
                tq.tq_decompress(m, buf[: m.info.rows * m.info.cols])

    def timed(fn, reps):
        for _ in range(3):
            fn()
        stream.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(reps):
            fn()
        e1.record(stream)
        stream.synchronize()
        return e0.elapsed_time(e1) / reps

    ms = timed(run_dec, 10)
    rd = sum(algorithmic_bytes(i, 0) for i in infos)
    out["decompress"] = {"ms": ms, "GB_per_s": (rd + n_weights) / (ms * 1e-3) / 1e9,
                         "launch": "one persistent launch (tq_decompress_stack)" if args.layout == "tiles" and not args.per_layer
                         else "one launch per matrix (tq_decompress)",
                         "bytes": {"read": rd, "written": n_weights},
                         "frac_of_measured_hbm": (rd + n_weights) / (ms * 1e-3) / 1e9 / measured_peaks()[0]}
    if args.layout == "tiles" and not args.per_layer and not args.shapes and "xs" in extra:
        # The same products launched the way a decoder with real data dependencies could launch them:
        # one stack per set of layers that may run together ({q,k,v}, {o}, {gate,up}, {down} per decoder
        # layer, then the output head), replayed as one CUDA graph.  Every launch reloads the table.
        names = [n.split(".")[-1] for n, _, _ in shapes]
        sets, cur, last = [], [], None
        kind = {"q": 0, "k": 0, "v": 0, "o": 1, "gate": 2, "up": 2, "down": 3, "lm_head": 4}
        for i, n in enumerate(names):
            k = kind.get(n, 5)
            if cur and k != last:
                sets.append(cur)
                cur = []
            cur.append(i)
            last = k
        sets.append(cur)
        dep_stacks = [tq.tq_stack_create([mats[i] for i in g], [extra["xs"][i] for i in g], [extra["ys"][i] for i in g])
                      for g in sets]

        def run_dep():
            for st in dep_stacks:
                tq.tq_fused_gemv_stack(st)

        run_dep()
        stream.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            run_dep()
        ms = timed(g.replay, 20)
        alg = sum(algorithmic_bytes(i, args.batch) for i in infos)
        out["dependent_launches"] = {"launches_per_token": sum(s_.launches for s_ in dep_stacks), "ms": ms,
                                     "GB_per_s": alg / (ms * 1e-3) / 1e9,
                                     "frac_of_measured_hbm": alg / (ms * 1e-3) / 1e9 / measured_peaks()[0],
                                     "grouping": "{q,k,v} {o} {gate,up} {down} per decoder layer, then the output head"}
        del dep_stacks, g
    if args.layout == "tiles" and not args.per_layer and not args.shapes and "xs" in extra and args.batch == 1 and args.model == "3b":
        # the other batch sizes of the same workload (one pass of the tcgen05 kernel over all 197 matrices) ...
        peak = measured_peaks()[0]
        for b in (8, 32):
            xs_b, ys_b = batch_operands(shapes, b, device)
            st_b = tq.tq_stack_create(mats, xs_b, ys_b)
            ms_b = time_stack(tq, st_b, stream, 100)
            alg_b = sum(algorithmic_bytes(i, b) for i in infos)
            out["batch%d" % b] = {"workload": f"llama3.2-3b linear stack ({len(mats)} matrices), batch {b}", "ms": ms_b,
                                  "launches": st_b.launches, "GB_per_s": alg_b / (ms_b * 1e-3) / 1e9,
                                  "frac_of_measured_hbm": alg_b / (ms_b * 1e-3) / 1e9 / peak,
                                  "us_per_token": ms_b * 1e3 / b, "kernel": "wide_prepare_kernel + gemv_wide_kernel"}
            del st_b, xs_b, ys_b
        # ... and the LLaMA-3.2-1B stack at batch 1, with its own table
        shapes1 = synth.llama32_linear_shapes("1b")
        m1, xs1, ys1, hd1, _, _, _, _, _, _ = build_model(tq, shapes1, 1, device, 0, None, layout=2)
        st1 = tq.tq_stack_create(m1, xs1, ys1)
        ms1 = time_stack(tq, st1, stream, 300)
        alg1 = sum(algorithmic_bytes(m.info, 1) for m in m1)
        out["llama1b_batch1"] = {"workload": f"llama3.2-1b linear stack ({len(m1)} matrices), batch 1", "ms": ms1, "us_per_token": ms1 * 1e3,
                                 "launches": st1.launches, "algorithmic_bytes": alg1, "GB_per_s": alg1 / (ms1 * 1e-3) / 1e9,
                                 "frac_of_measured_hbm": alg1 / (ms1 * 1e-3) / 1e9 / peak, "K": hd1.K}
        del st1, m1, xs1, ys1, hd1
        torch.cuda.empty_cache()
    if args.layout != "stream":
        M = args.prefill_tokens
        max_rows = max(i.rows for i in infos)
        Y = torch.empty(M * max_rows, dtype=torch.float32, device=device)
        Xs = {c: synth.activations(M, c, 99, device=device) for c in sorted({i.cols for i in infos})}
        if args.layout == "tiles":
            # phase 1 for a group of decoder layers (7 matrices each) in one launch, then all their tensor-core
            # products in one persistent launch (tq_gemm_plan: the tiles of all products in one sequence)
            per_group = 7 * max(1, args.prefill_layers_per_launch)
            groups = [list(range(i, min(i + per_group, len(mats)))) for i in range(0, len(mats), per_group)]
            n_slots = max(len(g) for g in groups)
            slot_bytes = [max(tq.tq_gemm_workspace_size(mats[g[k]]) for g in groups if k < len(g)) for k in range(n_slots)]
            slot_rows = [max(mats[g[k]].info.rows for g in groups if k < len(g)) for k in range(n_slots)]
            wsets = [[torch.empty(b, dtype=torch.uint8, device=device) for b in slot_bytes] for _ in range(2)]
            Yslots = [torch.empty(M * r, dtype=torch.float32, device=device) for r in slot_rows]  # reused by every group
            del Y
            gstacks = [tq.tq_stack_create([mats[i] for i in g]) for g in groups]
            plans = [tq.tq_gemm_plan_create([mats[i] for i in g], [Xs[mats[i].info.cols] for i in g], wsets[gi % 2][: len(g)],
                                            [Yslots[k][: M * mats[i].info.rows].view(M, mats[i].info.rows) for k, i in enumerate(g)])
                     for gi, g in enumerate(groups)]

            # Weights do not depend on activations, so the decode of group g + 1 runs on a stream of its
            # own, ahead of the products of group g: two workspace sets alternate.
            dec_stream = torch.cuda.Stream(device)
            ev_dec = [torch.cuda.Event() for _ in groups]
            ev_used = [torch.cuda.Event() for _ in groups]   # the products of a group have read its workspaces
            ev_start, ev_end = torch.cuda.Event(), torch.cuda.Event()

            def run_gemm():
                ev_start.record(stream)
                dec_stream.wait_event(ev_start)
                for gi, (g, st) in enumerate(zip(groups, gstacks)):
                    if gi >= 2:
                        dec_stream.wait_event(ev_used[gi - 2])
                    tq.tq_decode_bf16_stack(st, wsets[gi % 2][: len(g)], stream=dec_stream)
                    ev_dec[gi].record(dec_stream)
                    stream.wait_event(ev_dec[gi])
                    tq.tq_gemm_plan_run(plans[gi], stream=stream)
                    ev_used[gi].record(stream)
                ev_end.record(dec_stream)
                stream.wait_event(ev_end)
        else:
            def run_gemm():
                for m in mats:
                    tq.tq_fused_gemm(m, Xs[m.info.cols], Y[: M * m.info.rows].view(M, m.info.rows))

        ms = timed(run_gemm, 3)
        reps = max(3, int(1100.0 / ms) + 1)  # at least a second of timed work: the power cap has acted, the sustained peak is the denominator
        ms = timed(run_gemm, reps)
        flops = 2.0 * M * n_weights
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json"))) if os.path.exists(os.path.join(ROOT, "MEASURED_PEAKS.json")) else {}
        pk = float(peaks.get("bf16_tflops_sustained", 1400.0))
        pk_burst = float(peaks.get("bf16_tflops", 1590.0))
        ws_bytes = sum(sum(b for b in slot_bytes) for _ in range(2)) if args.layout == "tiles" else 0
        out["prefill"] = {"tokens": M, "ms": ms, "reps": reps, "timed_region_ms": ms * reps, "workspace_bytes": ws_bytes,
                          "frac_of_measured_bf16_burst": flops / (ms * 1e-3) / 1e12 / pk_burst,
                          "call": ("tq_decode_bf16_stack + tq_gemm_plan_run (TMA-fed tcgen05 GEMM over all products of the group) per %d decoder layer(s)" % max(1, args.prefill_layers_per_launch)) if args.layout == "tiles"
                          else "tq_fused_gemm (decode inside the GEMM)", "TFLOP_per_s": flops / (ms * 1e-3) / 1e12,
                          "frac_of_measured_bf16_sustained": flops / (ms * 1e-3) / 1e12 / pk, "peak_TFLOP_per_s": pk}
        status = 0
        for m in mats:
            status |= tq.tq_device_status(m)
        if args.layout == "tiles":
            for pl in plans:
                status |= tq.tq_gemm_plan_status(pl)
        assert status == 0, f"device status {status}"
    return out


def pick_sample(shapes, max_weights):
    idx, tot = [], 0
    for i, (_, r, c) in enumerate(shapes):
        if tot + r * c > max_weights and idx:
            break
        idx.append(i)
        tot += r * c
    return idx


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="tq", choices=["tq", "reference"])
    ap.add_argument("--model", default="3b", choices=["1b", "3b", "11b", "90b"])
    ap.add_argument("--bits", type=int, default=8, help="bit count of the per-tensor quantizer (--quantizer paper)")
    ap.add_argument("--quantizer", default="rows", choices=["rows", "paper"],
                    help="rows: per-row symmetric int8 (the workload definition); paper: Listing 1, per tensor, unsigned levels "
                         "with a zero point (a regime where nearly every group is in the table); single GPU, no CPU baseline")
    ap.add_argument("--batch", type=int, default=1)
    ap.add_argument("--layers", type=int, default=None, help="decoder layers to build (default: all)")
    ap.add_argument("--no-lm-head", action="store_true")
    ap.add_argument("--shapes", default=None, help="custom workload, e.g. 32768x3072,3072x8192 (profiling cases)")
    ap.add_argument("--layout", default="tiles", choices=["stream", "planes", "tiles"])
    ap.add_argument("--per-layer", action="store_true", help="tiles layout: one launch per matrix instead of one persistent launch for the stack")
    ap.add_argument("--no-graph", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--e2e-groups", type=int, default=E2E_GROUPS, help="host-buffer calls per step of the pipelined end-to-end leg")
    ap.add_argument("--no-extras", action="store_true", help="skip the tq_decompress / tq_fused_gemm timings")
    ap.add_argument("--shard", default="replicas", choices=["replicas", "rows"],
                    help="N > 1 GPUs: replicas = every rank runs the whole model (weak scaling, no collective); rows = every "
                         "matrix split by output rows over the ranks, one all-gather of the outputs per step (strong scaling)")
    ap.add_argument("--prefill-tokens", type=int, default=2048)
    ap.add_argument("--prefill-layers-per-launch", type=int, default=14, help="decoder layers per decode + GEMM launch pair of the prefill leg")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    shapes = synth.llama32_linear_shapes(args.model, args.layers, lm_head=not args.no_lm_head)
    workload = f"llama3.2-{args.model} linear stack ({len(shapes)} matrices), batch {args.batch}"
    if args.quantizer == "paper":
        workload += ", per-tensor quantizer of Listing 1" + ("" if args.bits == 8 else " at %d bits" % args.bits)
        assert int(os.environ.get("WORLD_SIZE", "1")) == 1 and not args.per_layer
    if args.shapes:
        shapes = [(f"m{i}", int(t.split("x")[0]), int(t.split("x")[1])) for i, t in enumerate(args.shapes.split(","))]
        workload = f"custom shapes {args.shapes}, batch {args.batch}"
    n_weights = sum(r * c for _, r, c in shapes)

    if args.impl == "reference":
        if rank != 0:
            return
        run_reference(args, shapes, workload)
        return

    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU fallback)"
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)
    from paper_2509_22951_b200 import binding as tq

    ncores = os.cpu_count() or 1
    threads = max(1, ncores // world)
    table_entries = None
    if world > 1:
        # the table is a property of the model: rank 0 builds it, the others receive the entries
        import torch.distributed as dist
        if rank == 0:
            q0 = []
            for i, (name, rows, cols) in enumerate(shapes):
                w = synth.weight(rows, cols, synth.matrix_seed(i), device=device)
                q0.append(tq.tq_quantize_rows_device(w)[0])
                del w
            # windows counted on the GPU, candidates ranked on the host: the same table as tq_build_dictionary
            ent = torch.from_numpy(np.ascontiguousarray(tq.tq_build_dictionary_device([q.view(-1) for q in q0]).entries)).to(device)
            del q0
            torch.cuda.empty_cache()
            meta = torch.tensor([ent.shape[0]], device=device)
        else:
            meta = torch.zeros(1, dtype=torch.int64, device=device)
        dist.broadcast(meta, 0)
        if rank != 0:
            ent = torch.empty((int(meta.item()), 4), dtype=torch.uint8, device=device)
        dist.broadcast(ent, 0)
        table_entries = ent.cpu().numpy()

    mats, xs, ys, hd, q_host, scales, stats, x_arena, y_arena, dd = build_model(tq, shapes, args.batch, device, threads, table_entries, layout={"stream": 0, "planes": 1, "tiles": 2}[args.layout], quantizer=args.quantizer, bits=args.bits)
    infos = [m.info for m in mats]
    hits = sum(i.n_hits for i in infos)
    miss = sum(i.n_miss for i in infos)
    alg_bytes = sum(algorithmic_bytes(i, args.batch) for i in infos)
    stream_bytes = sum(i.stream_bytes for i in infos)
    payload_bytes = sum(i.payload_bytes for i in infos)
    log(f"[rank {rank}] built {len(mats)} matrices, {n_weights/1e9:.3f} G weights, hit rate {hits/(hits+miss):.4f}, "
        f"stream {stream_bytes/1e9:.3f} GB, setup {stats}")

    if args.shard == "rows" and world > 1:
        run_row_sharded(tq, args, shapes, workload, device, rank, world, local_rank, dd, mats, scales, xs, alg_bytes, stats)
        return

    stream = torch.cuda.Stream(device)
    use_stack = args.layout == "tiles" and not args.per_layer
    hit_rate_device = 1.0 - sum(i.n_raw_words for i in infos) / (hits + miss)
    if use_stack:
        stack = tq.tq_stack_create(mats, xs, ys)
        launches_per_step = stack.launches

        def step_plain():
            tq.tq_fused_gemv_stack(stack)
    else:
        per_pass = 4 if args.layout != "tiles" else 32
        launches_per_step = len(mats) * (-(-args.batch // per_pass)) * (2 if args.layout == "tiles" and args.batch > 2 else 1)

        def step_plain():
            for m, x, y in zip(mats, xs, ys):
                tq.tq_fused_gemv(m, x, y)

    with torch.cuda.stream(stream):
        step_plain()  # sets kernel attributes before any capture
        stream.synchronize()
        graph = None
        if not args.no_graph:
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                step_plain()
        run_step = graph.replay if graph is not None else step_plain

        for _ in range(max(args.warmup, 3)):
            run_step()
        stream.synchronize()

        def barrier():
            if world > 1:
                import torch.distributed as dist
                dist.barrier()

        sampler = ClockSampler(local_rank)
        sampler.start()
        sampler.wait_first()
        barrier()
        torch.cuda.synchronize()
        t_start = time.time()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record(stream)
        for _ in range(args.steps):
            run_step()
        ev1.record(stream)
        stream.synchronize()
        ms_flushed = None
        if payload_bytes < 2 * L2_BYTES:
            # a workload that fits L2 would be read from L2 from the second step on: write a buffer larger
            # than L2 between steps and time every step on its own
            flush = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device=device)
            pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
            for a, b in pairs:
                flush.zero_()
                a.record(stream)
                run_step()
                b.record(stream)
            stream.synchronize()
            ms_flushed = sum(a.elapsed_time(b) for a, b in pairs)
            del flush
        torch.cuda.synchronize()
        t_end = time.time()
        barrier()
        extended = False
        if t_end - t_start < 0.6:  # too short for nvidia-smi's 100 ms period: keep the same load running, untimed
            extended = True
            while time.time() - t_start < 0.8:
                run_step()
                stream.synchronize()
            t_end = time.time()
        clocks = sampler.stop(t_start, t_end)
        clocks["sampled_over"] = "timed region" if not extended else "timed region plus identical untimed steps"
        ms_unflushed = ev0.elapsed_time(ev1) / args.steps
        ms_total = ev0.elapsed_time(ev1) if ms_flushed is None else ms_flushed

        status = 0
        for m in mats:
            status |= tq.tq_device_status(m)
        assert status == 0, f"device status {status}"

        # ---- end to end through the host-buffer call: H2D of x and D2H of y every step ----
        e2e = None
        if not args.no_e2e:
            hx = [x.cpu().pin_memory() for x in xs]
            hy = [torch.empty(y.shape, dtype=torch.float32).pin_memory() for y in ys]
            e_steps = max(3, min(args.steps, 10))

            if use_stack:
                hxa = x_arena.cpu().pin_memory()
                hya = torch.empty(y_arena.shape, dtype=torch.float32).pin_memory()

                def step_e2e():
                    tq.tq_fused_gemv_stack_host(stack, hxa, x_arena, hya, y_arena)
            else:
                def step_e2e():
                    for m, a, b, dx, dy in zip(mats, hx, hy, xs, ys):
                        tq.tq_fused_gemv_host(m, a, b, dx, dy)

            def time_e2e(step_fn):
                for _ in range(3):
                    step_fn()
                stream.synchronize()
                barrier()
                t0 = time.perf_counter()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                for _ in range(e_steps):
                    step_fn()
                    stream.synchronize()  # the step's result is on the host
                e1.record(stream)
                stream.synchronize()
                wall = time.perf_counter() - t0
                return max(e0.elapsed_time(e1), wall * 1e3) / e_steps

            e2e_ms = time_e2e(step_e2e)
            e2e = {"ms_per_step": e2e_ms, "steps": e_steps,
                   "h2d": sum(2 * args.batch * i.cols for i in infos),
                   "d2h": sum(4 * args.batch * i.rows for i in infos),
                   "calls": "one tq_fused_gemv_stack_host call per step" if use_stack else "one tq_fused_gemv_host call per matrix"}
            if use_stack and len(mats) >= 8:
                # The same step as --e2e-groups host-buffer calls on two streams: consecutive matrices grouped by bytes,
                # each call copies its slice of x, runs its matrices and copies its slice of y back, so the copies of
                # one group pass under the kernel of the next.  Same bytes in and out, same public call.
                ab = [algorithmic_bytes(i, args.batch) for i in infos]
                cuts, acc, tot = [0], 0, sum(ab)
                for i, v in enumerate(ab):
                    acc += v
                    if acc >= tot * len(cuts) / args.e2e_groups and len(cuts) < args.e2e_groups and i + 1 < len(ab):
                        cuts.append(i + 1)
                cuts.append(len(mats))
                x0, y0 = x_arena.data_ptr(), y_arena.data_ptr()
                xo = [(x.data_ptr() - x0) // 2 for x in xs] + [x_arena.numel()]
                yo = [(y.data_ptr() - y0) // 4 for y in ys] + [y_arena.numel()]
                side = [torch.cuda.Stream(), torch.cuda.Stream()]
                groups = []
                for a_, b_ in zip(cuts[:-1], cuts[1:]):
                    st_ = tq.tq_stack_create(mats[a_:b_], xs[a_:b_], ys[a_:b_])
                    groups.append((st_, hxa[xo[a_]:xo[b_]], x_arena[xo[a_]:xo[b_]], hya[yo[a_]:yo[b_]], y_arena[yo[a_]:yo[b_]]))
                done = [torch.cuda.Event() for _ in side]

                def step_pipelined():
                    for sd in side:
                        sd.wait_stream(stream)
                    for k, (st_, hx_, dx_, hy_, dy_) in enumerate(groups):
                        tq.tq_fused_gemv_stack_host(st_, hx_, dx_, hy_, dy_, stream=side[k % 2])
                    for sd, ev in zip(side, done):
                        ev.record(sd)
                        stream.wait_event(ev)

                p_ms = time_e2e(step_pipelined)
                e2e["single_call_ms_per_step"] = e2e_ms
                e2e["pipelined_ms_per_step"] = p_ms
                if p_ms < e2e_ms:
                    e2e["ms_per_step"] = p_ms
                    e2e["calls"] = ("%d tq_fused_gemv_stack_host calls per step (consecutive matrices grouped by bytes) on two "
                                    "streams: the copies of one group pass under the kernel of the next" % len(groups))
                del groups

        # ---- the other device calls on the same resident model (single GPU only) ----
        extras = {}
        if not args.no_extras and world == 1:
            extras = time_extras(tq, mats, infos, shapes, args, device, stream,
                                 {"hd": hd, "dd": dd, "q_host": q_host, "scales": scales, "xs": xs, "ys": ys})

    ms_step = ms_total / args.steps
    if world > 1:
        import torch.distributed as dist
        t = torch.tensor([ms_step, e2e["ms_per_step"] if e2e else 0.0], device=device, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms_step = float(t[0].item())
        if e2e:
            e2e["ms_per_step"] = float(t[1].item())

    if rank != 0:
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
            dist.destroy_process_group()
        return

    peak, peak_src = measured_peaks()
    value = world * alg_bytes / (ms_step * 1e-3) / 1e9
    per_gpu = alg_bytes / (ms_step * 1e-3) / 1e9
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": DTYPE[args.layout],
        "data": "synthetic",
        "config": {"workload": workload, "n_weights": n_weights, "hit_rate": hits / (hits + miss),
                   "hit_rate_device_layout": hit_rate_device, "K": stats["K"],
                   "launch": ("one persistent launch over all matrices (tq_fused_gemv_stack)" if use_stack
                              else "one launch per matrix (tq_fused_gemv)"),
                   "layout": {"stream": "paper token stream, per-row segments", "planes": "two planes: fixed-stride tokens + packed raw words",
                              "tiles": "1 KB token tiles of 16 rows x 32 groups in integer-MMA operand order + one raw-word stream; "
                                       "table limited to the %d words shared memory holds" % tq.TQ_TILES_TABLE_WORDS}[args.layout],
                   "cuda_graph": graph is not None,
                   "l2": ("inputs larger than L2: each step streams %.2f GB" % (payload_bytes / 1e9) if ms_flushed is None else
                          "L2 flushed between steps (a %d MB buffer written), every step timed on its own; back to back without "
                          "the flush a step takes %.5f ms (%.1f MB served from L2)"
                          % (2 * L2_BYTES >> 20, ms_unflushed, payload_bytes / 1e6)),
                   "multi_gpu": "independent replicas, no data-path collective" if world > 1 else "single GPU"},
        "us_per_independent_pass": ms_step * 1e3 / args.batch,
        "bytes_per_step": {"algorithmic": alg_bytes, "paper_stream": stream_bytes, "device_payload": payload_bytes,
                           "int8_equivalent": n_weights},
        "pct_of_8TBs_nominal": 100.0 * per_gpu / 8000.0,
        "gpu_launches": launches_per_step * args.steps,
        "clocks": clocks,
        "roofline": {"bound": "hbm", "achieved": per_gpu, "peak": peak, "unit": "GB/s", "frac": per_gpu / peak,
                     "traffic": (TRAFFIC_RATIO["tiles_stack"] * alg_bytes / launches_per_step
                                 if use_stack and args.batch == 1 else TRAFFIC.get(args.layout)),
                     "traffic_note": ("not a counter of this run: profile constant %.3f (dram bytes / algorithmic bytes in the ncu capture of a "
                                      "14-matrix stack of this kernel, profiles/gemv_tiles_stack_llama3b_b1.md) x the algorithmic bytes of the launch"
                                      % TRAFFIC_RATIO["tiles_stack"] if use_stack and args.batch == 1 else None),
                     "kernel": {"stream": "gemv_kernel", "planes": "gemv_planes_kernel", "tiles": "gemv_tiles_kernel" if args.batch == 1 else "gemv_wide_kernel"}[args.layout],
                     "peak_source": peak_src,
                     "note": "achieved = algorithmic bytes of the %d launch(es) of a step / step time (launch gaps included)" % launches_per_step},
        "setup_s": stats,
    }
    out.update(extras)
    # A decoder's layers feed one another: its per-token time is that of the dependency-respecting launch sequence
    # where it was measured, else (custom workloads) that of the independent pass.
    dep = extras.get("dependent_launches")
    out["us_per_token"] = (dep["ms"] * 1e3 if dep else ms_step * 1e3) / args.batch
    out["us_per_token_source"] = ("dependent_launches leg (layers that feed one another launched one group after the other)" if dep
                                  else "independent pass (no dependency-respecting leg for this workload)")
    if e2e:
        out["e2e"] = {"value": world * alg_bytes / (e2e["ms_per_step"] * 1e-3) / 1e9, "unit": UNIT,
                      "h2d_bytes_per_step": e2e["h2d"], "d2h_bytes_per_step": e2e["d2h"],
                      "ms_per_step": e2e["ms_per_step"], "steps": e2e["steps"],
                      **{k: e2e[k] for k in ("calls", "single_call_ms_per_step", "pipelined_ms_per_step") if k in e2e}}

    if not args.no_cpu_baseline and args.quantizer == "rows":
        sample = pick_sample(shapes, 3_300_000_000)  # ~6-13 s of single-thread oracle work for the 3B stack
        nw = sum(shapes[i][1] * shapes[i][2] for i in sample)
        desc = f"first {len(sample)} matrices of the workload ({nw/1e6:.1f} M weights), Listing-4 decode + fp64 product, one pass"
        total, t_all, d_all = oracle_sample_run(hd.entries, q_host, scales, shapes, args.batch, sample, reps=1, workers=ncores, decode_only=True)
        total1, t_one, d_one = oracle_sample_run(hd.entries, q_host, scales, shapes, args.batch, sample, reps=1, workers=1, decode_only=True)
        used = min(ncores, len(sample))
        out["cpu_baseline"] = {
            "value": total / min(t_all) / 1e9, "unit": UNIT, "cores": used, "kind": "oracle",
            "sample": desc + f", {min(t_all):.2f} s; the single-threaded oracle on {used} worker threads, matrices dealt largest first",
            "one_core": {"value": total1 / min(t_one) / 1e9, "unit": UNIT, "cores": 1, "seconds": min(t_one)},
            "decode_only": {"note": "Listing-4 decode alone (no product), same sample; GB/s on the same algorithmic bytes",
                            "all_cores": {"value": total / min(d_all) / 1e9, "seconds": min(d_all), "cores": used},
                            "one_core": {"value": total1 / min(d_one) / 1e9, "seconds": min(d_one), "cores": 1}},
            "host_cores_available": ncores}
    print(json.dumps(out), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
        dist.destroy_process_group()


def run_row_sharded(tq, args, shapes, workload, device, rank, world, local_rank, dd, full_mats, scales, xs, alg_bytes, stats):
    """N GPUs, one model: every matrix split by output rows in whole 16-row blocks (paper_2509_22951_b200/sharding.py),
    the table and the activations replicated.  A step is this rank's tq_fused_gemv_stack launch over its shards
    followed by ONE NCCL all-gather of the output arenas; no kernel reads another GPU's memory.  The shards are cut
    out of the matrices the replica path builds (each rank decompresses its rows again and re-encodes them as
    matrices of their own), so both modes run on the same weights."""
    import torch.distributed as dist
    from paper_2509_22951_b200 import sharding
    assert args.layout == "tiles" and args.quantizer == "rows"
    so = sharding.ShardedOutputs(shapes, args.batch, world)
    shard_mats, keep = [], []
    for i, m in enumerate(full_mats):
        r0, r1 = so.ranges[rank][i]
        if r1 > r0:
            q = tq.tq_decompress(m).view(torch.int8).view(m.info.rows, m.info.cols)
            shard_mats.append(tq.tq_upload_device_rows(dd, q, r0, r1, torch.from_numpy(scales[i]).to(device)))
            keep.append(i)
            del q
    del full_mats
    torch.cuda.empty_cache()
    arena = torch.zeros(so.arena_len, dtype=torch.float32, device=device)
    gathered = torch.empty(world * so.arena_len, dtype=torch.float32, device=device)
    views = so.local_views(arena, rank)
    stack = tq.tq_stack_create(shard_mats, [xs[i] for i in keep], [views[i] for i in keep])
    stream = torch.cuda.Stream(device)

    def step():
        tq.tq_fused_gemv_stack(stack, stream=stream)
        with torch.cuda.stream(stream):
            so.all_gather(arena, gathered)

    for _ in range(max(args.warmup, 3)):
        step()
    stream.synchronize()
    sampler = ClockSampler(local_rank)
    sampler.start()
    sampler.wait_first()
    dist.barrier()
    torch.cuda.synchronize()
    t_start = time.time()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    stream.synchronize()
    torch.cuda.synchronize()
    dist.barrier()
    clocks = sampler.stop(t_start, time.time())
    t = torch.tensor([e0.elapsed_time(e1) / args.steps], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    ms_step = float(t[0].item())
    status = 0
    for m in shard_mats:
        status |= tq.tq_device_status(m)
    assert status == 0, f"device status {status}"
    if rank == 0:
        peak, peak_src = measured_peaks()
        value = alg_bytes / (ms_step * 1e-3) / 1e9  # the bytes of ONE model, streamed once per step by all ranks together
        print(json.dumps({
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "strong", "vs_baseline": None, "dtype": DTYPE[args.layout],
            "data": "synthetic",
            "config": {"workload": workload, "multi_gpu": "rows of every matrix split over %d GPUs in whole 16-row blocks, table and "
                       "activations replicated, one NCCL all-gather of %d bytes per rank per step" % (world, 4 * so.arena_len),
                       "l2": "inputs larger than L2: each rank streams %.2f GB per step" % (alg_bytes / world / 1e9)},
            "us_per_independent_pass": ms_step * 1e3 / args.batch, "gpu_launches": stack.launches * args.steps, "clocks": clocks,
            "roofline": {"bound": "hbm", "achieved": value / world, "peak": peak, "unit": "GB/s", "frac": value / world / peak,
                         "traffic": None, "kernel": "gemv_tiles_kernel" if args.batch == 1 else "gemv_wide_kernel", "peak_source": peak_src,
                         "note": "per GPU: its share of the algorithmic bytes / step time, the all-gather included"},
            "setup_s": stats}), flush=True)
    dist.barrier()
    dist.destroy_process_group()


def run_reference(args, shapes, workload):
    """The oracle as it stands on the host cores: each step = one bounded sample of the workload."""
    from oracle import oracle
    t0 = time.time()
    sample = pick_sample(shapes, 60_000_000)
    q_host, scales = {}, {}
    for i in sample:
        name, rows, cols = shapes[i]
        w = synth.weight(rows, cols, synth.matrix_seed(i)).numpy()
        q_host[i], scales[i] = oracle.quantize_rows(w)
    od = oracle.Dictionary.build([q_host[i] for i in sample])  # the oracle's own table over the sample
    log(f"reference setup {time.time()-t0:.1f} s, sample {sample}")
    total, times, _ = oracle_sample_run(od.entries, q_host, scales, shapes, args.batch, sample,
                                        reps=max(args.warmup, 1) + args.steps)
    times = times[max(args.warmup, 1):]
    ms = 1e3 * sum(times) / len(times)
    v = total / (ms * 1e-3) / 1e9
    nw = sum(shapes[i][1] * shapes[i][2] for i in sample)
    desc = f"first {len(sample)} matrices of the workload ({nw/1e6:.1f} M weights) per step, table built over the sample"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": max(args.warmup, 1), "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int8 weights x bf16 activations, fp64 accumulate", "data": "synthetic",
        "config": {"workload": workload, "sample": desc},
        "cpu_baseline": {"value": v, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": desc},
        "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }), flush=True)


if __name__ == "__main__":
    main()
