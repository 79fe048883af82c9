#!/usr/bin/env python
"""Benchmark of the fused few-bit GEMM + threshold hot path on B200.

Workload (one "step"): the microbenchmark sweep of fused GEMM+threshold over
every (w, a) in {1,2,3,4}^2 at M = N = K = 4096 -- weights two's complement
(bipolar when w = 1), activations unsigned, 2^a - 1 sorted thresholds per row.
Per (w, a) a step packs the logical activations into the operand format
(packer), then runs the fused GEMM + threshold epilogue; weights are packed
once, outside the timed region.  Metric: effective few-bit MAC/s = 16 * 4096^3
MAC per step / step time (the paper's GOPS is twice this number).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

N > 1 (under torchrun): every rank runs the same sweep on its own GPU, with no
data-path collective (weak scaling); time = max over ranks.
``--impl reference`` times the CPU oracle on the host cores on a bounded sample
of the same workload.
"""
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

import numpy as np

DIM = 4096
PAIRS = [(w, a) for w in (1, 2, 3, 4) for a in (1, 2, 3, 4)]
METRIC = "effective few-bit MAC/s, fused WwAa GEMM+threshold sweep (w,a in 1..4, M=N=K=4096)"
UNIT = "MAC/s"
WORKLOAD = "configs[1]: 16-point (w,a) sweep of GEMM+threshold at M=N=K=4096"


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "bf16_burst": p["bf16_tflops"],
                "bf16_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_burst": 1590.0, "bf16_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while a region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0, t1):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.12)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        inside = [l for (t, l) in self.lines if t0 <= t <= t1 + 0.06] or [l for (_, l) in self.lines[-3:]]
        sm, mx, pw, reasons = [], [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for l in inside:
            f = [x.strip() for x in l.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1])); pw.append(float(f[2]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None,
                "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(pw) if pw else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def oracle_sample_run(rows: int, pairs, seed_base=2000):
    """Oracle GEMM+threshold on the first `rows` weight rows of the given (w,a) problems.
    Returns (MACs, seconds, threads)."""
    from oracle import oracle as orc
    from paper_1709_04060_b200 import synth
    cases = []
    for (w, a) in pairs:
        c = synth.gemm_case(seed_base + 10 * w + a, rows, DIM, DIM, w, a)
        cases.append(c)
    orc.gemm(cases[0].W[:8], cases[0].At[:8])          # load the library
    t0 = time.perf_counter()
    for c in cases:
        orc.qgemm(c.W, c.At, c.thr)
    dt = time.perf_counter() - t0
    return float(len(pairs)) * rows * DIM * DIM, dt, orc.num_threads()


def run_reference(args):
    """The CPU oracle as the reference arm: each step is a bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import build as ob
    ob.build()
    rows = 256
    pairs = [(1, 2), (4, 4)]
    for _ in range(args.warmup):
        oracle_sample_run(rows, pairs[:1])
    macs = secs = 0.0
    threads = 1
    for _ in range(args.steps):
        m, s, threads = oracle_sample_run(rows, pairs)
        macs += m; secs += s
    value = macs / secs
    sample = f"per step: first {rows} weight rows x all {DIM} columns, K={DIM}, (w,a) in {pairs}"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * secs / max(args.steps, 1),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int64",
        "data": "synthetic", "config": {"workload": WORKLOAD, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def oracle_other_configs():
    """The oracle as it stands on the other configurations (or a bounded sample of them):
    config 1 in full, one conv2-shaped image, one AlexNet-shaped image, config 5 at N = 1."""
    from oracle import oracle as orc, alexnet as onet
    from paper_1709_04060_b200 import synth
    res = {}
    c1 = synth.gemm_case(1, 64, 256, 576, 1, 2)
    orc.qgemm(c1.W, c1.At, c1.thr)
    t0 = time.perf_counter()
    for _ in range(20):
        orc.qgemm(c1.W, c1.At, c1.thr)
    dt = (time.perf_counter() - t0) / 20
    res["config1"] = {"us": 1e6 * dt, "mac_per_s": 64 * 256 * 576 / dt, "sample": "the whole problem, mean of 20"}
    c3 = synth.conv2_alexnet_case(1)
    t0 = time.perf_counter()
    orc.qconv(c3.In, c3.Wt, c3.thr, c3.stride, c3.pad)
    dt = time.perf_counter() - t0
    res["config3"] = {"images_per_s": 1.0 / dt, "mac_per_s": 729 * 256 * 2400 / dt, "sample": "one image (direct convolution)"}
    net = synth.alexnet_case(1)
    t0 = time.perf_counter()
    onet.forward(net, keep_intermediates=False)
    dt = time.perf_counter() - t0
    res["config4"] = {"images_per_s": 1.0 / dt, "mac_per_s": 1.135e9 / dt, "sample": "one image through the whole chain"}
    c5 = synth.gemm_case(5021, 8192, 1, 8192, 2, 2)
    t0 = time.perf_counter()
    orc.qgemm(c5.W, c5.At, c5.thr)
    dt = time.perf_counter() - t0
    res["config5"] = {"us": 1e6 * dt, "mac_per_s": 8192 * 8192 / dt, "sample": "W2A2, N = 1, the whole problem"}
    res["cores"] = orc.num_threads()
    return res


def sustained_mma_peak(torch, qb, seconds=1.5):
    """The widest CTA-pair MMA issued back to back for `seconds`: the int8 tensor peak the GPU
    holds under its power cap (TOP/s), i.e. the denominator for kernels timed inside a long loop."""
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    st, ops = qb.qnn_peak_mma_i8(1, 256, 65536)         # ~4.6 ms per launch
    qb.check(st)
    torch.cuda.synchronize()
    n = max(1, int(seconds / 4.6e-3))
    e0.record()
    for _ in range(n):
        qb.check(qb.qnn_peak_mma_i8(1, 256, 65536)[0])
    e1.record()
    torch.cuda.synchronize()
    return round(n * ops / (e0.elapsed_time(e1) * 1e-3) / 1e12, 1)


def roofline_entry(achieved_tops, gemm_avg_ms, timed_seconds, clocks, peaks, measured):
    """Tensor roofline of the dominant kernel.  The denominator is the int8 MMA issue rate measured
    in this run: the sustained figure when the timed region ran for a second or more under the
    power cap, else the burst figure; the other candidates are printed beside it."""
    long_run = timed_seconds >= 1.0 or (clocks and "sw_power_cap" in (clocks.get("reasons") or []))
    cands = {"2x_bf16_cublas_sustained_of_" + peaks["source"]: 2.0 * peaks["bf16_sustained"],
             "2x_bf16_cublas_burst_of_" + peaks["source"]: 2.0 * peaks["bf16_burst"],
             "nominal_dense_int8": 4500.0}
    if measured:
        cands["int8_mma_burst_measured"] = measured["mma_i8"]["mode1_n256"]
        cands["int8_mma_sustained_measured"] = measured["mma_i8_sustained"]
        key = "int8_mma_sustained_measured" if long_run else "int8_mma_burst_measured"
    else:
        key = "2x_bf16_cublas_sustained_of_" + peaks["source"] if long_run else "2x_bf16_cublas_burst_of_" + peaks["source"]
    peak = cands[key]
    return {"bound": "tensor", "achieved": achieved_tops, "peak": peak, "unit": "TOP/s",
            "frac": achieved_tops / peak, "peak_source": key,
            "frac_vs": {k: round(achieved_tops / v, 3) for k, v in cands.items()},
            "peaks_tops": cands,
            "traffic": TRAFFIC_BYTES_PER_LAUNCH,
            "traffic_source": "ncu dram__bytes of one 4096^3 W1A2 launch (constant from that capture)",
            "kernel": "qgemm_tc2_kernel (CTA-pair tcgen05 kernel, 4096^3, int8 operands)",
            "avg_launch_ms": gemm_avg_ms, "algorithmic_ops_per_launch": 2.0 * DIM ** 3}


def measure_other_configs(torch, qb, synth, peaks, measured):
    """Configurations 1, 3, 4 (per layer) and 5 in compact form, each with the roofline that
    bounds it: latency for the small GEMM, HBM for lowering and the few-column fully connected
    layers (weights rotated through more than twice the L2 size), tensor for the rest."""
    from paper_1709_04060_b200.alexnet import AlexNetPlan
    PL, I8 = qb.QNN_FMT_BITPLANES, qb.QNN_FMT_INT8
    hbm = peaks["hbm_gbs"]
    tpeak = measured["mma_i8"]["mode1_n256"]             # burst: these kernels are timed in short loops
    res = {"hbm_peak_gbs": hbm, "tensor_peak_tops": tpeak, "peak_source": f"HBM: {peaks['source']} copy; tensor: int8 MMA burst measured in this run"}

    # config 1: one small W1A2 GEMM + threshold (launch-latency bound)
    c = synth.gemm_case(1, 64, 256, 576, 1, 2)
    row = {}
    for fmt, name in ((I8, "int8"), (PL, "bitplanes")):
        Wp = qb.pack(qb.to_device_logical(c.W, c.w_enc), 1, c.w_enc, fmt)
        Ap = qb.pack(qb.to_device_logical(c.At, c.a_enc), 2, c.a_enc, fmt)
        thr = torch.from_numpy(c.thr).cuda()
        d = qb.gemm_desc(64, 256, 576, 1, 2, 2, c.w_enc, c.a_enc, fmt, I8)
        out = torch.empty(qb.qnn_gemm_out_bytes(d, True), dtype=torch.uint8, device="cuda")
        ms = _time_calls(torch, lambda i: qb.check(qb.qnn_qgemm(d, Wp, Ap, thr, out)), 50, graph=True)
        row[name + "_us"] = round(1e3 * ms, 2)
    row.update({"bound": "latency", "mac": 64 * 256 * 576, "gmacs_int8": round(64 * 256 * 576 / row["int8_us"] / 1e3, 1)})
    res["config1"] = row

    # config 3: conv2-shaped W1A2 layer, 8-bit maps: explicit lowering (HBM) and the whole layer (tensor)
    conv = {}
    for B in (1, 64):
        c = synth.conv2_alexnet_case(B)
        x = torch.from_numpy(c.In.astype(np.uint8)).cuda()
        Wp = qb.pack(qb.to_device_logical(c.Wt.reshape(c.OC, -1), c.w_enc), 1, c.w_enc, I8)
        d = qb.qnn_conv_desc(B, 27, 27, 96, 96, 256, 5, 5, 1, 2, 1, 2, 2, c.w_enc, c.a_enc, I8, I8, 0)
        thr = torch.from_numpy(c.thr).cuda()
        ws = torch.empty(qb.qnn_conv_workspace_bytes(d), dtype=torch.uint8, device="cuda")
        out = torch.empty(qb.qnn_conv_out_bytes(d, True), dtype=torch.uint8, device="cuda")
        ms_low = _time_calls(torch, lambda i: qb.check(qb.qnn_im2col(d, x, ws)), 20, graph=True)
        ms_all = _time_calls(torch, lambda i: qb.check(qb.qnn_qconv(d, Wp, x, thr, out, ws, ws.numel())), 20, graph=True)
        low_bytes = qb.qnn_conv_lowered_bytes(d) + x.numel()
        macs = B * 729 * 256 * 2400
        conv[f"B{B}"] = {"im2col_us": round(1e3 * ms_low, 2), "im2col_gbs": round(low_bytes / ms_low / 1e6, 1),
                         "im2col_hbm_frac": round(low_bytes / ms_low / 1e6 / hbm, 3),
                         "qconv_us": round(1e3 * ms_all, 2), "images_per_s": round(B / ms_all * 1e3, 1),
                         "tmacs": round(macs / ms_all / 1e9, 1), "tensor_frac": round(2 * macs / ms_all / 1e9 / tpeak, 3)}
        del ws, out
    conv["note"] = "lowered matrix of B = 1 (1.75 MB) stays in L2; B = 64 (112 MB) is close to the L2 size"
    res["config3"] = conv

    # config 5: M = K = 8192; few columns (HBM bound, packed bytes) and N = 8192 (tensor bound)
    M = K = 8192
    skinny = []
    for bits in (2, 4):
        c = synth.gemm_case(5000 + bits, M, 16, K, bits, bits)
        Wd = qb.to_device_logical(c.W, c.w_enc)
        thr = torch.from_numpy(c.thr).cuda()
        packed_bytes = M * K * bits // 8
        for wfmt, afmt, name in SKINNY_FORMATS(qb):
            Wp = qb.pack(Wd, bits, c.w_enc, wfmt)
            copies = max(2, int(300e6 // Wp.numel()) + 1)          # > 2 x L2 in rotation
            Wrot = [Wp] + [Wp.clone() for _ in range(copies - 1)]
            for N in (1, 4, 16):
                Ap = qb.pack(qb.to_device_logical(c.At[:N], c.a_enc), bits, c.a_enc, afmt)
                d = qb.qnn_gemm_desc(M, N, K, bits, bits, bits, c.w_enc, c.a_enc, wfmt, afmt, I8, 0)
                out = torch.empty(qb.qnn_gemm_out_bytes(d, True), dtype=torch.uint8, device="cuda")
                ms = _time_calls(torch, lambda i: qb.check(qb.qnn_qgemm(d, Wrot[i % copies], Ap, thr, out)),
                                 2 * copies, graph=True)
                alg = packed_bytes + N * K * bits // 8 + thr.numel() * 4 + N * M
                skinny.append({"w": bits, "a": bits, "N": N, "fmt": name, "us": round(1e3 * ms, 2),
                               "gbs_packed": round(alg / ms / 1e6, 1), "hbm_frac_packed": round(alg / ms / 1e6 / hbm, 3),
                               "bytes_read_per_call": Wp.numel() + Ap.numel() + thr.numel() * 4})
            del Wrot, Wp
    res["config5_skinny"] = {"rows": skinny, "bound": "hbm",
                             "note": "hbm_frac_packed = bytes of the w-bit packed problem (weights w*M*K/8, activations, "
                                     "thresholds, codes) / time / HBM peak, whatever operand format the kernel reads"}
    sets = [(torch.randint(-2, 2, (M, K), dtype=torch.int8, device="cuda"),
             torch.randint(0, 4, (M, K), dtype=torch.uint8, device="cuda")) for _ in range(2)]
    thr_l = torch.sort(torch.randint(-300, 300, (M, 3), dtype=torch.int32, device="cuda"), dim=1).values.contiguous()
    out_l = torch.empty(M * M, dtype=torch.uint8, device="cuda")
    dl = qb.gemm_desc(M, M, K, 2, 2, 2, qb.QNN_ENC_SIGNED, qb.QNN_ENC_UNSIGNED, I8, I8)
    ms_l = _time_calls(torch, lambda i: qb.check(qb.qnn_qgemm(dl, sets[i % 2][0], sets[i % 2][1], thr_l, out_l)), 6, graph=True)
    res["config5_n8192"] = {"us": round(1e3 * ms_l, 1), "tmacs": round(M ** 3 / ms_l / 1e9, 1),
                            "tensor_frac": round(2 * M ** 3 / ms_l / 1e9 / tpeak, 3), "bound": "tensor"}
    del sets, out_l

    # config 4: per-layer times of the AlexNet-shaped chain at batch 256
    B = 256
    net = synth.alexnet_case(B)
    plan = AlexNetPlan(net, B, "auto")
    img = torch.from_numpy(net.image.astype(np.uint8)).cuda()
    plan.forward(img)
    per_layer, prev, total_us = {}, None, 0.0
    macs = {"conv1": 1.054e8, "conv2": 4.479e8, "conv3": 1.495e8, "conv4": 2.243e8, "conv5": 1.495e8,
            "fc6": 3.77e7, "fc7": 1.68e7, "fc8": 4.10e6}
    for (kind, d, Wp, thr, out), name in zip(plan.steps, plan.names):
        x_in = img if prev is None else prev
        if kind == "conv":
            f = lambda i: qb.check(qb.qnn_qconv(d, Wp, x_in, thr, out, plan.workspace, plan.workspace.numel()))
        elif kind == "pool":
            f = lambda i: qb.check(qb.qnn_maxpool(d, x_in, out))
        else:
            f = lambda i: qb.check(qb.qnn_qgemm(d, Wp, x_in, thr, out, None, 0))
        us = 1e3 * _time_calls(torch, f, 10, graph=True)
        entry = {"us": round(us, 1)}
        if name in macs:
            entry["tensor_frac"] = round(2 * macs[name] * B / us / 1e6 / tpeak, 3)
        else:
            nbytes = x_in.numel() + out.numel()
            entry["gbs"] = round(nbytes / us / 1e3, 1)
            entry["hbm_frac"] = round(nbytes / us / 1e3 / hbm, 3)
        per_layer[name] = entry
        total_us += us
        prev = out
    matrix_us = sum(v["us"] for k, v in per_layer.items() if k in macs)
    res["config4_batch256_layers"] = {"per_layer": per_layer, "sum_us": round(total_us, 1),
                                      "share_8bit_layers": round((per_layer["conv1"]["us"] + per_layer["fc8"]["us"]) / total_us, 3),
                                      "share_matrix_layers": round(matrix_us / total_us, 3),
                                      "chain_tensor_frac": round(2 * 1.135e9 * B / total_us / 1e6 / tpeak, 3)}
    st, dev = qb.qnn_device_status()
    assert st == 0 and dev == 0
    return res


def SKINNY_FORMATS(qb):
    """(weight format, activation format, label) triples the few-column benchmark runs."""
    PL, I8 = qb.QNN_FMT_BITPLANES, qb.QNN_FMT_INT8
    fmts = [(PL, PL, "bitplanes"), (I8, I8, "int8")]
    if hasattr(qb, "QNN_FMT_FIELDS"):
        fmts.insert(0, (qb.QNN_FMT_FIELDS, I8, "fields"))
    return fmts


def run_b200(args):
    import torch
    from paper_1709_04060_b200 import dist as qdist, synth
    rank, world = qdist.init("nccl")
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    import __graft_entry__ as ge
    if rank == 0:
        ge.build()
    qdist.barrier()
    from paper_1709_04060_b200 import binding as qb

    INT8 = qb.QNN_FMT_INT8
    peaks = load_peaks()

    # ---- inputs: seeded synthetic logical tensors, packed weights resident in HBM
    problems = []
    for (w, a) in PAIRS:
        c = synth.gemm_case(2000 + 10 * w + a, DIM, DIM, DIM, w, a)
        Wd = qb.to_device_logical(c.W, c.w_enc)
        prob = {
            "w": w, "a": a, "case": c,
            "Wp": qb.pack(Wd, w, c.w_enc, INT8),
            "A_log": torch.from_numpy(c.At.astype(np.uint8)).cuda(),
            "A_packed": torch.empty(DIM * DIM, dtype=torch.uint8, device="cuda"),
            "thr": torch.from_numpy(c.thr).cuda(),
            "out": torch.empty(DIM * DIM, dtype=torch.uint8, device="cuda"),
            "pd": qb.qnn_pack_desc(DIM, DIM, a, c.a_enc, INT8),
            "gd": qb.gemm_desc(DIM, DIM, DIM, w, a, a, c.w_enc, c.a_enc, INT8, INT8),
        }
        # End-to-end leg: few-bit data crosses the host link packed.  The activations wait in pinned
        # host memory as bit planes (a bits per element; packed once, at set-up, by the library's
        # packer), are widened to 8-bit containers on the device, and the output codes go back as
        # bit planes (a bits per code).
        PL = qb.QNN_FMT_BITPLANES
        planes_dev = qb.pack(prob["A_log"], a, c.a_enc, PL)
        prob["rd"] = qb.qnn_pack_desc(DIM, DIM, a, c.a_enc, PL)
        prob["A_planes"] = planes_dev
        prob["A_planes_host"] = planes_dev.cpu().pin_memory()
        prob["gd_pl"] = qb.gemm_desc(DIM, DIM, DIM, w, a, a, c.w_enc, c.a_enc, INT8, PL)
        prob["out_pl"] = torch.empty(qb.qnn_gemm_out_bytes(prob["gd_pl"], True), dtype=torch.uint8, device="cuda")
        prob["out_pl_host"] = torch.empty(prob["out_pl"].numel(), dtype=torch.uint8).pin_memory()
        del Wd
        problems.append(prob)
    # scratch the library may use to split a half-empty last round of tiles between SM pairs (its
    # leading flag words start out zero and the library leaves them zero); the GEMMs of a step run
    # one after the other on one stream, so they share it
    gemm_ws = torch.zeros(max(16, max(qb.qnn_gemm_workspace_bytes(p["gd"]) for p in problems)),
                          dtype=torch.uint8, device="cuda")
    torch.cuda.synchronize()

    # The packer of problem i + 1 (HBM bound) runs on a second stream while the GEMM of
    # problem i (tensor bound) runs on the main one; events order each GEMM after its packer
    # and each packer after the GEMM that last read its output buffer.
    s_pack = torch.cuda.Stream() if args.overlap else None
    s_out = torch.cuda.Stream()

    def step(gemm_events=None, host_io=False):
        main = torch.cuda.current_stream()
        if s_pack is not None:
            s_pack.wait_stream(main)
        for p in problems:
            if s_pack is not None:
                if "gemm_done" in p:
                    s_pack.wait_event(p["gemm_done"])
                with torch.cuda.stream(s_pack):
                    if host_io:
                        p["A_planes"].copy_(p["A_planes_host"], non_blocking=True)
                        qb.check(qb.qnn_planes_to_int8(p["rd"], p["A_planes"], p["A_packed"]))
                    else:
                        qb.check(qb.qnn_pack(p["pd"], p["A_log"], p["A_packed"]))
                    p["packed"] = torch.cuda.Event()
                    p["packed"].record(s_pack)
                main.wait_event(p["packed"])
            elif host_io:
                p["A_planes"].copy_(p["A_planes_host"], non_blocking=True)
                qb.check(qb.qnn_planes_to_int8(p["rd"], p["A_planes"], p["A_packed"]))
            else:
                qb.check(qb.qnn_pack(p["pd"], p["A_log"], p["A_packed"]))
            if gemm_events is not None:
                e0 = torch.cuda.Event(enable_timing=True); e0.record()
            if host_io:
                qb.check(qb.qnn_qgemm(p["gd_pl"], p["Wp"], p["A_packed"], p["thr"], p["out_pl"], gemm_ws, gemm_ws.numel()))
            else:
                qb.check(qb.qnn_qgemm(p["gd"], p["Wp"], p["A_packed"], p["thr"], p["out"], gemm_ws, gemm_ws.numel()))
            if gemm_events is not None:
                e1 = torch.cuda.Event(enable_timing=True); e1.record()
                gemm_events.append((e0, e1))
            if s_pack is not None:
                p["gemm_done"] = torch.cuda.Event()
                p["gemm_done"].record(main)
            if host_io:
                # the read-back runs on its own stream, so that the next GEMM does not queue behind it
                s_out.wait_stream(main)
                with torch.cuda.stream(s_out):
                    p["out_pl_host"].copy_(p["out_pl"], non_blocking=True)
        if host_io:
            main.wait_stream(s_out)

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    # Three steps are 3 ms: not enough for the SM clock and the power state to settle after the idle
    # seconds of set-up (a run was seen with its first 25 timed steps 25 % slow).  More untimed
    # steps of the same work, for about 0.3 s, before the timed region.
    t_spin = time.time()
    while time.time() - t_spin < 0.3:
        for _ in range(20):
            step()
        torch.cuda.synchronize()

    # ---- device-resident timing
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.15)
    qdist.barrier()
    torch.cuda.synchronize()
    # Per-launch event pairs (for the roofline entry) on a sample of the timed steps, spread over
    # the region: a pair around every launch keeps consecutive kernels from overlapping set-up and
    # tail, which costs a step about 10 %, so at most one step in eight carries them (at most 25).
    n_event_steps = max(1, min(25, args.steps // 8))
    event_every = max(1, args.steps // n_event_steps)
    gemm_events = []
    launches0 = qb.qnn_launch_count()
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_wall0 = time.time()
    start.record()
    for s in range(args.steps):
        step(gemm_events if (s % event_every == 0 and s // event_every < n_event_steps) else None)
    end.record()
    torch.cuda.synchronize()
    t_wall1 = time.time()
    qdist.barrier()
    launches = qb.qnn_launch_count() - launches0
    ms_local = start.elapsed_time(end)
    ms = qdist.max_over_ranks(ms_local, device="cuda")
    clocks = sampler.stop(t_wall0, t_wall1) if rank == 0 else None
    st, dev = qb.qnn_device_status()
    assert st == 0 and dev == 0, f"device status {dev}"

    macs_per_step = float(len(PAIRS)) * DIM ** 3
    value = world * macs_per_step * args.steps / (ms * 1e-3)

    gemm_ms = [a.elapsed_time(b) for (a, b) in gemm_events]
    gemm_avg_ms = float(np.mean(gemm_ms))
    achieved_tops = 2.0 * DIM ** 3 / (gemm_avg_ms * 1e-3) / 1e12
    per_pair = {}
    for i, (w, a) in enumerate(PAIRS):
        t = float(np.mean(gemm_ms[i::len(PAIRS)]))
        per_pair[f"W{w}A{a}"] = round(DIM ** 3 / (t * 1e-3) / 1e12, 1)

    # ---- end to end: host buffers, copies inside the timed region
    e2e_steps = max(1, min(args.steps, 5))
    step(host_io=True)
    torch.cuda.synchronize()
    qdist.barrier()
    s2, e2 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    s2.record()
    for _ in range(e2e_steps):
        step(host_io=True)
    e2.record()
    torch.cuda.synchronize()
    qdist.barrier()
    ms_e2e = qdist.max_over_ranks(s2.elapsed_time(e2), device="cuda")
    e2e_value = world * macs_per_step * e2e_steps / (ms_e2e * 1e-3)

    if rank != 0:
        qdist.finalize()
        return

    # ---- CPU baseline: the oracle on a bounded sample of the same workload (N = 1 only)
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        rows, pairs = 2048, [(1, 2), (4, 4)]
        m, s, threads = oracle_sample_run(rows, pairs)
        cpu = {"value": m / s, "unit": UNIT, "cores": threads, "kind": "oracle",
               "sample": f"first {rows} weight rows x all {DIM} columns, K={DIM}, (w,a) in {pairs}: "
                         f"{m:.3g} MAC in {s:.1f} s",
               "other_configs": oracle_other_configs()}

    # ---- roofline denominators measured in this run, and the other configurations
    measured = other = None
    if world == 1:
        measured = measure_peaks(torch, qb, ((1, 256), (0, 256)), mmas=8192, popc_iters=8192, reps=3)
        measured["mma_i8_sustained"] = sustained_mma_peak(torch, qb, seconds=1.5)
        if not args.no_other_configs:
            other = measure_other_configs(torch, qb, synth, peaks, measured)

    # ---- second half of the metric: AlexNet-shaped W1A2 chain, images/s (N = 1 only)
    alexnet = None
    if world == 1 and not args.no_alexnet:
        from paper_1709_04060_b200.alexnet import AlexNetPlan
        alexnet = {}
        for B in (256, 1):
            net = synth.alexnet_case(B)
            plan = AlexNetPlan(net, B, "auto")
            img = torch.from_numpy(net.image.astype(np.uint8)).cuda()
            graph, _ = plan.capture(img)
            ms_b = _time_calls(torch, lambda i: graph.replay(), 20 if B > 1 else 50)
            alexnet[f"batch{B}"] = {"images_per_s": B / ms_b * 1e3, "ms": ms_b,
                                    "kernels_per_forward": plan.launches_per_forward()}
            del graph, plan
        if cpu is not None:
            alexnet["oracle_images_per_s_batch1"] = cpu["other_configs"]["config4"]["images_per_s"]
            alexnet["oracle_cores"] = cpu["other_configs"]["cores"]
        alexnet["note"] = ("random-init AlexNet-shaped W1A2 chain (conv1/fc8 8-bit), uint8 images resident "
                           "in HBM, one CUDA-graph replay per forward pass")

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int8 operands, int32 accumulate",
        "data": "synthetic",
        "config": {"workload": WORKLOAD, "path": "tcgen05 kind::i8 + fused threshold epilogue",
                   "step": "per (w,a): pack activations to int8 containers, fused GEMM+threshold; weights pre-packed",
                   "l2": "inputs larger than L2: one step streams 1 GiB of operands/outputs across 16 problems",
                   "spin_up": "about 0.3 s of further untimed steps after the warm-up steps, so that clocks have settled",
                   "gops_paper_convention": 2 * value / 1e9},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT,
                "h2d_bytes_per_step": int(sum(p["A_planes_host"].numel() for p in problems)),
                "d2h_bytes_per_step": int(sum(p["out_pl_host"].numel() for p in problems)),
                "steps": e2e_steps,
                "note": "activations cross the host link as bit planes (a bits per element) and are widened to "
                        "8-bit containers on the device; output codes return as bit planes"},
        "gpu_launches": int(launches),
        "roofline": roofline_entry(achieved_tops, gemm_avg_ms, ms * 1e-3, clocks, peaks, measured),
        "per_pair_tmacs": per_pair,
        "measured_peaks": measured,
        "alexnet_w1a2": alexnet,
        "other_configs": other,
        "cpu_baseline": cpu,
    }
    print(json.dumps(out))
    qdist.finalize()


QUICK = False      # --quick: few iterations and no graph replay (profiler captures)


def _time_calls(torch, fn, iters, warmup=3, graph=False):
    """Mean device milliseconds of fn(i), CUDA events on the current stream.  With graph=True
    the `iters` calls are recorded into one CUDA graph and the graph is replayed, which takes
    the host's per-call cost (a few microseconds of Python and ctypes) out of the number."""
    if QUICK:
        iters, warmup, graph = min(iters, 2), 1, False
    for i in range(warmup):
        fn(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if graph:
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for i in range(iters):
                fn(i)
        g.replay()
        torch.cuda.synchronize()
        reps = 5
        e0.record()
        for _ in range(reps):
            g.replay()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / (iters * reps)
    e0.record()
    for i in range(iters):
        fn(warmup + i)
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters


def measure_peaks(torch, qb, mma_configs=((1, 256),), mmas=4096, popc_iters=4096, reps=5):
    """Issue-bound peaks of the two GEMM paths, timed with CUDA events (best of `reps`):
    tcgen05 kind::i8 MMAs on shared-memory-resident tiles (pair: cta_group::2) and XOR+POPC
    chains.  Returns {"mma_i8": {"mode<m>_n<n>": TOP/s, ...}, "popc_g_per_s": ..}; mode 0: one CTA per
    SM, 1: CTA pairs, 2: one CTA per SM with the 128-row operand in tensor memory."""
    out = {"mma_i8": {}}
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for (pair, n) in mma_configs:
        best = None
        for r in range(reps + 1):
            e0.record()
            st, ops = qb.qnn_peak_mma_i8(pair, n, mmas)
            e1.record()
            qb.check(st)
            torch.cuda.synchronize()
            if r > 0:
                ms = e0.elapsed_time(e1)
                best = ms if best is None else min(best, ms)
        out["mma_i8"][f"mode{pair}_n{n}"] = round(ops / (best * 1e-3) / 1e12, 1)
    sink = torch.empty(qb.qnn_peak_popc_sink_bytes(), dtype=torch.uint8, device="cuda")
    best = None
    for r in range(reps + 1):
        e0.record()
        st, popcs = qb.qnn_peak_popc(popc_iters, sink)
        e1.record()
        qb.check(st)
        torch.cuda.synchronize()
        if r > 0:
            ms = e0.elapsed_time(e1)
            best = ms if best is None else min(best, ms)
    out["popc_g_per_s"] = round(popcs / (best * 1e-3) / 1e9, 1)
    out["binary_tmac_per_s"] = round(32 * popcs / (best * 1e-3) / 1e12, 2)
    st, dev = qb.qnn_device_status()
    assert st == 0 and dev == 0
    return out


def run_peaks(args):
    """Roofline denominators measured on this GPU: the int8 tensor-pipe issue rate for a range of
    MMA widths (one CTA per SM, and CTA pairs) and the POPC issue rate, with the SM clock sampled
    meanwhile.  Prints one JSON line."""
    import torch
    import __graft_entry__ as ge
    ge.build()
    from paper_1709_04060_b200 import binding as qb
    torch.cuda.set_device(0)
    sampler = ClockSampler(0)
    sampler.start()
    time.sleep(0.15)
    t0 = time.time()
    cfgs = ([(0, n) for n in (16, 32, 64, 128, 256)] + [(1, n) for n in (32, 64, 128, 256)] +
            [(2, n) for n in (16, 32, 64, 128)])          # mode 2: 128-row operand from tensor memory
    res = measure_peaks(torch, qb, cfgs, mmas=16384, popc_iters=16384, reps=8)
    # a seconds-long run of the widest pair MMA: the sustained figure under the power cap
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    total = 0.0
    for _ in range(400):
        st, ops = qb.qnn_peak_mma_i8(1, 256, 65536)
        qb.check(st)
        total += ops
    e1.record()
    torch.cuda.synchronize()
    res["mma_i8_sustained_mode1_n256"] = round(total / (e0.elapsed_time(e1) * 1e-3) / 1e12, 1)
    res["sustained_seconds"] = round(e0.elapsed_time(e1) * 1e-3, 2)
    clocks = sampler.stop(t0, time.time())
    peaks = load_peaks()
    res.update({"workload": "peaks", "clocks": clocks,
                "nominal": {"int8_dense_tops": 4500.0, "popc_per_clk_per_sm": 16,
                            "popc_g_per_s_at_max_clock": 16 * 148 * 1.965},
                "measured_bf16_tflops": {"burst": peaks["bf16_burst"], "sustained": peaks["bf16_sustained"],
                                         "source": peaks["source"]}})
    print(json.dumps(res))


def run_extras(args):
    """The other paper-shaped workloads on one GPU (not the headline line): the large/skinny
    fully connected sweep (HBM roofline, weight buffers rotated so that every call streams
    its weights from DRAM), the conv2-shaped layer via lowering, and the AlexNet-shaped
    chain.  Prints one JSON line."""
    import torch
    import __graft_entry__ as ge
    ge.build()
    from paper_1709_04060_b200 import binding as qb, synth
    from paper_1709_04060_b200.alexnet import AlexNetPlan
    torch.cuda.set_device(0)
    peaks = load_peaks()
    PL, I8 = qb.QNN_FMT_BITPLANES, qb.QNN_FMT_INT8
    res = {"workload": "extras", "hbm_peak_gbs": peaks["hbm_gbs"], "peak_source": peaks["source"]}

    only = args.extras_only
    # ---- large GEMMs (config 5 at N = 8192 and a many-column layer): one-CTA vs CTA-pair kernel
    large = []
    for (Mg, Ng, Kg) in ((8192, 8192, 8192), (4096, 18944, 4096), (4096, 18944, 512)) if only in (None, "large") else ():
        nsets = 2
        sets = [(torch.randint(-2, 2, (Mg, Kg), dtype=torch.int8, device="cuda"),
                 torch.randint(0, 4, (Ng, Kg), dtype=torch.uint8, device="cuda")) for _ in range(nsets)]
        thr_l = torch.sort(torch.randint(-300, 300, (Mg, 3), dtype=torch.int32, device="cuda"), dim=1).values.contiguous()
        out_l = torch.empty(Ng * Mg, dtype=torch.uint8, device="cuda")
        dl = qb.gemm_desc(Mg, Ng, Kg, 2, 2, 2, qb.QNN_ENC_SIGNED, qb.QNN_ENC_UNSIGNED, I8, I8)
        row = {"M": Mg, "N": Ng, "K": Kg}
        for kern in ("single", "pair", "default"):
            if kern == "default":
                os.environ.pop("QNN_TC_KERNEL", None)
            else:
                os.environ["QNN_TC_KERNEL"] = kern
            ms_l = _time_calls(torch, lambda i: qb.check(qb.qnn_qgemm(dl, sets[i % nsets][0], sets[i % nsets][1], thr_l, out_l)),
                               8, graph=True)
            row[kern + "_us"] = round(1e3 * ms_l, 1)
        row["tmacs_default"] = round(Mg * Ng * Kg / (row["default_us"] * 1e-6) / 1e12, 1)
        large.append(row)
        del sets, thr_l, out_l
    res["large_gemm"] = large
    # ---- config 5: M = K = 8192, N in {1, 4, 16}; W2A2 and W4A4
    M = K = 8192
    skinny = []
    for bits in (2, 4) if only in (None, "skinny") else ():
        c = synth.gemm_case(5000 + bits, M, 16, K, bits, bits)
        Wd = qb.to_device_logical(c.W, c.w_enc)
        thr = torch.from_numpy(c.thr).cuda()
        for fmt, afmt, name in SKINNY_FORMATS(qb):
            Wp = qb.pack(Wd, bits, c.w_enc, fmt)
            copies = max(2, int(300e6 // Wp.numel()) + 1)          # > 2 x L2 in rotation
            Wrot = [Wp] + [Wp.clone() for _ in range(copies - 1)]
            for N in (1, 4, 16):
                Ad = qb.to_device_logical(c.At[:N], c.a_enc)
                Ap = qb.pack(Ad, bits, c.a_enc, afmt)
                d = qb.qnn_gemm_desc(M, N, K, bits, bits, bits, c.w_enc, c.a_enc, fmt, afmt, I8, 0)
                out = torch.empty(qb.qnn_gemm_out_bytes(d, True), dtype=torch.uint8, device="cuda")
                ms = _time_calls(torch, lambda i: qb.check(qb.qnn_qgemm(d, Wrot[i % copies], Ap, thr, out)),
                                 4 * copies, graph=True)
                ms_warm = _time_calls(torch, lambda i: qb.check(qb.qnn_qgemm(d, Wp, Ap, thr, out)), 50, graph=True)
                alg = Wp.numel() + Ap.numel() + thr.numel() * 4 + N * M
                skinny.append({"w": bits, "a": bits, "N": N, "fmt": name, "us": 1e3 * ms, "us_l2_warm": 1e3 * ms_warm,
                               "algorithmic_bytes": alg, "gbs": alg / ms / 1e6,
                               "hbm_frac": alg / ms / 1e6 / peaks["hbm_gbs"], "tmacs": M * N * K / ms / 1e9})
            del Wrot
    res["skinny_fc"] = skinny

    # ---- config 3: conv2-shaped W1A2 layer via lowering, B = 1 and 64
    conv = []
    for B in (1, 64) if only in (None, "conv2") else ():
        c = synth.conv2_alexnet_case(B)
        for fmt, name in ((I8, "int8"), (PL, "bitplanes")):
            if fmt == PL:
                x = qb.pack(qb.to_device_logical(c.In.reshape(-1, c.C), c.a_enc), c.a_bits, c.a_enc, PL)
                pitch = 0
            else:
                x = torch.from_numpy(c.In.astype(np.uint8)).cuda()
                pitch = c.C
            Wp = qb.pack(qb.to_device_logical(c.Wt.reshape(c.OC, -1), c.w_enc), 1, c.w_enc, fmt)
            d = qb.qnn_conv_desc(B, 27, 27, 96, pitch, 256, 5, 5, 1, 2, 1, 2, 2, c.w_enc, c.a_enc, fmt, I8, 0)
            thr = torch.from_numpy(c.thr).cuda()
            ws = torch.empty(qb.qnn_conv_workspace_bytes(d), dtype=torch.uint8, device="cuda")
            out = torch.empty(qb.qnn_conv_out_bytes(d, True), dtype=torch.uint8, device="cuda")
            ms_low = _time_calls(torch, lambda i: qb.check(qb.qnn_im2col(d, x, ws)), 50, graph=True)
            ms_all = _time_calls(torch, lambda i: qb.check(qb.qnn_qconv(d, Wp, x, thr, out, ws, ws.numel())), 50,
                                 graph=True)
            low_bytes = qb.qnn_conv_lowered_bytes(d) + x.numel()
            conv.append({"B": B, "fmt": name, "im2col_us": 1e3 * ms_low, "im2col_gbs": low_bytes / ms_low / 1e6,
                         "qconv_us": 1e3 * ms_all, "images_per_s": B / ms_all * 1e3,
                         "tmacs": B * 729 * 256 * 2400 / ms_all / 1e9})
    res["conv2"] = conv

    # ---- config 4: AlexNet-shaped chain, B = 1 and 256
    net_res = []
    for B in ((1, 256) if not QUICK else (32,)) if only in (None, "alexnet") else ():
        net = synth.alexnet_case(B)
        for mode in ("auto", "tensor", "bitserial") if B == 1 else ("auto",):
            plan = AlexNetPlan(net, B, mode)
            img = torch.from_numpy(net.image.astype(np.uint8)).cuda()
            ms = _time_calls(torch, lambda i: plan.forward(img), 30 if B == 1 else 10)
            per_layer = {}
            for (kind, d, Wp, thr, out), name in zip(plan.steps, plan.names):
                x_in = img if name == "conv1" else prev
                if kind == "conv":
                    f = lambda i: qb.check(qb.qnn_qconv(d, Wp, x_in, thr, out, plan.workspace, plan.workspace.numel()))
                    per_layer[name + "_lowering"] = round(
                        1e3 * _time_calls(torch, lambda i: qb.check(qb.qnn_im2col(d, x_in, plan.workspace)), 20,
                                          graph=True), 2)
                elif kind == "pool":
                    f = lambda i: qb.check(qb.qnn_maxpool(d, x_in, out))
                else:
                    f = lambda i: qb.check(qb.qnn_qgemm(d, Wp, x_in, thr, out, None, 0))
                per_layer[name] = round(1e3 * _time_calls(torch, f, 20, graph=True), 2)
                prev = out
            if QUICK:
                ms_graph = ms
            else:
                graph, _ = plan.capture(img)
                ms_graph = _time_calls(torch, lambda i: graph.replay(), 30 if B == 1 else 10)
                del graph
            net_res.append({"B": B, "mode": mode, "ms": ms, "images_per_s": B / ms * 1e3,
                            "ms_graph": ms_graph, "images_per_s_graph": B / ms_graph * 1e3,
                            "launches": plan.launches_per_forward(), "per_layer_us": per_layer})
            del plan
    res["alexnet"] = net_res
    st, dev = qb.qnn_device_status()
    assert st == 0 and dev == 0
    print(json.dumps(res))


def run_shapes(args):
    """Size sweep of Section 4.1.2 of the paper: every (rows, depth, cols) in {2^6 .. 2^12}^3, for
    every (w, a) in {1..4}^2 (--pairs restricts them; weights bipolar when w = 1, else signed;
    activations unsigned), GEMM+threshold on 8-bit containers (tensor cores) and on bit planes
    (bit-serial kernels), each timed by replaying a CUDA graph of repeated calls.  Prints one JSON
    line per (w, a) with the per-shape times, the faster operand format and the kernel the library
    chose, and a summary line."""
    import torch
    import __graft_entry__ as ge
    ge.build()
    from paper_1709_04060_b200 import binding as qb
    torch.cuda.set_device(0)
    PL, I8 = qb.QNN_FMT_BITPLANES, qb.QNN_FMT_INT8
    dims = [2 ** e for e in range(6, 13)]
    if QUICK:
        dims = [64, 1024, 4096]
    g = torch.Generator(device="cuda").manual_seed(170904060)
    summary = []
    for (w, a) in PAIRS:
        w_enc = qb.QNN_ENC_BIPOLAR if w == 1 else qb.QNN_ENC_SIGNED
        a_enc = qb.QNN_ENC_UNSIGNED
        if w == 1:
            bigW = (2 * torch.randint(0, 2, (4096, 4096), dtype=torch.int8, device="cuda", generator=g) - 1).contiguous()
        else:
            bigW = torch.randint(-(1 << (w - 1)), 1 << (w - 1), (4096, 4096), dtype=torch.int8, device="cuda", generator=g)
        bigA = torch.randint(0, 1 << a, (4096, 4096), dtype=torch.uint8, device="cuda", generator=g)
        n_thr = (1 << a) - 1
        thr_all = torch.sort(torch.randint(-64, 65, (4096, n_thr), dtype=torch.int32, device="cuda", generator=g), dim=1).values.contiguous()
        rows = []
        for M in dims:
            for K in dims:
                Wl = bigW[:M, :K].contiguous()
                Wp = {f: qb.pack(Wl, w, w_enc, f) for f in (I8, PL)}
                thr = thr_all[:M].contiguous()
                for N in dims:
                    Al = bigA[4096 - N:, 4096 - K:].contiguous()
                    res = {"M": M, "K": K, "N": N}
                    for f, name in ((I8, "int8"), (PL, "bitplanes")):
                        Ap = qb.pack(Al, a, a_enc, f)
                        d = qb.gemm_desc(M, N, K, w, a, a, w_enc, a_enc, f, I8)
                        out = torch.empty(max(qb.qnn_gemm_out_bytes(d, True), 16), dtype=torch.uint8, device="cuda")
                        reps = 10 if M * N * K < 2 ** 30 else 3
                        ms = _time_calls(torch, lambda i: qb.check(qb.qnn_qgemm(d, Wp[f], Ap, thr, out)), reps, graph=True)
                        res[name + "_us"] = round(1e3 * ms, 2)
                        res[name + "_kernel"] = qb.qnn_qgemm_kernel(d, True)
                    res["gmacs_best"] = round(M * N * K / (min(res["int8_us"], res["bitplanes_us"]) * 1e-6) / 1e9, 1)
                    res["faster"] = "int8" if res["int8_us"] <= res["bitplanes_us"] else "bitplanes"
                    rows.append(res)
        ratios = sorted(r["bitplanes_us"] / r["int8_us"] for r in rows)
        line = {"workload": "shapes", "w": w, "a": a, "shapes": len(rows),
                "bitplanes_faster": sum(r["faster"] == "bitplanes" for r in rows),
                "ratio_bitplanes_over_int8": {"min": round(ratios[0], 2), "median": round(ratios[len(ratios) // 2], 2),
                                              "max": round(ratios[-1], 2)},
                "rows": rows}
        print(json.dumps(line), flush=True)
        summary.append({k: line[k] for k in ("w", "a", "shapes", "bitplanes_faster", "ratio_bitplanes_over_int8")})
    print(json.dumps({"workload": "shapes_summary", "summary": summary}))


# dram__bytes_read.sum + dram__bytes_write.sum of one 4096^3 W1A2 launch of the (CTA-pair)
# tensor-core kernel, from an ncu capture of that launch (the output codes were still in L2 when
# the capture ended, so the write counter is small; the partial sums that the pairs of the split
# last round exchange stay in L2 as well).
TRAFFIC_BYTES_PER_LAUNCH = 33677056 + 861440


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-alexnet", action="store_true", help="skip the AlexNet-shaped chain measurement")
    ap.add_argument("--no-other-configs", action="store_true",
                    help="skip the compact measurements of configurations 1, 3, 4 (per layer) and 5")
    ap.add_argument("--overlap", type=int, default=1,
                    help="1: activation packer on a second stream, overlapping the previous GEMM (default); 0: one stream")
    ap.add_argument("--extras-only", default=None, choices=["large", "skinny", "conv2", "alexnet"],
                    help="extras: run one group only")
    ap.add_argument("--quick", action="store_true",
                    help="extras: a couple of plain calls per case (for profiler captures; AlexNet at batch 32)")
    ap.add_argument("--workload", default="sweep", choices=["sweep", "extras", "shapes", "peaks"],
                    help="sweep: the headline line; extras: the other paper-shaped workloads (one GPU); "
                         "shapes: the 2^6..2^12 size sweep of both operand formats")
    ap.add_argument("--pairs", default=None,
                    help="restrict the sweep, e.g. '1x2,4x4' (profiling only; the default is all 16)")
    args = ap.parse_args()
    if args.pairs:
        PAIRS[:] = [tuple(int(v) for v in p.split("x")) for p in args.pairs.split(",")]
    if args.workload in ("extras", "shapes", "peaks"):
        global QUICK
        QUICK = args.quick
        {"extras": run_extras, "shapes": run_shapes, "peaks": run_peaks}[args.workload](args)
        return
    if args.impl == "reference":
        if args.steps is None:
            args.steps = 10
        run_reference(args)
    else:
        if args.steps is None:
            args.steps = 1000
        run_b200(args)


if __name__ == "__main__":
    main()
