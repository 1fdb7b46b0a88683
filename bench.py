#!/usr/bin/env python
"""Benchmark of the ENEC codec on B200: decompress / compress GB/s (uncompressed bytes) and compression ratio on
a seeded synthetic Llama-3-8B-shaped bf16 weight set.

One step = one pass of the whole hot path over the set: enec_compress (histogram, parameter search, split,
transform, group widths, Algorithm 2 packing, block-offset prefix sum) of every tensor, then enec_decompress
(unpack, reconstruct) of every tensor, tensor by tensor on one stream.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload llama8b|layer|tensor] [--impl reference]

Prints one JSON line (rank 0). `--impl reference` times the CPU oracle on a bounded sample instead.
"""
import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "bf16 weight decompress GB/s (uncompressed bytes); compress GB/s and compression ratio alongside"
WORKLOADS = {
    "llama8b": (3, "full 32-layer Llama-3-8B-shaped bf16 weight set, 291 tensors, 16.06 GB"),
    "layer": (2, "one Llama-3-8B-shaped decoder layer in bf16, 9 tensors, 436 MB"),
    "tensor": (1, "one bf16 tensor 1024x4096, 8 MB"),
    "layer_fp32": (7, "one OLMo-1B-shaped decoder layer in fp32, 7 tensors, 268 MB (side measurement)"),
    "heavy": (4, "heavy-tailed stress set: 64 fp16 + 64 bf16 tensors 4096x4096 (Laplace / Student-t, outliers, zeros), 4.3 GB"),
    "moe": (5, "many-small-tensor MoE set: 768 bf16 expert matrices + 4096 vectors of 2048, 4864 tensors, 4.4 GB; "
               "the step uses the batched entry points"),
    "olmo1b_fp32": (6, "OLMo-1B-shaped fp32 weight set, 115 tensors, 5.1 GB (side measurement: Sec. 6.2 fp32 support)"),
}
SMI_QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")


def dtype_code(dtype):
    """enec_dtype of a torch dtype."""
    return {"torch.bfloat16": 0, "torch.float16": 1, "torch.float32": 2}[str(dtype)]


def decode_traffic_per_element():
    """dram__bytes_read.sum + dram__bytes_write.sum of enec_decode_kernel per element, from the counters of the
    last ncu capture (a small text file kept beside the capture's summary), or None when the kernel's source has
    changed since the capture was taken."""
    import hashlib
    path = os.path.join(ROOT, "profiles", "decode_kernel_dram_counters.txt")
    try:
        rec = dict(line.split(":", 1) for line in open(path) if ":" in line and not line.startswith("#"))
        rec = {k.strip(): v.strip() for k, v in rec.items()}
        h = hashlib.sha256()
        for name in rec["source_files"].split():
            h.update(open(os.path.join(ROOT, "paper_2604_03298_b200", "csrc", name), "rb").read())
        if h.hexdigest() != rec["source_sha256"]:
            return None, "the decode kernel's source has changed since the ncu capture"
        per_elem = (float(rec["dram_bytes_read"]) + float(rec["dram_bytes_write"])) / float(rec["elements"])
        return per_elem, f"scaled per element from the ncu capture of {rec['workload']}"
    except Exception as e:   # no file, or not readable: no figure
        return None, f"no counters on file ({type(e).__name__})"


def launch_ranks(n, argv):
    """Starts this script again as n ranks on this node (torch.distributed.run, one process per GPU) and returns
    their exit code. The ranks find RANK / LOCAL_RANK / WORLD_SIZE / MASTER_* in their environment."""
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__), *argv]
    return subprocess.call(cmd)


def run_spawn_selftest(args):
    """The host logic of an N-rank run without any GPU: rendezvous (gloo), max / sum over ranks, one line from
    rank 0. Used by the CPU tests of the launch path."""
    import torch.distributed as dist
    from paper_2604_03298_b200 import runner
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo")
    slowest = runner.max_over_ranks(10.0 + rank)
    total = runner.sum_over_ranks(100.0)
    dist.barrier()
    if rank == 0:
        print(json.dumps({"spawn_selftest": True, "n_gpus": world, "max_over_ranks": slowest, "sum_over_ranks": total}))
    dist.destroy_process_group()


def measured_peak_gbs():
    """HBM copy bandwidth measured on this machine (generated file), else the stated fallback."""
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    def __init__(self, index):
        self.index = index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={SMI_QUERY}", "--format=csv,noheader,nounits",
                                          "-lms", "50", "-i", str(self.index)],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return None
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1])); mx.append(float(f[2]))
                except ValueError:
                    continue
                for nm, v in zip(names, f[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(nm)
            os.unlink(self.path)
        except Exception:
            pass
        if not sm:
            return None
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": max(mx), "samples": len(sm), "reasons": sorted(reasons)}


def host_words(t):
    """Raw bit patterns of a tensor as a flat numpy array on the host (uint16, or uint32 for fp32)."""
    import numpy as np
    import torch
    if t.element_size() == 4:
        return t.reshape(-1).view(torch.int32).cpu().numpy().view(np.uint32)
    return t.reshape(-1).view(torch.int16).cpu().numpy().view(np.uint16)


def oracle_module():
    sys.path.insert(0, os.path.join(ROOT, "oracle"))
    import enec_oracle
    enec_oracle.lib()
    return enec_oracle


def time_oracle(words_list, dt=0):
    """Single-threaded oracle over a list of numpy arrays of raw words (uint16, or uint32 for fp32). Returns (compress s, decompress s, raw bytes,
    stream bytes)."""
    oracle = oracle_module()
    tc = td = 0.0
    raw = comp = 0
    for w in words_list:
        t0 = time.perf_counter()
        s = oracle.compress(w, dt)
        t1 = time.perf_counter()
        back = oracle.decompress(s, dt, w.size)
        t2 = time.perf_counter()
        assert (back == w).all()
        tc += t1 - t0
        td += t2 - t1
        raw += w.nbytes
        comp += s.size
    return tc, td, raw, comp


def time_oracle_all_cores(words_list, dt):
    """Independent oracle instances over the tensors of the sample, one per host thread (the library calls run
    outside the interpreter lock). Returns (decompress GB/s, compress GB/s, threads used)."""
    from concurrent.futures import ThreadPoolExecutor
    oracle = oracle_module()
    workers = max(1, min(len(words_list), os.cpu_count() or 1))
    raw = sum(w.nbytes for w in words_list)
    with ThreadPoolExecutor(workers) as pool:
        t0 = time.perf_counter()
        streams = list(pool.map(lambda w: oracle.compress(w, dt), words_list))
        t1 = time.perf_counter()
        backs = list(pool.map(lambda sw: oracle.decompress(sw[0], dt, sw[1].size), zip(streams, words_list)))
        t2 = time.perf_counter()
    for w, back in zip(words_list, backs):
        assert (w == back).all()
    return raw / (t2 - t1) / 1e9, raw / (t1 - t0) / 1e9, workers


def time_cpu_simd(words_list, dt, expected_stream_bytes):
    """The AVX2 / multi-threaded CPU codec of baseline/cpu_simd on a list of word arrays: second pass over warm
    buffers. None when the host cannot run it."""
    import numpy as np
    sys.path.insert(0, os.path.join(ROOT, "baseline", "cpu_simd"))
    try:
        import enec_cpu
        if not enec_cpu.available():
            return None
        enec_cpu.lib()
    except Exception:
        return None
    bufs = [np.empty(enec_cpu.max_compressed_size(dt, w.size), dtype=np.uint8) for w in words_list]
    backs = [np.empty_like(w) for w in words_list]
    tc = td = 0.0
    for rep in range(2):   # the first pass touches the buffers' pages
        tc = td = 0.0
        sizes = []
        for w, buf, back in zip(words_list, bufs, backs):
            t0 = time.perf_counter()
            n = enec_cpu.compress_into(w, dt, buf)
            t1 = time.perf_counter()
            enec_cpu.decompress_into(buf, n, dt, back)
            t2 = time.perf_counter()
            tc += t1 - t0
            td += t2 - t1
            sizes.append(n)
    for w, back in zip(words_list, backs):
        assert (w == back).all()
    assert sum(sizes) == expected_stream_bytes, "the CPU codec's streams differ in size from the GPU's"
    raw = sum(w.nbytes for w in words_list)
    return {"value": raw / td / 1e9, "unit": "GB/s", "cores": os.cpu_count(), "kind": "AVX2 multi-threaded CPU codec",
            "compress": {"value": raw / tc / 1e9, "unit": "GB/s"}}


def run_reference(args):
    """The CPU oracle as it stands, on the host cores: each step compresses and decompresses a bounded sample of
    the workload (the four attention projections of one layer, 100 MB of bf16)."""
    import numpy as np
    import torch
    from paper_2604_03298_b200 import synth
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg, desc = WORKLOADS[args.workload]
    specs = synth.config_specs(cfg)
    big = [s for s in specs if s.numel >= 1 << 20]
    sample = [s for s in big if s.name.split(".")[-1] in ("q", "k", "v", "o")][:4] or big[:1]
    words = [host_words(synth.make_tensor(s, "cpu")) for s in sample]
    dt = dtype_code(sample[0].dtype)
    for _ in range(args.warmup):
        time_oracle(words[:1], dt)
    t_comp = t_dec = 0.0
    t_all0 = time.perf_counter()
    for _ in range(args.steps):
        tc, td, raw, comp = time_oracle(words, dt)
        t_comp += tc
        t_dec += td
    t_all = time.perf_counter() - t_all0
    dec_gbs = raw * args.steps / t_dec / 1e9
    sample_desc = f"{'+'.join(s.name for s in sample)} of the workload ({raw / 1e6:.0f} MB raw) per step"
    line = {
        "impl": "reference", "metric": METRIC, "value": dec_gbs, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": t_all / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u8", "data": "synthetic",
        "config": {"workload": desc, "sample": sample_desc},
        "compress": {"value": raw * args.steps / t_comp / 1e9, "unit": "GB/s"},
        "compression_ratio": raw / comp,
        "cpu_baseline": {"value": dec_gbs, "unit": "GB/s", "cores": 1, "kind": "oracle", "sample": sample_desc},
        "e2e": {"value": dec_gbs, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def run_ours(args):
    import numpy as np
    import torch
    import torch.distributed as dist
    import paper_2604_03298_b200 as enec
    from paper_2604_03298_b200 import runner, synth

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU path")
    if world != args.gpus:
        raise RuntimeError(f"--gpus {args.gpus} but {world} rank(s) are running: start it as `python bench.py --gpus N` "
                           "or under torch.distributed.run with --nproc-per-node N")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    enec.lib()  # fails loudly if libenec.so is missing

    cfg, desc = WORKLOADS[args.workload]
    batched_step = cfg == 5   # the set made for enec_compress_batched / enec_decompress_batched
    specs = synth.config_specs(cfg)
    # weak scaling: every rank holds a full copy of the set drawn with its own seeds
    import dataclasses
    specs = [dataclasses.replace(s, seed=s.seed + 100003 * rank) for s in specs]
    raw = [synth.make_tensor(s, "cuda") for s in specs]
    cs = runner.CodecSet.allocate(raw)
    raw_bytes = cs.raw_bytes

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # warm-up steps, then one verified round trip (outside the timed region)
    def compress_pass():
        if batched_step:
            cs.compress_batched()
        else:
            cs.compress_all(n_streams=args.streams)

    def decompress_pass():
        if batched_step:
            cs.decompress_batched()
        else:
            cs.decompress_all(n_streams=args.streams)

    for _ in range(max(args.warmup, 1)):
        compress_pass()
        decompress_pass()
    torch.cuda.synchronize()
    cs.check_status()
    cs.verify_roundtrip()
    comp_bytes = cs.compressed_bytes()

    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    try:
        gpu_id = "GPU-" + str(torch.cuda.get_device_properties(local).uuid)
    except Exception:
        gpu_id = str(local)
    sampler = ClockSampler(gpu_id)
    if rank == 0:
        sampler.start()
    launches0 = enec.enec_launch_count()
    barrier()
    t0 = time.perf_counter()
    for k in range(args.steps):
        ev[k][0].record()
        compress_pass()
        ev[k][1].record()
        decompress_pass()
        ev[k][2].record()
    barrier()
    wall_ms = (time.perf_counter() - t0) * 1e3
    launches = enec.enec_launch_count() - launches0
    clocks = sampler.stop() if rank == 0 else None
    cs.check_status()
    ms_comp = sum(e[0].elapsed_time(e[1]) for e in ev) / args.steps
    ms_dec = sum(e[1].elapsed_time(e[2]) for e in ev) / args.steps
    ms_step = ev[0][0].elapsed_time(ev[-1][2]) / args.steps
    dec_times = sorted(e[1].elapsed_time(e[2]) for e in ev)
    ms_dec_median = runner.max_over_ranks(dec_times[len(dec_times) // 2])
    ms_dec_best = runner.max_over_ranks(dec_times[0])
    ms_comp, ms_dec, ms_step = (runner.max_over_ranks(v) for v in (ms_comp, ms_dec, ms_step))
    total_raw = runner.sum_over_ranks(raw_bytes)
    total_comp = runner.sum_over_ranks(comp_bytes)
    total_launches = int(runner.sum_over_ranks(launches))

    # end to end through host buffers (pinned): host stream -> device -> decompress -> host tensor, and the
    # compress direction likewise, on a sample of this rank's set: its first tensors up to about 2 GB of raw bytes
    # (the link, not the codec, bounds this number, and pinning the whole set would take tens of GB of host memory)
    layer, e2e_budget = [], 2.2e9
    for i, t in enumerate(cs.raw):
        if specs[i].numel * t.element_size() > 600e6:
            continue   # the embedding alone would be the whole sample
        layer.append(i)
        e2e_budget -= specs[i].numel * t.element_size()
        if e2e_budget <= 0:
            break
    e2e_steps = max(1, min(args.steps, 5))
    h_streams = [torch.empty(int(cs.sizes[i].item()), dtype=torch.uint8).pin_memory() for i in layer]
    h_raw = [torch.empty(cs.raw[i].numel(), dtype=cs.raw[i].dtype).pin_memory() for i in layer]
    for h, i in zip(h_streams, layer):
        h.copy_(cs.streams[i][:h.numel()])
    for h, i in zip(h_raw, layer):
        h.copy_(cs.raw[i].reshape(-1))
    torch.cuda.synchronize()
    e2e_raw = sum(h.numel() * h.element_size() for h in h_raw)
    e2e_comp = sum(h.numel() for h in h_streams)

    # each tensor's copy in, codec call and copy out follow one another on one stream; with several streams the
    # copies of different tensors run in both directions of the link at once
    def e2e_decompress_one(j):
        i, h_in, h_out = layer[j], h_streams[j], h_raw[j]
        cs.streams[i][:h_in.numel()].copy_(h_in, non_blocking=True)
        st = enec.enec_decompress(cs.streams[i], h_in.numel(), dtype_code(cs.raw[i].dtype), cs.raw[i].numel(),
                                  cs.outs[i], cs.status)
        assert st == 0
        h_out.copy_(cs.outs[i], non_blocking=True)

    def e2e_compress_one(j):
        i, h_in, h_out = layer[j], h_raw[j], h_streams[j]
        cs.outs[i].copy_(h_in, non_blocking=True)
        st = enec.enec_compress(cs.outs[i], dtype_code(cs.raw[i].dtype), cs.raw[i].numel(),
                                cs.streams[i], cs.streams[i].numel(), cs.sizes[i:i + 1], cs.status)
        assert st == 0
        h_out.copy_(cs.streams[i][:h_out.numel()], non_blocking=True)

    def e2e_decompress():
        cs.spread(args.spread_streams, e2e_decompress_one, len(layer))

    def e2e_compress():
        cs.spread(args.spread_streams, e2e_compress_one, len(layer))

    def time_e2e(fn, steps=None):
        steps = steps or args.steps
        for _ in range(2):
            fn()
        barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(steps):
            fn()
        b.record()
        barrier()
        return runner.max_over_ranks(a.elapsed_time(b) / steps)

    # the same decompress pass as one batched launch (not part of `value`: the workload says tensor by tensor)

    def batched_pass():
        cs.decompress_batched()

    ms_batched = time_e2e(batched_pass)
    ms_comp_batched = time_e2e(cs.compress_batched)
    # the same steps again with the calls spread over several streams (the timed step itself keeps the
    # workload's "tensor by tensor on one stream" unless --streams says otherwise)
    for _ in range(2):
        cs.compress_all(n_streams=args.spread_streams)
        cs.decompress_all(n_streams=args.spread_streams)
    ev2 = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    barrier()
    for k in range(args.steps):
        ev2[k][0].record()
        cs.compress_all(n_streams=args.spread_streams)
        ev2[k][1].record()
        cs.decompress_all(n_streams=args.spread_streams)
        ev2[k][2].record()
    barrier()
    ms_comp_ms = runner.max_over_ranks(sum(e[0].elapsed_time(e[1]) for e in ev2) / args.steps)
    ms_dec_ms = runner.max_over_ranks(sum(e[1].elapsed_time(e[2]) for e in ev2) / args.steps)

    # ablation: the frequency-rank variant (table look-ups instead of the linear transform), same steps, one stream
    for _ in range(2):
        cs.compress_all(ranked=True)
        cs.decompress_all(ranked=True)
    torch.cuda.synchronize()
    cs.check_status()
    cs.verify_roundtrip()
    ranked_bytes = runner.sum_over_ranks(cs.compressed_bytes())
    ev3 = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    barrier()
    for k in range(args.steps):
        ev3[k][0].record()
        cs.compress_all(ranked=True)
        ev3[k][1].record()
        cs.decompress_all(ranked=True)
        ev3[k][2].record()
    barrier()
    ms_comp_ranked = runner.max_over_ranks(sum(e[0].elapsed_time(e[1]) for e in ev3) / args.steps)
    ms_dec_ranked = runner.max_over_ranks(sum(e[1].elapsed_time(e[2]) for e in ev3) / args.steps)
    # ablation: parameters per block (Sec. 5.5 on every block's own histogram), same steps, one stream
    for _ in range(2):
        cs.compress_all(blockwise=True)
        cs.decompress_all(blockwise=True)
    torch.cuda.synchronize()
    cs.check_status()
    cs.verify_roundtrip()
    blockwise_bytes = runner.sum_over_ranks(cs.compressed_bytes())
    ev4 = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    barrier()
    for k in range(args.steps):
        ev4[k][0].record()
        cs.compress_all(blockwise=True)
        ev4[k][1].record()
        cs.decompress_all(blockwise=True)
        ev4[k][2].record()
    barrier()
    ms_comp_blockwise = runner.max_over_ranks(sum(e[0].elapsed_time(e[1]) for e in ev4) / args.steps)
    ms_dec_blockwise = runner.max_over_ranks(sum(e[1].elapsed_time(e[2]) for e in ev4) / args.steps)

    # the same comparison on two side sets where parameters per block could matter: the heavy-tailed stress set
    # (a sample of it) and one Gaussian decoder layer with the generator's exact zeros left in
    def per_block_side_set(side_specs, keep_zeros):
        side_raw = [synth.make_tensor(sp, "cuda", keep_zeros=keep_zeros) for sp in side_specs]
        side = runner.CodecSet.allocate(side_raw)
        res = {"raw_bytes": side.raw_bytes, "tensors": len(side_raw)}
        for name, kw in (("per_tensor", {}), ("per_block", {"blockwise": True})):
            for _ in range(3):
                side.compress_all(**kw)
                side.decompress_all(**kw)
            torch.cuda.synchronize()
            side.check_status()
            side.verify_roundtrip()
            e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
            reps = 5
            e[0].record()
            for _ in range(reps):
                side.compress_all(**kw)
            e[1].record()
            for _ in range(reps):
                side.decompress_all(**kw)
            e[2].record()
            torch.cuda.synchronize()
            res[name] = {"compression_ratio": side.raw_bytes / side.compressed_bytes(),
                         "compress_gbs": side.raw_bytes * reps / (e[0].elapsed_time(e[1]) * 1e-3) / 1e9,
                         "decompress_gbs": side.raw_bytes * reps / (e[1].elapsed_time(e[2]) * 1e-3) / 1e9}
        return res

    per_block_sides = None
    if rank == 0:
        heavy = synth.config_specs(4)
        per_block_sides = {
            "heavy_tailed_sample": dict(per_block_side_set(heavy[:8] + heavy[32:40] + heavy[64:72] + heavy[96:104], False),
                                        sample="sample: 32 of the 128 tensors of the heavy-tailed stress set (8 each of "
                                               "fp16 Laplace, fp16 Student-t, bf16 Laplace, bf16 Student-t)"),
            "gaussian_layer_zeros_kept": dict(per_block_side_set(synth.config_specs(2), True),
                                              sample="one Llama-3-8B-shaped bf16 decoder layer, the normal generator's "
                                                     "exact zeros left in"),
        }

    cs.compress_all()      # back to the linear streams for what follows
    torch.cuda.synchronize()
    cs.check_status()
    cs.verify_roundtrip()

    ms_e2e_dec = time_e2e(e2e_decompress, e2e_steps)
    ms_e2e_comp = time_e2e(e2e_compress, e2e_steps)
    cs.check_status()
    for h, i in zip(h_raw, layer):  # the host copy of the last decompress must be the tensor
        assert (host_words(h) == host_words(cs.raw[i])).all()

    # side number: the ratio when the normal generator's rare exact zeros are left in (one zero sets the lowest
    # occupied exponent of its tensor to 0 and with it n = 8): the largest tensor of the set and the sample's tensors
    zeros_kept = None
    if rank == 0 and cfg in (1, 2, 3):
        biggest = max(range(len(specs)), key=lambda i: specs[i].numel)
        zr = zc = zeros = 0
        for i in sorted(set([biggest] + layer[:9])):
            t = synth.make_tensor(specs[i], "cuda", keep_zeros=True)
            zeros += int((t == 0).sum().item())
            st = enec.enec_compress(t, dtype_code(t.dtype), t.numel(), cs.streams[i], cs.streams[i].numel(),
                                    cs.sizes[i:i + 1], cs.status)
            assert st == 0
            zr += t.numel() * t.element_size()
            zc += int(cs.sizes[i].item())
            del t
        zeros_kept = {"compression_ratio": zr / zc, "exact_zeros": zeros, "raw_bytes": zr,
                      "sample": f"{len(set([biggest] + layer[:9]))} tensors: the largest of the set and one decoder layer"}
        cs.compress_all()
        torch.cuda.synchronize()
        cs.check_status()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_peak_gbs()
    n_dec = len({t.dtype for t in cs.raw}) if batched_step else len(cs.raw)   # decode launches of a step
    dec_moved = (raw_bytes + comp_bytes)                       # algorithmic bytes of one decompress pass (this rank)
    achieved = dec_moved / (ms_dec * 1e-3) / 1e9
    elems = sum(t.numel() for t in cs.raw)
    all_bf16 = all(t.dtype == torch.bfloat16 for t in cs.raw)   # the DRAM counters on file are bf16's
    traffic_per_elem, traffic_note = decode_traffic_per_element()
    roofline = {
        "kernel": "enec_decode_kernel", "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
        "frac": achieved / peak, "peak_kind": peak_kind + " copy bandwidth",
        "algorithmic_bytes_per_launch": dec_moved / n_dec, "launches_per_step": n_dec,
        "avg_launch_us": ms_dec * 1e3 / n_dec,
        "avg_launch_note": "duration of the decompress pass / its launches (launches of different streams overlap)",
        "traffic": traffic_per_elem * elems / n_dec if traffic_per_elem and all_bf16 else None,
        "traffic_note": traffic_note if all_bf16 else "the counters on file are for bf16 streams",
        "compress": {"achieved": (raw_bytes + comp_bytes) / (ms_comp * 1e-3) / 1e9,
                     "frac": (raw_bytes + comp_bytes) / (ms_comp * 1e-3) / 1e9 / peak,
                     "note": "algorithmic bytes = read raw once + write stream; the histogram pass reads raw again"},
    }

    # CPU baseline: the oracle on a bounded sample of the same workload (rank 0, N = 1 only)
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        sample_idx = [i for i, s in enumerate(specs) if s.numel >= 1 << 20 and s.name.startswith("l0.")][:7]
        if not sample_idx:   # no decoder layer in the set: its first tensor
            sample_idx = [0]
        words = [host_words(cs.raw[i]) for i in sample_idx]
        tc, td, sraw, scomp = time_oracle(words, dtype_code(cs.raw[sample_idx[0]].dtype))
        gpu_sizes = [int(cs.sizes[i].item()) for i in sample_idx]
        assert sum(gpu_sizes) == scomp, "GPU and oracle stream sizes differ on the sample"
        cpu = {"value": sraw / td / 1e9, "unit": "GB/s", "cores": 1, "kind": "oracle",
               "sample": f"sample: {len(sample_idx)} tensors of the workload ({sraw / 1e6:.0f} MB raw), single thread",
               "compress": {"value": sraw / tc / 1e9, "unit": "GB/s"}, "compression_ratio": sraw / scomp}
        all_dec, all_comp, all_threads = time_oracle_all_cores(words, dtype_code(cs.raw[sample_idx[0]].dtype))
        cpu["all_cores"] = {"value": all_dec, "unit": "GB/s", "cores": all_threads, "compress": {"value": all_comp, "unit": "GB/s"},
                            "note": "independent oracle instances, one tensor of the sample per host thread"}

    # a stronger host baseline beside the oracle: the vectorised, multi-threaded CPU codec on the same sample
    cpu_vec = None
    if cpu is not None:
        cpu_vec = time_cpu_simd(words, dtype_code(cs.raw[sample_idx[0]].dtype), scomp)

    line = {
        "metric": METRIC, "value": total_raw / (ms_dec * 1e-3) / 1e9, "unit": "GB/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "u8", "data": "synthetic",
        "config": {"workload": desc, "tensors_per_rank": len(cs.raw), "raw_bytes_per_rank": raw_bytes,
                   "step": "enec_compress_batched of the set, then enec_decompress_batched of the set, one stream"
                           if batched_step else
                           "enec_compress of every tensor, then enec_decompress of every tensor; tensor i on side "
                           f"stream i mod {args.streams}, forked from and joined to the timed stream with events"
                           if args.streams > 1 else
                           "enec_compress of every tensor, then enec_decompress of every tensor, one stream",
                   "streams": args.streams,
                   "value_is": "uncompressed bytes / time of the step's decompress pass",
                   "l2": "inputs larger than L2 (each pass streams the whole set)" if raw_bytes > 256e6 else
                         "set fits in L2: HBM fraction not meaningful",
                   "sharding": "replica per rank, no collective"},
        "ms_decompress_per_step": ms_dec, "ms_decompress_median": ms_dec_median, "ms_decompress_best": ms_dec_best,
        "ms_compress_per_step": ms_comp, "wall_ms_per_step": wall_ms / args.steps,
        "compress": {"value": total_raw / (ms_comp * 1e-3) / 1e9, "unit": "GB/s"},
        "roundtrip": {"value": total_raw / (ms_step * 1e-3) / 1e9, "unit": "GB/s"},
        "multi_stream": {"streams": args.spread_streams,
                         "decompress": {"value": total_raw / (ms_dec_ms * 1e-3) / 1e9, "unit": "GB/s",
                                        "roofline_frac": (total_raw + total_comp) / (ms_dec_ms * 1e-3) / 1e9 / peak / world},
                         "compress": {"value": total_raw / (ms_comp_ms * 1e-3) / 1e9, "unit": "GB/s"},
                         "note": "the same steps, same calls, tensor i on side stream i mod streams (forked "
                                 "from and joined to the timed stream with events): independent tensors need no "
                                 "ordering, so the start of one launch overlaps the end of another"},
        "decompress_batched": {
            "value": total_raw / (ms_batched * 1e-3) / 1e9, "unit": "GB/s",
            "launches_per_pass": len({t.dtype for t in cs.raw}),
            "note": "same streams through enec_decompress_batched (one launch per dtype of the set), passes timed "
                    "back to back"},
        "compress_batched": {"value": total_raw / (ms_comp_batched * 1e-3) / 1e9, "unit": "GB/s",
                             "launches_per_pass": 2 * len({t.dtype for t in cs.raw}),
                             "note": "same tensors through enec_compress_batched (one call per dtype of the set)"},
        "compression_ratio": total_raw / total_comp,
        "compression_ratio_zeros_kept": zeros_kept,
        "ablation_per_block": {
            "compression_ratio": total_raw / blockwise_bytes,
            "decompress": {"value": total_raw / (ms_dec_blockwise * 1e-3) / 1e9, "unit": "GB/s"},
            "compress": {"value": total_raw / (ms_comp_blockwise * 1e-3) / 1e9, "unit": "GB/s"},
            "side_sets": per_block_sides,
            "note": "enec_compress_blockwise / enec_decompress_blockwise tensor by tensor on one stream: the search of "
                    "Sec. 5.5 on every 16384-element block's own histogram, a 16-byte table entry per block; compare "
                    "compression_ratio and the one-stream rates of this workload"},
        "ablation_frequency_ranks": {
            "compression_ratio": total_raw / ranked_bytes,
            "decompress": {"value": total_raw / (ms_dec_ranked * 1e-3) / 1e9, "unit": "GB/s"},
            "compress": {"value": total_raw / (ms_comp_ranked * 1e-3) / 1e9, "unit": "GB/s"},
            "note": "enec_compress_ranked / enec_decompress_ranked tensor by tensor on one stream: stored value = rank of the "
                    "exponent by falling count, looked up in a table (Sec. 4.2, Algorithm 1; the ablation's V1)"},
        "roofline": roofline,
        "cpu_baseline": cpu,
        "cpu_vectorised": cpu_vec,
        "e2e": {"value": e2e_raw * world / (ms_e2e_dec * 1e-3) / 1e9, "unit": "GB/s",
                "h2d_bytes_per_step": e2e_comp, "d2h_bytes_per_step": e2e_raw,
                "workload": f"sample: the first {len(layer)} tensors of the set without its embedding ({e2e_raw / 1e9:.2f} GB raw), "
                            "tensor by tensor: pinned host stream -> device -> enec_decompress -> pinned host"
                            + (f", tensors spread over {args.spread_streams} streams" if args.spread_streams > 1 else ""),
                "steps": e2e_steps,
                "compress": {"value": e2e_raw * world / (ms_e2e_comp * 1e-3) / 1e9, "unit": "GB/s",
                             "h2d_bytes_per_step": e2e_raw, "d2h_bytes_per_step": e2e_comp}},
        "gpu_launches": total_launches,
        "clocks": clocks,
        "paper_context": "Ascend 910B2, Llama-3.1-8B bf16: CR 1.36, 376.8 / 219.4 GB/s compress / decompress",
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama8b", choices=sorted(WORKLOADS))
    ap.add_argument("--streams", type=int, default=1,
                    help="streams the per-tensor calls of the timed step are spread over (1 = one stream, as the "
                         "workload is defined)")
    ap.add_argument("--spread-streams", type=int, default=8,
                    help="streams of the extra multi-stream measurement and of the end-to-end pass")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--spawn-selftest", action="store_true", help=argparse.SUPPRESS)
    args = ap.parse_args()
    if args.gpus < 1:
        ap.error("--gpus must be at least 1")
    if args.impl == "reference":
        run_reference(args)
        return
    if args.gpus > 1 and "RANK" not in os.environ:
        # started by hand for several GPUs: become the launcher of N ranks, one per GPU
        if not args.spawn_selftest:
            import torch
            have = torch.cuda.device_count()
            if have < args.gpus:
                print(f"bench.py: --gpus {args.gpus} needs {args.gpus} CUDA devices, {have} visible", file=sys.stderr)
                sys.exit(2)
        sys.exit(launch_ranks(args.gpus, sys.argv[1:]))
    if args.spawn_selftest:
        run_spawn_selftest(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
