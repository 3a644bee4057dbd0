#!/usr/bin/env python
"""Benchmark of the Fastrack GPU hot path on B200.

One step = one pass of the whole hot path over one batch: GPU authenticated decryption
(AES-256-CTR keystream + XOR + per-chunk GHASH + tag compare) of a 256 MiB buffer cut into 4 MiB
chunks (K = 64).  `value` is payload GB/s with the ciphertext already resident in HBM; `e2e` is the
same metric through fastrack_pipelined_h2d with the ciphertext in pinned HOST memory (PCIe copies
inside the timed region) plus the device->host read of the K verdict words.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

N > 1: launched under torch.distributed.run, one rank per GPU; the path has no exchange step, so every
rank runs an independent replica on its own buffer (weak scaling) and value = total bytes / max time.
`--impl reference` times the CPU oracle (oracle/) on the host cores instead.
Prints ONE JSON line on rank 0.
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
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

LEN = 256 << 20
CHUNK = 4 << 20
METRIC = "decrypt_verify_throughput"
UNIT = "GB/s"
WORKLOAD = "AES-256-GCM multi-chain decrypt+verify, 256 MiB uniform random bytes, chunk 4 MiB (K=64)"

# Roofline of the fused kernel: it is bound by shared-memory lookups (one 128-byte wavefront per clock
# per SM), not by HBM.  Per 512-byte row (32 blocks, one warp): AES-256 needs at least 197 table
# lookups per block when the first two rounds are shared between the 256 blocks that differ only in
# the last counter byte (224 without that sharing), each one conflict-free wavefront per warp; GHASH
# with 8-bit tables needs 16 128-bit lookups per block = 64 wavefronts per warp.
SMS = 148
WAVEFRONTS_PER_ROW_BEST = 197 + 64
ROW_BYTES = 512
# dram__bytes_read.sum + dram__bytes_write.sum of one decrypt+verify launch on this exact workload, from the
# ncu capture summarised in profiles/fr_crypt_kernel_decrypt_verify_256MiB_chunk4MiB.md (algorithmic: 2 x 256 MiB).
DRAM_TRAFFIC_BYTES_PER_LAUNCH = 501.9e6


def build_bench_helper(source: str, target: str, shared: bool = False) -> str:
    """Compile one of the measurement helpers under bench/ (they are not part of the library) if it is stale."""
    src, out = os.path.join(ROOT, "bench", source), os.path.join(ROOT, "bench", target)
    deps = [src, os.path.join(ROOT, "include", "fastrack.h")]
    if not os.path.exists(out) or any(os.path.getmtime(out) < os.path.getmtime(d) for d in deps):
        nvcc = os.environ.get("NVCC", "nvcc")
        cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-o", out + ".tmp", src]
        if shared:
            cmd += ["-shared", "-Xcompiler", "-fPIC"]
        subprocess.check_call(cmd)
        os.replace(out + ".tmp", out)
    return out


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "sm_max_mhz": float(p.get("sm_max_mhz", 1965.0)), "source": "measured"}
    return {"hbm_gbs": 6650.0, "sm_max_mhz": 1965.0, "source": "fallback"}


class ClockSampler:
    """nvidia-smi samples (SM clock, throttle reasons) taken while the timed regions run."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.samples, self.proc, self.thread = [], None, None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={gpu_index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            parts = [x.strip() for x in line.split(",")]
            if len(parts) >= 7:
                self.samples.append((time.time(), parts))

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()

    def summary(self, windows):
        inside = [p for t, p in self.samples if any(a <= t <= b for a, b in windows)]
        use = inside if inside else [p for _, p in self.samples]
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": len(inside)}
        if not use:
            return out
        try:
            out["sm_mhz"] = statistics.median(float(p[0]) for p in use)
            out["sm_max_mhz"] = max(float(p[1]) for p in use)
            out["power_w_max"] = max(float(p[2]) for p in use)
        except ValueError:
            pass
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        out["reasons"] = [n for i, n in enumerate(names) if any(p[3 + i].lower().startswith("active") for p in use)]
        return out


class OracleSample:
    """A bounded sample of the workload for the CPU oracle: `n_chunks` chunks of `chunk` bytes each
    (chunk <= 4 MiB; the oracle's cost is linear in bytes), encrypted once, decrypted+verified per step."""

    def __init__(self, n_chunks: int, chunk: int, threads: int):
        import oracle
        from paper_2410_15240_b200 import synth
        self.oracle, self.threads, self.chunk = oracle, threads, chunk
        self.key, self.iv = synth.key_and_iv(4)
        self.n = n_chunks * chunk
        self.plain = synth.random_bytes(self.n, 4)
        self.cipher, self.tags = oracle.mc_encrypt(self.key, self.iv, chunk, self.plain, threads)

    def step(self) -> float:
        t0 = time.perf_counter()
        back, ok = self.oracle.mc_decrypt(self.key, self.iv, self.chunk, self.cipher, self.tags, self.threads)
        dt = time.perf_counter() - t0
        assert ok.all() and (back == self.plain).all()
        return dt


def run_reference(args):
    """The reference arm: the CPU oracle, as it stands, on the host cores (rank 0 only).

    Each step decrypts+verifies one chunk per host thread; the chunk is the workload's 4 MiB when the
    requested number of steps allows it, otherwise shortened so that the timed region stays near a minute."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import oracle
    threads = oracle.host_threads()
    calib = OracleSample(threads, 64 << 10, threads)
    rate = calib.n / min(calib.step() for _ in range(2))           # bytes/s over all threads
    budget_s = 60.0
    chunk = int(budget_s * rate / max(1, args.steps) / threads) // 16 * 16
    chunk = max(64 << 10, min(CHUNK, chunk))
    sample = OracleSample(threads, chunk, threads)
    for _ in range(args.warmup):
        calib.step()
    times = [sample.step() for _ in range(args.steps)]
    total = sum(times)
    value = sample.n * len(times) / total / 1e9
    what = f"{threads} chunks of {chunk} bytes per step (workload chunk: {CHUNK}), {threads} threads over chunks"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": total / len(times) * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "u8", "data": "synthetic",
        "config": {"workload": WORKLOAD, "bytes_per_step": sample.n},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": what},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


class Ranks:
    """One process per GPU; the path has no exchange step, so the ranks are independent replicas and the only
    collectives are the barrier around the timed region and the MAX of the per-rank times."""

    def __init__(self, backend: str, device: str):
        self.rank = int(os.environ.get("RANK", "0"))
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.local = int(os.environ.get("LOCAL_RANK", "0"))
        self.device = device
        self.dist = None
        if self.world > 1:
            import torch
            import torch.distributed as dist
            kwargs = {"device_id": torch.device("cuda", self.local)} if backend == "nccl" else {}
            dist.init_process_group(backend, **kwargs)
            self.dist = dist

    def barrier(self):
        import torch
        if self.device == "cuda":
            torch.cuda.synchronize()
        if self.dist is not None:
            self.dist.barrier()
        if self.device == "cuda":
            torch.cuda.synchronize()

    def max_over_ranks(self, x: float) -> float:
        if self.dist is None:
            return x
        import torch
        t = torch.tensor([x], dtype=torch.float64, device=self.device)
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return float(t.item())

    def aggregate_throughput(self, bytes_per_rank: int, seconds_this_rank: float) -> float:
        """Whole-job bytes per second: every rank moved bytes_per_rank, the job took the slowest rank's time."""
        return self.world * bytes_per_rank / self.max_over_ranks(seconds_this_rank)

    def close(self):
        if self.dist is not None:
            self.dist.destroy_process_group()


def build_pipeline_timing() -> str:
    """Compile bench/pipeline_timing.c (plain C: the library header and the CUDA runtime only) if it is stale."""
    from paper_2410_15240_b200 import build as lib_build
    lib = lib_build.build()
    cuda = os.environ.get("CUDA_HOME", "/usr/local/cuda")
    src, out = os.path.join(ROOT, "bench", "pipeline_timing.c"), os.path.join(ROOT, "bench", "pipeline_timing")
    deps = [src, os.path.join(ROOT, "include", "fastrack.h"), lib]
    if not os.path.exists(out) or any(os.path.getmtime(out) < os.path.getmtime(d) for d in deps):
        subprocess.check_call(["gcc", "-std=c99", "-O2", "-Wall", "-I", os.path.join(ROOT, "include"), "-I", os.path.join(cuda, "include"),
                               src, "-o", out + ".tmp", lib, "-L", os.path.join(cuda, "lib64"), "-lcudart",
                               "-Wl,-rpath," + os.path.dirname(lib), "-Wl,-rpath," + os.path.join(cuda, "lib64")])
        os.replace(out + ".tmp", out)
    return out


def pipeline_timing(direction: str, length: int, cells, reps: int, batches: int):
    """Run the C harness on a list of (chunk_bytes, n_streams) cells; returns its JSON objects."""
    exe = build_pipeline_timing()
    cmd = [exe, direction, str(length), str(reps), str(batches)] + [f"{cb}:{ns}" for cb, ns in cells]
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=600)
    if out.returncode != 0:
        raise RuntimeError(f"pipeline_timing failed ({out.returncode}): {out.stderr[-500:]}")
    return [json.loads(line) for line in out.stdout.splitlines() if line.startswith("{")]


def traffic_from_profile():
    """dram__bytes_read.sum + dram__bytes_write.sum of one launch of the headline kernel, from the committed ncu
    summary (a line `dram_bytes_per_launch = <number>`); None when the file does not carry it."""
    import re
    path = os.path.join(ROOT, "profiles", "fr_crypt_kernel_decrypt_verify_256MiB_chunk4MiB.md")
    try:
        m = re.search(r"dram_bytes_per_launch\s*=\s*([0-9.eE+]+)", open(path).read())
        return (float(m.group(1)), os.path.relpath(path, ROOT)) if m else (None, None)
    except OSError:
        return None, None


def run_gpu(args):
    import numpy as np
    import torch
    from paper_2410_15240_b200 import fastrack, synth

    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback (use --impl reference for the oracle)")
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    ranks = Ranks("nccl", "cuda")
    rank, world, local = ranks.rank, ranks.world, ranks.local
    barrier, max_over_ranks = ranks.barrier, ranks.max_over_ranks
    pk = peaks()
    alu_peak = SMS * ROW_BYTES * pk["sm_max_mhz"] * 1e6 / WAVEFRONTS_PER_ROW_BEST / 1e9

    key, iv = synth.key_and_iv(4)
    K = LEN // CHUNK
    ctx = fastrack.Context(key, CHUNK)
    stream = torch.cuda.current_stream()
    st = stream.cuda_stream

    # inputs: random payload, encrypted once on the GPU (bench input, not a parity claim)
    plain_h = torch.from_numpy(synth.random_bytes(LEN, 4, salt=rank)).pin_memory()
    d_plain_src = plain_h.cuda()
    d_cipher = torch.empty_like(d_plain_src)
    d_tags = torch.empty(16 * K, dtype=torch.uint8, device="cuda")
    ctx.encrypt_tag(iv, d_plain_src.data_ptr(), LEN, d_cipher.data_ptr(), d_tags.data_ptr(), st)
    d_out = torch.empty_like(d_cipher)
    d_ok = torch.zeros(K, dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    h_cipher = d_cipher.cpu().pin_memory()
    h_tags = d_tags.cpu().pin_memory()
    h_ok = torch.zeros(K, dtype=torch.int32).pin_memory()

    def step():
        ctx.decrypt_verify(iv, d_cipher.data_ptr(), LEN, d_tags.data_ptr(), d_out.data_ptr(), d_ok.data_ptr(), st)

    if args.kernel_only and args.kernel_pass != "decrypt_verify":       # profiling aid: another pass over the same buffers
        if args.kernel_pass == "encrypt_tag":
            d_tags2 = torch.empty_like(d_tags)

            def step():
                ctx.encrypt_tag(iv, d_plain_src.data_ptr(), LEN, d_out.data_ptr(), d_tags2.data_ptr(), st)
        elif args.kernel_pass == "ctr_crypt":
            def step():
                ctx.ctr_crypt(iv, d_cipher.data_ptr(), LEN, d_out.data_ptr(), st)
        else:
            def step():
                ctx.verify(iv, d_cipher.data_ptr(), LEN, d_tags.data_ptr(), d_ok.data_ptr(), st)

    def e2e_step():
        ctx.pipelined_h2d(iv, h_cipher.data_ptr(), LEN, h_tags.data_ptr(), d_out.data_ptr(), d_ok.data_ptr(), args.streams)
        h_ok.copy_(d_ok, non_blocking=True)
        torch.cuda.current_stream().synchronize()

    sampler = ClockSampler(local) if rank == 0 else None
    windows = []
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def timed_batch(fn, n):
        """Exactly n calls between two events on the launching stream, a barrier and a synchronise on both sides;
        returns milliseconds (this rank)."""
        barrier()
        w0 = time.time()
        e0.record(stream)
        for _ in range(n):
            fn()
        e1.record(stream)
        barrier()
        windows.append((w0, time.time()))
        return e0.elapsed_time(e1)

    # ---- device-resident metric: batches of exactly `steps` steps, CUDA events on the launching stream, max over ranks
    for _ in range(args.warmup):
        step()
    launches0 = ctx.launches
    batch_ms = [max_over_ranks(timed_batch(step, args.steps)) for _ in range(args.batches)]
    gpu_launches = ctx.launches - launches0
    ms_total = statistics.median(batch_ms)
    ms_per_step = ms_total / args.steps
    if not (args.kernel_only and args.kernel_pass in ("encrypt_tag", "ctr_crypt")):
        assert bool((d_ok == 1).all()), "verification failed inside the benchmark"
    if not (args.kernel_only and args.kernel_pass in ("encrypt_tag", "verify")):
        assert bool((d_out == d_plain_src).all()), "decryption mismatch inside the benchmark"
    if args.kernel_only and args.kernel_pass == "encrypt_tag":
        assert bool((d_out == d_cipher).all()) and bool((d_tags2 == d_tags).all()), "encryption mismatch inside the benchmark"
    value = world * LEN * args.steps / (ms_total * 1e-3) / 1e9

    if args.kernel_only:
        if sampler is not None:
            sampler.stop()
        if rank == 0:
            print(json.dumps({"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                              "warmup": args.warmup, "ms_per_step": ms_per_step, "gpu_launches": gpu_launches,
                              "config": {"workload": WORKLOAD, "pass": args.kernel_pass}, "kernel_only": True}))
        ctx.close()
        ranks.close()
        return

    # ---- encrypt+tag (mirror path), same size
    enc_steps = max(3, min(args.steps, 50))

    def enc_step():
        ctx.encrypt_tag(iv, d_plain_src.data_ptr(), LEN, d_out.data_ptr(), d_tags.data_ptr(), st)
    for _ in range(3):
        enc_step()
    enc_ms = statistics.median(max_over_ranks(timed_batch(enc_step, enc_steps)) for _ in range(args.batches))
    enc_gbs = world * LEN * enc_steps / (enc_ms * 1e-3) / 1e9

    # ---- end to end: pinned host ciphertext -> pipelined H2D + decrypt/verify -> verdicts back on the host
    e2e_steps = max(3, min(args.steps, 30))
    for _ in range(3):
        e2e_step()

    def wall_batch(fn, n):
        barrier()
        w0 = time.time()
        t0 = time.perf_counter()
        for _ in range(n):
            fn()
        torch.cuda.synchronize()
        dt = max_over_ranks(time.perf_counter() - t0)
        windows.append((w0, time.time()))
        return dt
    e2e_batches = [wall_batch(e2e_step, e2e_steps) for _ in range(args.batches)]
    e2e_s = statistics.median(e2e_batches)
    assert bool((h_ok == 1).all())
    e2e_gbs = world * LEN / (e2e_s / e2e_steps) / 1e9

    # ---- raw pinned cudaMemcpyAsync of the same bytes, same run (what the pipeline is compared with)
    def raw_step():
        d_out.copy_(h_cipher, non_blocking=True)
        torch.cuda.current_stream().synchronize()
    raw_s = statistics.median(wall_batch(raw_step, e2e_steps) for _ in range(args.batches))
    raw_gbs = world * LEN / (raw_s / e2e_steps) / 1e9

    # ---- mirror pipeline: GPU encrypt+tag -> pinned host (device->host copies overlapped)
    def d2h_step():
        ctx.pipelined_d2h(iv, d_plain_src.data_ptr(), LEN, d_out.data_ptr(), h_cipher.data_ptr(), h_tags.data_ptr(), args.streams)
    d2h_s = statistics.median(wall_batch(d2h_step, e2e_steps) for _ in range(args.batches))
    d2h_gbs = world * LEN / (d2h_s / e2e_steps) / 1e9
    ctx.close()
    del d_plain_src, d_cipher, d_out, h_cipher, plain_h

    # ---- the other configurations (rank 0, single GPU): paper-sized launches, chain sweep, pipelined transfers
    extra = {"encrypt_tag_gbs": enc_gbs, "pipelined_d2h_encrypt_gbs": d2h_gbs}
    if rank == 0 and world == 1 and not args.headline_only:
        extra.update(other_configs(args, alu_peak, windows))

    if sampler is not None:
        sampler.stop()
    if rank == 0:
        clocks = sampler.summary(windows)
        per_gpu = value / world
        hbm_payload_peak = pk["hbm_gbs"] / 2.0
        traffic, traffic_source = traffic_from_profile()
        import oracle
        threads = oracle.host_threads()
        n_sample = max(1, min(64, threads))
        cpu_s = OracleSample(n_sample, CHUNK, threads).step()
        cpu_gbs = n_sample * CHUNK / cpu_s / 1e9
        cpu_one_gbs = CHUNK / OracleSample(1, CHUNK, 1).step() / 1e9       # the same oracle on one thread, one chunk
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "u8", "data": "synthetic",
            "config": {"workload": WORKLOAD, "len_bytes": LEN, "chunk_bytes": CHUNK, "chains": K,
                       "l2": "inputs larger than L2 (256 MiB in + 256 MiB out per step)",
                       "parallelism": "replicas only" if world > 1 else "single GPU", "pipeline_streams": args.streams},
            "timing": {"batches": args.batches, "steps_per_batch": args.steps, "value_from": "median batch",
                       "ms_per_step_min": min(batch_ms) / args.steps, "ms_per_step_max": max(batch_ms) / args.steps},
            "clocks": clocks,
            "e2e": {"value": e2e_gbs, "unit": UNIT, "h2d_bytes_per_step": LEN + 16 * K, "d2h_bytes_per_step": 4 * K,
                    "steps": e2e_steps, "batches": args.batches, "raw_pinned_h2d_gbs": raw_gbs,
                    "fraction_of_raw_pcie": e2e_gbs / raw_gbs,
                    "value_min": world * LEN / (max(e2e_batches) / e2e_steps) / 1e9,
                    "value_max": world * LEN / (min(e2e_batches) / e2e_steps) / 1e9},
            "gpu_launches": gpu_launches,
            "roofline": {"bound": "alu", "achieved": per_gpu, "peak": alu_peak, "unit": "GB/s", "frac": per_gpu / alu_peak,
                         "traffic": traffic, "traffic_source": traffic_source,
                         "peak_source": f"shared-memory lookup rate: {SMS} SMs x 1 wavefront/clk x {pk['sm_max_mhz']:.0f} MHz x "
                                        f"{ROW_BYTES} B per {WAVEFRONTS_PER_ROW_BEST} wavefronts (payload GB/s)",
                         "hbm": {"achieved": 2 * per_gpu, "peak": pk["hbm_gbs"], "frac": 2 * per_gpu / pk["hbm_gbs"],
                                 "unit": "GB/s", "peak_source": f"{pk['source']} copy bandwidth",
                                 "payload_peak": hbm_payload_peak}},
            "cpu_baseline": {"value": cpu_gbs, "unit": UNIT, "cores": threads, "kind": "oracle",
                             "sample": f"{n_sample} of the 64 chunks (4 MiB each), {threads} threads over chunks, {cpu_s:.1f} s",
                             "one_thread_value": cpu_one_gbs},
            "extra": extra,
        }
        print(json.dumps(line))
    ranks.close()


def other_configs(args, alu_peak, windows):
    """Benchmark configurations beside the headline cell, for the `extra` object of the bench line.  Device-resident
    cells: median of `batches` batches of back-to-back calls, CUDA events on the launching stream.  Pipelined cells:
    the C harness under bench/ (wall clock around the blocking calls, raw copy in the same process)."""
    import torch
    from paper_2410_15240_b200 import fastrack, synth
    key, iv = synth.key_and_iv(1)
    stream = torch.cuda.current_stream()
    st = stream.cuda_stream
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def timed(fn, n_bytes):
        reps = max(5, min(100, int(1.5e9 // max(n_bytes, 1))))
        for _ in range(3):
            fn()
        out = []
        for _ in range(args.batches):
            torch.cuda.synchronize()
            w0 = time.time()
            e0.record(stream)
            for _ in range(reps):
                fn()
            e1.record(stream)
            torch.cuda.synchronize()
            windows.append((w0, time.time()))
            out.append(e0.elapsed_time(e1) / reps * 1e-3)
        return out

    def gbs(n, ts):
        return {"gbs": n / statistics.median(ts) / 1e9, "gbs_min": n / max(ts) / 1e9, "gbs_max": n / min(ts) / 1e9,
                "us": statistics.median(ts) * 1e6, "frac_of_roofline": n / statistics.median(ts) / 1e9 / alu_peak}

    def device_cell(n, cb):
        K = (n + cb - 1) // cb
        with fastrack.Context(key, cb) as ctx:
            d_p = torch.randint(0, 256, (n,), dtype=torch.uint8, device="cuda")
            d_c, d_o = torch.empty_like(d_p), torch.empty_like(d_p)
            d_t = torch.empty(16 * K, dtype=torch.uint8, device="cuda")
            d_ok = torch.zeros(K, dtype=torch.int32, device="cuda")
            t_enc = timed(lambda: ctx.encrypt_tag(iv, d_p.data_ptr(), n, d_c.data_ptr(), d_t.data_ptr(), st), n)
            t_dec = timed(lambda: ctx.decrypt_verify(iv, d_c.data_ptr(), n, d_t.data_ptr(), d_o.data_ptr(), d_ok.data_ptr(), st), n)
            assert bool((d_ok == 1).all()) and bool((d_o == d_p).all())
        return {"len": n, "chunk": cb, "K": K, "decrypt_verify": gbs(n, t_dec), "encrypt_tag": gbs(n, t_enc)}

    def sample_batch_cell(sample_bytes, n_samples, chains):
        cb = (sample_bytes // chains + 15) // 16 * 16
        with fastrack.Context(key, cb) as ctx:
            ctx.set_framing(chains)
            n = sample_bytes * n_samples
            K = n_samples * ((sample_bytes + cb - 1) // cb)
            d_iv = torch.randint(0, 256, (12 * n_samples,), dtype=torch.uint8, device="cuda")
            d_p = torch.randint(0, 256, (n,), dtype=torch.uint8, device="cuda")
            d_c, d_o = torch.empty_like(d_p), torch.empty_like(d_p)
            d_t = torch.empty(16 * K, dtype=torch.uint8, device="cuda")
            d_ok = torch.zeros(K, dtype=torch.int32, device="cuda")
            ctx.encrypt_tag_samples(d_iv.data_ptr(), sample_bytes, n_samples, d_p.data_ptr(), d_c.data_ptr(), d_t.data_ptr(), st)
            t_dec = timed(lambda: ctx.decrypt_verify_samples(d_iv.data_ptr(), sample_bytes, n_samples, d_c.data_ptr(),
                                                             d_t.data_ptr(), d_o.data_ptr(), d_ok.data_ptr(), st), n)
            assert bool((d_ok == 1).all()) and bool((d_o == d_p).all())
        return {"sample_bytes": sample_bytes, "n_samples": n_samples, "chains_per_sample": chains, "chunk": cb, "len": n,
                "decrypt_verify": gbs(n, t_dec)}

    out = {"timing": f"median of {args.batches} batches of back-to-back calls per cell, min and max beside it"}
    # paper-sized launches (Sections 5.1 / 5.2: batches of tens of MB), 4 MiB chunks, and a ResNet-style batch of
    # 64 fp16 images cut into 16 chains each under per-image IVs
    out["paper_sized"] = [device_cell(n, 4 << 20) for n in (4 << 20, 16 << 20, 64 << 20)]
    out["sample_batch"] = sample_batch_cell(3 * 224 * 224 * 2, 64, 16)
    # config 1: 64 MiB cut into K = 1 .. 1024 chains
    out["config1_chain_sweep"] = [device_cell(64 << 20, (64 << 20) // k) for k in (1, 4, 16, 64, 256, 1024)]
    # many chains at the headline size: 16 KiB chunks against 4 MiB chunks
    out["chunk_16KiB"] = [device_cell(n, 16 << 10) for n in (64 << 20, 256 << 20)]
    # chunks below the benchmark's range at the headline size (samples of tens to thousands of bytes): the planner picks the
    # packed rows for the small ones and the row kernels with folded tails from 4 KiB up
    out["small_chunks_256MiB"] = [device_cell(256 << 20, cb) for cb in (64, 256, 1024, 4096)]
    # config 3: 670 MB of bf16-sized state, device-resident, and the mirror pipeline
    out["config3_device"] = device_cell(670_000_000, 4 << 20)
    torch.cuda.empty_cache()
    # config 2: the 77 MB fp16 image batch through fastrack_pipelined_h2d, 4 chunk sizes x 2-4 streams
    w0 = time.time()
    cells = [(cb, ns) for cb in (256 << 10, 1 << 20, 4 << 20, 8 << 20) for ns in (2, 3, 4)]
    out["config2_pipelined_h2d"] = pipeline_timing("h2d", 77_070_336, cells, 10, args.batches)
    out["config3_pipelined_d2h"] = pipeline_timing("d2h", 670_000_000, [(4 << 20, 2), (4 << 20, 4)], 3, args.batches)
    out["small_transfers_h2d"] = [pipeline_timing("h2d", n, [(65536, 2)], 50, args.batches)[0]
                                  for n in (256 << 10, 1 << 20, 4 << 20, 16 << 20)]
    windows.append((w0, time.time()))
    return out


def run_sweep(args):
    """Device-resident and pipelined throughput over the benchmark configurations (one JSON line per cell)."""
    import torch
    from paper_2410_15240_b200 import fastrack, synth
    torch.cuda.set_device(0)
    key, iv = synth.key_and_iv(1)
    stream = torch.cuda.current_stream()

    def timed(fn, reps):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(reps):
            fn()
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps * 1e-3

    def device_cell(n, cb, label):
        K = (n + cb - 1) // cb
        with fastrack.Context(key, cb) as ctx:
            d_p = torch.randint(0, 256, (n,), dtype=torch.uint8, device="cuda")
            d_c, d_o = torch.empty_like(d_p), torch.empty_like(d_p)
            d_t = torch.empty(16 * K, dtype=torch.uint8, device="cuda")
            d_ok = torch.zeros(K, dtype=torch.int32, device="cuda")
            st = stream.cuda_stream
            reps = max(5, min(200, int(2e9 // max(n, 1))))
            t_enc = timed(lambda: ctx.encrypt_tag(iv, d_p.data_ptr(), n, d_c.data_ptr(), d_t.data_ptr(), st), reps)
            t_dec = timed(lambda: ctx.decrypt_verify(iv, d_c.data_ptr(), n, d_t.data_ptr(), d_o.data_ptr(),
                                                     d_ok.data_ptr(), st), reps)
            assert bool((d_ok == 1).all()) and bool((d_o == d_p).all())
        print(json.dumps({"cell": label, "len": n, "chunk": cb, "K": K, "decrypt_verify_gbs": n / t_dec / 1e9,
                          "encrypt_tag_gbs": n / t_enc / 1e9, "decrypt_us": t_dec * 1e6}), flush=True)

    def pipeline_cell(n, cb, n_streams, label):
        K = (n + cb - 1) // cb
        with fastrack.Context(key, cb) as ctx:
            d_p = torch.randint(0, 256, (n,), dtype=torch.uint8, device="cuda")
            d_c = torch.empty_like(d_p)
            d_t = torch.empty(16 * K, dtype=torch.uint8, device="cuda")
            d_ok = torch.zeros(K, dtype=torch.int32, device="cuda")
            ctx.encrypt_tag(iv, d_p.data_ptr(), n, d_c.data_ptr(), d_t.data_ptr(), stream.cuda_stream)
            torch.cuda.synchronize()
            h_c, h_t = d_c.cpu().pin_memory(), d_t.cpu().pin_memory()
            d_o = torch.empty_like(d_p)
            reps = 20

            def wall(fn):
                """best of 5 batches (host and PCIe noise on a shared box only ever adds time)"""
                for _ in range(3):
                    fn()
                best = float("inf")
                for _ in range(5):
                    torch.cuda.synchronize()
                    t0 = time.perf_counter()
                    for _ in range(reps // 2):
                        fn()
                    torch.cuda.synchronize()
                    best = min(best, (time.perf_counter() - t0) / (reps // 2))
                return best

            t_pipe = wall(lambda: ctx.pipelined_h2d(iv, h_c.data_ptr(), n, h_t.data_ptr(), d_o.data_ptr(),
                                                    d_ok.data_ptr(), n_streams))
            assert bool((d_ok == 1).all()) and bool((d_o == d_p).all())

            def raw():
                d_o.copy_(h_c, non_blocking=True)
                torch.cuda.current_stream().synchronize()
            t_raw = wall(raw)
        print(json.dumps({"cell": label, "len": n, "chunk": cb, "K": K, "streams": n_streams,
                          "pipelined_h2d_gbs": n / t_pipe / 1e9, "raw_pinned_h2d_gbs": n / t_raw / 1e9,
                          "fraction_of_raw": t_raw / t_pipe}), flush=True)

    def d2h_cell(n, cb, n_streams, label):
        K = (n + cb - 1) // cb
        with fastrack.Context(key, cb) as ctx:
            d_p = torch.randint(0, 256, (n,), dtype=torch.uint8, device="cuda")
            d_c = torch.empty_like(d_p)
            h_c = torch.empty(n, dtype=torch.uint8).pin_memory()
            h_t = torch.empty(16 * K, dtype=torch.uint8).pin_memory()
            reps = 10

            def wall(fn):
                for _ in range(2):
                    fn()
                best = float("inf")
                for _ in range(3):
                    torch.cuda.synchronize()
                    t0 = time.perf_counter()
                    for _ in range(reps // 2):
                        fn()
                    torch.cuda.synchronize()
                    best = min(best, (time.perf_counter() - t0) / (reps // 2))
                return best

            t_pipe = wall(lambda: ctx.pipelined_d2h(iv, d_p.data_ptr(), n, d_c.data_ptr(), h_c.data_ptr(), h_t.data_ptr(),
                                                    n_streams))

            def raw():
                h_c.copy_(d_p, non_blocking=True)
                torch.cuda.current_stream().synchronize()
            t_raw = wall(raw)
        print(json.dumps({"cell": label, "len": n, "chunk": cb, "K": K, "streams": n_streams,
                          "pipelined_d2h_gbs": n / t_pipe / 1e9, "raw_pinned_d2h_gbs": n / t_raw / 1e9,
                          "fraction_of_raw": t_raw / t_pipe}), flush=True)

    def modes_cell(n, cb, label):
        """Split passes and the sequential-chain comparator, device-resident."""
        K = (n + cb - 1) // cb
        with fastrack.Context(key, cb) as ctx:
            st = stream.cuda_stream
            d_p = torch.randint(0, 256, (n,), dtype=torch.uint8, device="cuda")
            d_c, d_o, d_pad = torch.empty_like(d_p), torch.empty_like(d_p), torch.empty_like(d_p)
            d_t = torch.empty(16 * K, dtype=torch.uint8, device="cuda")
            d_m = torch.empty(16 * K, dtype=torch.uint8, device="cuda")
            d_ok = torch.zeros(K, dtype=torch.int32, device="cuda")
            ctx.encrypt_tag(iv, d_p.data_ptr(), n, d_c.data_ptr(), d_t.data_ptr(), st)
            reps = 20
            out = {"cell": label, "len": n, "chunk": cb, "K": K}
            out["ctr_crypt_gbs"] = n / timed(lambda: ctx.ctr_crypt(iv, d_c.data_ptr(), n, d_o.data_ptr(), st), reps) / 1e9
            out["verify_gbs"] = n / timed(lambda: ctx.verify(iv, d_c.data_ptr(), n, d_t.data_ptr(), d_ok.data_ptr(), st), reps) / 1e9
            out["keystream_gbs"] = n / timed(lambda: ctx.keystream(iv, n, d_pad.data_ptr(), d_m.data_ptr(), st), reps) / 1e9
            out["xor_verify_gbs"] = n / timed(lambda: ctx.xor_verify(iv, d_c.data_ptr(), n, d_pad.data_ptr(), d_m.data_ptr(),
                                                                     d_t.data_ptr(), d_o.data_ptr(), d_ok.data_ptr(), st), reps) / 1e9
            assert bool((d_ok == 1).all()) and bool((d_o == d_p).all())
            out["verify_sequential_us"] = timed(lambda: ctx.verify_sequential(iv, d_c.data_ptr(), n, d_t.data_ptr(),
                                                                                d_ok.data_ptr(), st), 1 if K < 64 else 5) * 1e6
            out["verify_us"] = n / out["verify_gbs"] / 1e3
            assert bool((d_ok == 1).all())
        print(json.dumps(out), flush=True)

    def samples_cell(sample_bytes, n_samples, chains, label):
        """The paper's data model: a batch of samples, each split into `chains` chunks under its own IV."""
        cb = (sample_bytes // chains + 15) // 16 * 16
        with fastrack.Context(key, cb) as ctx:
            ctx.set_framing(chains)
            st = stream.cuda_stream
            n = sample_bytes * n_samples
            K = n_samples * ((sample_bytes + cb - 1) // cb)
            d_iv = torch.randint(0, 256, (12 * n_samples,), dtype=torch.uint8, device="cuda")
            d_p = torch.randint(0, 256, (n,), dtype=torch.uint8, device="cuda")
            d_c, d_o = torch.empty_like(d_p), torch.empty_like(d_p)
            d_t = torch.empty(16 * K, dtype=torch.uint8, device="cuda")
            d_ok = torch.zeros(K, dtype=torch.int32, device="cuda")
            ctx.encrypt_tag_samples(d_iv.data_ptr(), sample_bytes, n_samples, d_p.data_ptr(), d_c.data_ptr(), d_t.data_ptr(), st)
            t_batch = timed(lambda: ctx.decrypt_verify_samples(d_iv.data_ptr(), sample_bytes, n_samples, d_c.data_ptr(),
                                                               d_t.data_ptr(), d_o.data_ptr(), d_ok.data_ptr(), st), 100)
            assert bool((d_ok == 1).all()) and bool((d_o == d_p).all())
            ivs_h = d_iv.cpu().numpy().tobytes()
            cps = K // n_samples

            def one_by_one():
                for s in range(n_samples):
                    ctx.decrypt_verify(ivs_h[12 * s:12 * s + 12], d_c.data_ptr() + s * sample_bytes, sample_bytes,
                                       d_t.data_ptr() + 16 * cps * s, d_o.data_ptr() + s * sample_bytes,
                                       d_ok.data_ptr() + 4 * cps * s, st)
            t_each = timed(one_by_one, 20) if n_samples <= 1024 else None        # a call per sample is pointless beyond that
            assert bool((d_ok == 1).all()) and bool((d_o == d_p).all())
        print(json.dumps({"cell": label, "sample_bytes": sample_bytes, "n_samples": n_samples, "chains_per_sample": chains,
                          "chunk": cb, "batch_call_us": t_batch * 1e6, "batch_call_gbs": n / t_batch / 1e9,
                          "one_call_per_sample_us": None if t_each is None else t_each * 1e6}), flush=True)

    for K in (1, 4, 16, 64, 256, 1024):                                   # config 1
        device_cell(64 << 20, (64 << 20) // K, "config1")
    for cb in (256 << 10, 1 << 20, 4 << 20, 8 << 20):                     # config 2
        for ns in (2, 3, 4):
            pipeline_cell(77_070_336, cb, ns, "config2")
    device_cell(670_000_000, 4 << 20, "config3")
    for ns in (2, 4):
        d2h_cell(670_000_000, 4 << 20, ns, "config3_d2h")
    samples_cell(3 * 224 * 224 * 2, 64, 16, "sample_batch")        # a ResNet-style batch: 64 fp16 images, 16 tags each
    samples_cell(3 * 224 * 224 * 2, 256, 16, "sample_batch")
    samples_cell(400, 1 << 18, 1, "small_sample_batch")             # 262 144 feature rows of 100 floats, one tag each
    samples_cell(64, 1 << 20, 1, "small_sample_batch")              # a million 64-byte records
    samples_cell(4096, 1 << 14, 16, "small_sample_batch")           # 4 KiB samples cut into 16 chunks of 256 bytes
    for cb in (16, 64, 256, 1024, 4096, 16384):                    # many small chunks (packed-row kernels below about 8 KiB)
        device_cell(256 << 20, cb, "small_chunks")
    modes_cell(256 << 20, 4 << 20, "split_passes")
    for K in (16, 64, 256, 1024, 4096):
        modes_cell(64 << 20, (64 << 20) // K, "split_passes_vs_K")
    for e in range(6, 17):                                                # config 4 (device-resident throughput)
        for cb in (16 << 10, 64 << 10, 256 << 10, 1 << 20, 4 << 20, 16 << 20):
            device_cell(4 ** e, cb, "config4")


def run_layouts(args):
    """The planner's choice against every forced layout of the packed rows: decrypt+verify GB/s per chunk size for
    the row kernels alone, for the planner, and for every number of lanes per chunk (one JSON line per chunk size)."""
    import torch
    from paper_2410_15240_b200 import fastrack, synth
    torch.cuda.set_device(0)
    key, iv = synth.key_and_iv(1)
    stream = torch.cuda.current_stream()
    st = stream.cuda_stream
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for n in (16 << 20, 256 << 20):
        p = torch.randint(0, 256, (n,), dtype=torch.uint8, device="cuda")
        c, o = torch.empty_like(p), torch.empty_like(p)
        for cb in (16, 64, 256, 1024, 4096, 16384):
            K = n // cb
            t = torch.empty(16 * K, dtype=torch.uint8, device="cuda")
            ok = torch.zeros(K, dtype=torch.int32, device="cuda")

            def measure(options):
                with fastrack.Context(key, cb, options) as ctx:
                    ctx.encrypt_tag(iv, p.data_ptr(), n, c.data_ptr(), t.data_ptr(), st)

                    def call():
                        ctx.decrypt_verify(iv, c.data_ptr(), n, t.data_ptr(), o.data_ptr(), ok.data_ptr(), st)
                    for _ in range(3):
                        call()
                    torch.cuda.synchronize()
                    reps, best = max(5, min(100, int(2e9 // n))), float("inf")
                    for _ in range(3):
                        e0.record(stream)
                        for _ in range(reps):
                            call()
                        e1.record(stream)
                        torch.cuda.synchronize()
                        best = min(best, e0.elapsed_time(e1) / reps)
                    assert bool((ok == 1).all()) and bool((o == p).all())
                return n / best / 1e6
            counters = cb // 16 + 1
            forced = {}
            for lanes in (1, 2, 3, 4, 5, 6, 7, 8, 9, 10, 12, 13, 16, 20, 24, 32, 41, 64, counters):
                run = -(-counters // lanes)
                if lanes <= counters and -(-counters // run) not in forced:
                    forced[-(-counters // run)] = measure({fastrack.OPT_PACK_RUN: run})
            rows_only, auto = measure({fastrack.OPT_PACK_MAX_BLOCKS: 0}), measure({})
            best = max(max(forced.values()), rows_only)
            print(json.dumps({"len": n, "chunk": cb, "rows_only_gbs": rows_only, "planner_gbs": auto, "best_forced_gbs": best,
                              "planner_over_best": auto / best, "forced_gbs_by_lanes": forced}), flush=True)


def run_trace(args):
    """Stage-level timelines of fastrack_pipelined_h2d (best of 20 traced calls), one JSON line per transfer."""
    import torch
    from paper_2410_15240_b200 import fastrack, synth
    torch.cuda.set_device(0)
    key, iv = synth.key_and_iv(2)
    for n, cb, ns in ((77_070_336, 4 << 20, 2), (LEN, CHUNK, args.streams)):
        with fastrack.Context(key, cb) as ctx:
            K = ctx.num_chunks(n)
            d_p = torch.randint(0, 256, (n,), dtype=torch.uint8, device="cuda")
            d_c = torch.empty_like(d_p)
            d_t = torch.empty(16 * K, dtype=torch.uint8, device="cuda")
            ctx.encrypt_tag(iv, d_p.data_ptr(), n, d_c.data_ptr(), d_t.data_ptr(), 0)
            torch.cuda.synchronize()
            h_c, h_t = d_c.cpu().pin_memory(), d_t.cpu().pin_memory()
            d_o = torch.empty_like(d_p)
            d_ok = torch.zeros(K, dtype=torch.int32, device="cuda")
            ctx.set_trace(True)
            best = None
            for _ in range(20):
                ctx.pipelined_h2d(iv, h_c.data_ptr(), n, h_t.data_ptr(), d_o.data_ptr(), d_ok.data_ptr(), ns)
                tr = ctx.get_trace()
                if best is None or tr[-1]["kernel_end_ms"] < best[-1]["kernel_end_ms"]:
                    best = tr
            assert bool((d_ok == 1).all()) and bool((d_o == d_p).all())
        print(json.dumps({"len": n, "chunk": cb, "streams": ns, "stages": best}), flush=True)


def run_peaks(args):
    """Unit rates behind the kernel roofline, measured on this GPU (integer pipes, shared-memory lookups, PCIe)."""
    import ctypes
    lib = ctypes.CDLL(build_bench_helper("peaks_probe.cu", "libpeaks_probe.so", shared=True))
    lib.fastrack_probe_peaks.argtypes = [ctypes.c_char_p, ctypes.c_size_t]
    lib.fastrack_probe_peaks.restype = ctypes.c_int
    buf = ctypes.create_string_buffer(1 << 16)
    rc = lib.fastrack_probe_peaks(buf, len(buf))
    sys.stdout.write(buf.value.decode())
    if rc != 0:
        raise RuntimeError(f"probe failed with CUDA error {rc}")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--streams", type=int, default=4)
    ap.add_argument("--batches", type=int, default=5,
                    help="every timed region is repeated this many times; the median is reported, min and max beside it")
    ap.add_argument("--headline-only", action="store_true", help="skip the other configurations (the `extra` cells)")
    ap.add_argument("--impl", default="fastrack", choices=["fastrack", "reference"])
    ap.add_argument("--kernel-only", action="store_true",
                    help="time only the device-resident decrypt+verify loop (short run for profilers)")
    ap.add_argument("--sweep", action="store_true",
                    help="print throughput over the benchmark configurations instead of the one bench line")
    ap.add_argument("--trace", action="store_true", help="print stage-level timelines of the pipelined H2D call")
    ap.add_argument("--layouts", action="store_true",
                    help="small chunks: the planner's choice against the row kernels and every forced packed layout")
    ap.add_argument("--peaks", action="store_true", help="measure the unit rates the kernel roofline is derived from")
    ap.add_argument("--pass", dest="kernel_pass", default="decrypt_verify",
                    choices=["decrypt_verify", "encrypt_tag", "ctr_crypt", "verify"],
                    help="with --kernel-only: which device-resident pass to time (profiling aid)")
    ap.add_argument("--shape", default=None, metavar="LEN_BYTES,CHUNK_BYTES",
                    help="with --kernel-only: time another buffer / chunk size than the headline one (profiling aid)")
    args = ap.parse_args()
    if args.shape:
        if not args.kernel_only:
            ap.error("--shape only applies to --kernel-only; the metric line is always the headline workload")
        global LEN, CHUNK, WORKLOAD
        LEN, CHUNK = (int(x) for x in args.shape.split(","))
        if LEN % CHUNK:
            ap.error("--shape: LEN_BYTES must be a multiple of CHUNK_BYTES")
        WORKLOAD = f"AES-256-GCM multi-chain decrypt+verify, {LEN} uniform random bytes, chunk {CHUNK} (K={LEN // CHUNK})"
    if args.peaks:
        run_peaks(args)
    elif args.trace:
        run_trace(args)
    elif args.layouts:
        run_layouts(args)
    elif args.sweep:
        run_sweep(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
