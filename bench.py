#!/usr/bin/env python
"""Throughput of the sumcheck matmul prover on synthetic transformer-shaped layers.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--config decoder|qkv|ffn|moe|attn|ldd|commit|glue] [--batched] [--fs] [--verify]
                    [--layers L] [--tokens T] [--no-e2e] [--no-cpu-baseline]

One step = one proving pass over the whole batch: eq tables, A~ / B~ partial evaluations, the
claim C~, every sumcheck round, transcripts written.  The default workload is the audited decoder
block: 32 layers x (QKV 4096x6144, O 4096x4096, FFN up 4096x14336, FFN down 14336x4096) at 8192
tokens, 128 proofs, 39.25 GiB of int8/int32 inputs resident in HBM (far larger than L2, so no
flush is needed between steps).  Rank 0 prints ONE JSON line.

--batched proves all products of the workload as one random-linear-combination proof;
--fs makes a step commit to every matrix (SHA-256 trees) and prove non-interactively (with --batched: one
non-interactive proof for the whole workload); --verify times
the verifier's pass over the same matrices; --config ldd
and --config commit time the logit distances and the response commitments, --config glue the
requantisation link between the FFN products (their own metrics).

--impl reference times the plain CPU oracle on the host cores, on a bounded sample of the same
workload.  With N > 1 (launched by torch.distributed.run) every rank proves an independent
replica of the workload on its own GPU: the path has no exchange step, so no collective is used
beyond the timing barrier.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import threading
import time
from concurrent.futures import ThreadPoolExecutor

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

METRIC = "proved field-MACs/sec"
UNIT = "field-MAC/s"
SEED = 1
BATCH_ID0 = 1 << 40            # ids of the batched proofs (--batched), clear of the proof ids


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100,
                    help="timed steps (default 100: a step takes milliseconds, and the clock sampler needs a region "
                         "of a good fraction of a second)")
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="decoder", choices=sorted(WORKLOADS),
                    help="decoder (default, the metric's workload) or one of the smaller parity configurations")
    ap.add_argument("--layers", type=int, default=32)
    ap.add_argument("--tokens", type=int, default=None, help="token count (default: the configuration's own)")
    ap.add_argument("--vocab", type=int, default=128256, help="ldd: entries per logit row")
    ap.add_argument("--topk", type=int, default=20, help="ldd: size of the committed index sets")
    ap.add_argument("--batched", action="store_true",
                    help="prove all products of the workload as one random-linear-combination proof "
                         "(device-resident timing only)")
    ap.add_argument("--fs", action="store_true",
                    help="non-interactive proofs: a step commits to every matrix (SHA-256 trees) and proves with "
                         "challenges hashed from the commitments and the transcript (device-resident timing only)")
    ap.add_argument("--cached-weights", action="store_true",
                    help="with --fs: the weight matrices (B of every product) are committed once, outside the "
                         "timed steps, as part of the model commitment; a step re-hashes only A and C")
    ap.add_argument("--gated", action="store_true",
                    help="with --config glue: the gated link instead (activation table of the gate projection times the "
                         "up projection, 9 bytes per entry)")
    ap.add_argument("--verify", action="store_true",
                    help="time the verifier's pass instead: its own (c0, a_fin, b_fin) of every proof "
                         "(device-resident timing only)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--e2e-steps", type=int, default=2)
    return ap.parse_args()


def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


# name -> (default tokens, description); the decoder block is the workload the metric is quoted on
WORKLOADS = {
    "decoder": (8192, "audited decoder block: {layers} layers x (QKV 4096x6144, O 4096x4096, FFN 4096x14336 x2), {tokens} tokens"),
    "qkv": (512, "dense-layer projection: A {tokens}x4096 times W 4096x4096, one proof"),
    "ffn": (2048, "dense FFN up/down pair: {tokens}x4096 times 4096x14336, requantised hidden times 14336x4096, two proofs"),
    "moe": (4096, "MoE expert batch: 8 experts 4096x14336, top-2 routing of {tokens} tokens, one proof per expert"),
    "attn": (2048, "attention products: {layers} layers x 32 heads x (Q K^T with k = 128, P V with k = {tokens}), {tokens} tokens, one proof per product"),
    "commit": (8192, "response commitments: {tokens} decision steps x vocabulary {vocab} (float32 logits) cut into "
                     "{tokens}/128 requests of uneven length, one SHA-256 tree commitment per request"),
    "ldd": (8192, "logit distance distribution: {tokens} decision steps x vocabulary {vocab} (float32), TV + KL + Top-{topk} distance + tail statistic"),
    "glue": (8192, "requantisation link of the FFN pair: hidden activations {tokens} x 14336, int32 accumulators of the up "
                   "projection against the int8 input of the down projection"),
}
L2_BYTES = 126 << 20


def workload_name(config, layers, tokens, vocab=128256, topk=20):
    if config == "attn":
        layers = min(layers, 8)
    return WORKLOADS[config][1].format(layers=layers, tokens=tokens, vocab=vocab, topk=topk)


def make_problems(config, seed, layers, tokens, device):
    from paper_2602_22700_b200 import synth
    if config == "decoder":
        return synth.decoder_block(seed, layers, tokens, device=device)
    if config == "qkv":
        return synth.qkv_projection(seed, tokens, device=device)
    if config == "ffn":
        return synth.ffn_pair(seed, tokens, device=device)
    if config == "attn":
        return synth.attention_block(seed, min(layers, 8), tokens, device=device)
    return synth.moe_experts(seed, tokens, device=device)


# ------------------------------------------------------------------------ clocks sampling


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU while the timed region runs: through NVML
    every 5 ms where the bindings load (read-only queries), else with nvidia-smi every 100 ms."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    # NVML's clocks-event-reason bits
    REASON_BITS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []
        self.nvml = None
        self.samples = []            # (time, sm MHz, max MHz, watts, reason bits)
        self.stop_flag = False

    def _nvml_loop(self):
        n, h = self.nvml
        while not self.stop_flag:
            try:
                sm = n.nvmlDeviceGetClockInfo(h, n.NVML_CLOCK_SM)
                try:
                    bits = n.nvmlDeviceGetCurrentClocksEventReasons(h)
                except AttributeError:
                    bits = n.nvmlDeviceGetCurrentClocksThrottleReasons(h)
                watts = n.nvmlDeviceGetPowerUsage(h) / 1000.0
                self.samples.append((time.time(), float(sm), self.nvml_max, watts, int(bits)))
            except Exception:
                pass
            time.sleep(0.005)

    def start(self):
        try:
            import pynvml as n
            n.nvmlInit()
            uuid = torch.cuda.get_device_properties(torch.cuda.current_device()).uuid
            h = None
            for i in range(n.nvmlDeviceGetCount()):
                hi = n.nvmlDeviceGetHandleByIndex(i)
                u = n.nvmlDeviceGetUUID(hi)
                u = u.decode() if isinstance(u, bytes) else u
                if str(uuid) in u:
                    h = hi
            if h is None:
                h = n.nvmlDeviceGetHandleByIndex(self.index)
            self.nvml_max = float(n.nvmlDeviceGetMaxClockInfo(h, n.NVML_CLOCK_SM))
            self.nvml = (n, h)
            self.thread = threading.Thread(target=self._nvml_loop, daemon=True)
            self.thread.start()
            return
        except Exception:
            self.nvml = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float):
        if self.nvml is not None:
            self.stop_flag = True
            self.thread.join(timeout=1)
            rows = [r for r in self.samples if t0 <= r[0] <= t1] or self.samples[-3:]
            if not rows:
                return None
            sm = sorted(r[1] for r in rows)
            reasons = set()
            for r in rows:
                for bit, name in self.REASON_BITS.items():
                    if r[4] & bit:
                        reasons.add(name)
            return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": rows[0][2], "power_w_max": max(r[3] for r in rows),
                    "samples": len(rows), "reasons": sorted(reasons), "source": "nvml, 5 ms period"}
        if self.proc is None:
            return None
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        rows = [l for (t, l) in self.lines if t0 <= t <= t1 + 0.1] or [l for (_, l) in self.lines[-3:]]
        sm, smax, reasons, power = [], [], set(), []
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for l in rows:
            f = [x.strip() for x in l.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0])); smax.append(float(f[1])); power.append(float(f[2]))
            except ValueError:
                continue
            for name, v in zip(names, f[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return None
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": max(smax), "power_w_max": max(power),
                "samples": len(sm), "reasons": sorted(reasons), "source": "nvidia-smi, 100 ms period"}


# ------------------------------------------------------------------------ oracle timing


def oracle_time_sample(sample, threads):
    """Wall seconds the CPU oracle takes to prove `sample` (numpy A, B, C, proof_id tuples) with one
    proof per thread; returns (seconds, transcripts)."""
    import oracle

    def one(p):
        A, B, C, pid = p
        return oracle.sumcheck_matmul_prove(A, B, C, SEED, pid)

    t0 = time.perf_counter()
    with ThreadPoolExecutor(max_workers=threads) as ex:
        out = list(ex.map(one, sample))
    return time.perf_counter() - t0, out


def oracle_build_line():
    from oracle import imm_oracle
    return "gcc " + " ".join(imm_oracle.BUILD_FLAGS) + " (plain C, single-threaded per proof, % on unsigned __int128)"


def field_macs(shapes):
    return sum(m * k + k * n + m * n + 5 * (1 << max(0, (k - 1).bit_length())) for (m, k, n) in shapes)


def sample_to_host(problems):
    return [(p.A.cpu().numpy(), p.B.cpu().numpy(), p.C.cpu().numpy(), p.proof_id) for p in problems]


def mem_available_bytes():
    try:
        with open("/proc/meminfo") as f:
            for line in f:
                if line.startswith("MemAvailable:"):
                    return int(line.split()[1]) * 1024
    except OSError:
        pass
    return 0


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except (OSError, KeyError, ValueError):
        return 6650.0, "fallback"


# DRAM traffic of the claim kernel per algorithmic byte, from the ncu capture summarised under
# profiles/ (dram__bytes_read.sum + dram__bytes_write.sum over 4*m*n); None until a capture of the
# current kernel exists.
LDD_TVKL_TRAFFIC_RATIO = (1.078953 + 0.004193) / 1.050673   # tv_kl_kernel<aligned, 512 threads>: (dram read + write) / (8 bytes per entry pair)
COMMIT_TRAFFIC_RATIO = (1.077891 + 0.018910) / 1.050673152                   # commit_leaf_kernel: (dram read + write) / message bytes
# SHA-256 leaf hashing against the integer ALU pipe (rotates, three-input logic, byte permutes): the
# pipe retires 64 thread instructions per cycle per SM; the kernel issues 17.18 of them per hashed
# byte (ncu: 564.2 M warp instructions on that pipe for 1.0507 GB), so at 1965 MHz the pipe allows
# 148 x 64 x 1.965e9 / 17.18 = 1083 GB/s.
COMMIT_ALU_PEAK_GBS_AT_1965 = 1083.0
GLUE_TRAFFIC_RATIO = (146.819072 + 3.869952) / 146.80064    # requant_check_kernel: (dram read + write) / (5 bytes per entry), 2048-token capture
GATED_TRAFFIC_RATIO = (264.269312 + 3.397632) / 264.241152   # gated_link_kernel: (dram read + write) / (9 bytes per entry), 2048-token capture
FUSED_TRAFFIC_RATIO = (308.909568 + 12.264448) / 306.184192   # fused_contract_kernel: (dram read + write) / algorithmic bytes, FFN-pair capture
CLAIM_KERNEL_TRAFFIC_RATIO = 239.64 / 234.881024  # bytedot_kernel<1,1,1>: (dram read + write) / (4 bytes per entry), small-case capture


# ------------------------------------------------------------------------ our arm


def run_ours(args):
    from paper_2602_22700_b200 import imm, synth
    from paper_2602_22700_b200.replicas import Replicas
    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the prover has no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    rep = Replicas("nccl", dev)
    imm.lib()
    warmup = max(args.warmup, 3)
    steps = max(args.steps, 1)

    problems = make_problems(args.config, rep.seed(SEED), args.layers, args.tokens, dev)
    shapes = [p.mkn for p in problems]
    macs = synth.prover_field_macs(problems)
    algo_bytes = synth.problem_bytes(problems)
    claim_bytes = sum(4 * m * n for (m, k, n) in shapes)
    groups = {}
    if args.batched and not args.fs:
        groups[max(imm.ceil_log2(p.mkn[1]) for p in problems)] = list(problems)
        provers = [imm.BatchedProver([(p.A, p.B, p.C, p.proof_id) for p in g], device=dev) for g in groups.values()]

        def prove_step():
            for gi, bp in enumerate(provers):
                bp.prove(SEED, BATCH_ID0 + gi)
    elif args.verify:
        ver = imm.Verifier([(p.A, p.B, p.C, p.proof_id) for p in problems], device=dev)
        provers = [ver]

        def prove_step():
            ver.expected(SEED)
    elif args.fs:
        triples = [(p.A, p.B, p.C, p.proof_id) for p in problems]
        nt = len(triples)
        weight_commit_ms = None
        if args.cached_weights:
            # the model commitment: every weight matrix hashed once, before any audited request
            com_w = imm.Committer([B for (A, B, C, _) in triples], device=dev)
            com_w.commit()
            w0, w1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            w0.record()
            com_w.commit()
            w1.record()
            torch.cuda.synchronize()
            weight_commit_ms = w0.elapsed_time(w1)
            com = imm.Committer([t for (A, B, C, _) in triples for t in (A, C)], device=dev)
            stmt = torch.empty((nt, 96), dtype=torch.uint8, device=dev)
            stmt.view(nt, 3, 32)[:, 1].copy_(com_w.digests.view(nt, 32))
            committed_bytes = sum(m * k + 4 * m * n for (m, k, n) in shapes)
        else:
            com = imm.Committer([t for (A, B, C, _) in triples for t in (A, B, C)], device=dev)
            stmt = com.digests.view(nt, 96)
            committed_bytes = algo_bytes
        if args.batched:
            fsp = imm.FsBatchedProver(triples, stmt, device=dev)
            fsp_prove = lambda: fsp.prove(BATCH_ID0)
        else:
            fsp = imm.FsProver(triples, stmt, device=dev)
            fsp_prove = fsp.prove
        if fsp.commitments.data_ptr() != stmt.data_ptr():
            raise SystemExit("the prover copied the statement: cached commitments would go stale")
        provers = [fsp]
        fs_ev = []

        def prove_step():
            e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
            e[0].record()
            com.commit()
            if args.cached_weights:                      # fresh com_A, com_C beside the cached com_B
                fresh = com.digests.view(nt, 2, 32)
                stmt.view(nt, 3, 32)[:, 0].copy_(fresh[:, 0])
                stmt.view(nt, 3, 32)[:, 2].copy_(fresh[:, 1])
            e[1].record()
            fsp_prove()
            e[2].record()
            fs_ev.append(e)
    else:
        prover = imm.Prover([(p.A, p.B, p.C, p.proof_id) for p in problems], device=dev)
        provers = [prover]

        def prove_step():
            prover.prove(SEED)
    calls_per_step = len(provers)
    barrier = rep.barrier

    for _ in range(warmup):
        prove_step()
    barrier()
    sampler = ClockSampler(local_rank if "CUDA_VISIBLE_DEVICES" not in os.environ else
                           int(os.environ["CUDA_VISIBLE_DEVICES"].split(",")[local_rank]))
    sampler.start()
    time.sleep(0.25)
    # inputs of at least twice the L2 size evict themselves between steps; smaller ones get an
    # explicit flush (a 512 MB buffer overwritten outside the per-step event pairs)
    flush = algo_bytes < 2 * L2_BYTES
    t0 = time.time()
    if flush:
        scrub = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
        pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for a, b in pairs:
            scrub.fill_(1)
            a.record()
            prove_step()
            b.record()
        barrier()
        elapsed_ms = sum(a.elapsed_time(b) for a, b in pairs)
    else:
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record()
        for _ in range(steps):
            prove_step()
        ev1.record()
        barrier()
        elapsed_ms = ev0.elapsed_time(ev1)
    t1 = time.time()
    clocks = sampler.stop(t0, t1)
    elapsed_ms = rep.max_over_ranks(elapsed_ms)
    # per-launch times from a second, shorter loop with the library's phase events on (kept out of the
    # timed region: the events between the launches of a small batch undo their programmatic overlap)
    psteps = min(steps, 20)
    imm.profile_enable(min(4096, (psteps + 4) * calls_per_step))
    first_call = imm.profile_calls()
    for _ in range(psteps):
        if flush:
            scrub.fill_(1)
        prove_step()
    torch.cuda.synchronize()
    phase_ms = [0.0] * len(imm.PROFILE_PHASES)
    for c in range(first_call, first_call + psteps * calls_per_step):
        for i, v in enumerate(imm.profile_read(c)):
            phase_ms[i] += v / psteps
    imm.profile_enable(0)

    # every proof of the timed batch must be accepted by the verifier
    accepted = 0
    if args.verify:
        # the timed pass's values must accept an honest prover's transcripts
        host_t = None
        vals = ver.values.cpu().numpy().view(np.uint64)
        assert int(ver.status.abs().max()) == 0
        pr2 = imm.Prover([(p.A, p.B, p.C, p.proof_id) for p in problems], device=dev)
        tr2 = pr2.prove(SEED).cpu().numpy().view(np.uint64)
        for i, p in enumerate(problems):
            b = imm.ceil_log2(p.A.shape[1])
            words = [int(v) for v in tr2[i, :3 * b + 3]]
            if imm.sumcheck_verify(words, b, SEED, p.proof_id, *[int(v) for v in vals[i]]) == (imm.OK, -1):
                accepted += 1
        del pr2
    elif args.fs and args.batched:
        host_t = None
        assert int(fsp.status.abs().max()) == 0
        words = [int(v) & 0xFFFFFFFFFFFFFFFF for v in fsp.transcript.cpu()]
        meta = [tuple(p.mkn) + (p.proof_id,) for p in problems]
        host_c = stmt.cpu().numpy().tobytes()
        if imm.sumcheck_verify_fs_batched(words, fsp.nrounds, meta, host_c, BATCH_ID0) == (imm.OK, -1):
            accepted = len(problems)
    elif args.fs:
        host_t = fsp.transcripts.cpu()
        assert int(fsp.status.abs().max()) == 0
        host_c = stmt.cpu().numpy()
        for i, p in enumerate(problems):
            m_, k_, n_ = p.mkn
            b = imm.ceil_log2(k_)
            words = [int(v) & 0xFFFFFFFFFFFFFFFF for v in host_t[i, :3 * b + 3]]
            if imm.sumcheck_verify_fs(words, b, bytes(host_c[i]), m_, k_, n_, p.proof_id) == (imm.OK, -1):
                accepted += 1
    elif args.batched:
        host_t = None
        for gi, (b, g) in enumerate(groups.items()):
            assert int(provers[gi].status.abs().max()) == 0
            words = [int(v) & 0xFFFFFFFFFFFFFFFF for v in provers[gi].transcript.cpu()]
            if imm.sumcheck_verify_batched(words, b, len(g), SEED, BATCH_ID0 + gi) == (imm.OK, -1):
                accepted += len(g)
    else:
        host_t = prover.transcripts.cpu()
        assert int(prover.status.abs().max()) == 0
        for i, p in enumerate(problems):
            b = imm.ceil_log2(p.A.shape[1])
            words = [int(v) & 0xFFFFFFFFFFFFFFFF for v in host_t[i, :3 * b + 3]]
            if imm.sumcheck_verify(words, b, SEED, p.proof_id) == (imm.OK, -1):
                accepted += 1
    if accepted != len(problems):
        raise SystemExit(f"only {accepted}/{len(problems)} proofs verified")

    ms_per_step = elapsed_ms / steps
    value = macs * world / (ms_per_step * 1e-3)
    peak, peak_kind = measured_peaks()
    fused = (not (args.batched or args.verify or args.fs)) and prover.launches == 3
    if fused:            # one contraction launch for A, B and C: its bytes are the whole batch's
        claim_bytes = algo_bytes
    claim_gbs = claim_bytes / (phase_ms[1] * 1e-3) / 1e9
    phase_bytes = ([0, algo_bytes, 0, 0, 0] if fused else
                   [0, claim_bytes, sum(m * k for (m, k, n) in shapes), sum(k * n for (m, k, n) in shapes), 0])
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "u64", "data": "synthetic",
        "config": {"workload": workload_name(args.config, args.layers, args.tokens) +
                               (", as one batched proof (every k padded to the largest 2^b)" if args.batched else "") +
                               (", the verifier's pass (its own c0, a_fin, b_fin per proof)" if args.verify else "") +
                               (", non-interactive: SHA-256 tree commitments to every matrix, then proofs with hashed "
                                "challenges" if args.fs else "") +
                               (" (weight commitments cached: a step hashes A and C only)" if args.fs and args.cached_weights else ""),
                   "layers": args.layers if args.config == "decoder" else min(args.layers, 8) if args.config == "attn" else None,
                   "tokens": args.tokens, "proofs_per_gpu": len(problems), "field": "Goldilocks 2^64-2^32+1",
                   "input_bytes_per_gpu": algo_bytes,
                   "l2": ("L2 flushed between steps (512 MB overwritten outside the timed event pairs)" if flush else
                          f"inputs ({algo_bytes / 2**30:.2f} GiB) exceed the 126 MB L2 several times over; no flush"),
                   "parallelism": "1 GPU" if world == 1 else f"{world} independent replicas, no collective"},
        "layers_per_s": (args.layers * world / (ms_per_step * 1e-3)) if args.config == "decoder" else None,
        "proofs_per_s": len(problems) * world / (ms_per_step * 1e-3),
        "proved_matmul_macs_per_s": synth.proved_matmul_macs(problems) * world / (ms_per_step * 1e-3),
        "hbm_gbs_whole_step": algo_bytes / (ms_per_step * 1e-3) / 1e9,
        "hbm_frac_of_8tbs_whole_step": algo_bytes / (ms_per_step * 1e-3) / 8e12,
        "proofs_verified": accepted,
        "phases": {name: {"ms": phase_ms[i],
                          "gbs": (phase_bytes[i] / (phase_ms[i] * 1e-3) / 1e9) if phase_bytes[i] and phase_ms[i] > 0 else None}
                   for i, name in enumerate(imm.PROFILE_PHASES)},
        "roofline": {"kernel": ("fused_contract_kernel (tiles of A, B and C in one grid; phase claim_C)" if fused else
                                "bytedot_kernel<int32 as bytes, POINT> (claim C~)"), "bound": "hbm", "achieved": claim_gbs,
                     "peak": peak, "peak_kind": peak_kind, "unit": "GB/s", "frac": claim_gbs / peak,
                     "frac_of_8tbs": claim_gbs / 8000.0,
                     # achieved GB/s per sampled SM MHz: comparable across pods whose clocks differ
                     "gbs_per_sm_mhz": (claim_gbs / clocks["sm_mhz"]) if clocks and clocks.get("sm_mhz") else None,
                     "traffic": (FUSED_TRAFFIC_RATIO if fused else CLAIM_KERNEL_TRAFFIC_RATIO) * claim_bytes},
        "phase_steps": psteps,
        "gpu_launches": ((fsp.launches + com.launches) if args.fs else sum(pv.launches for pv in provers)) * steps,
        "transcript_words_per_step": (int(fsp.length) if (args.fs and args.batched) else
                                      sum(int(bp.length) for bp in provers) if args.batched else
                                      sum(3 * imm.ceil_log2(k) + 3 for (m, k, n) in shapes)),
        "clocks": clocks,
    }

    # ---- end to end: pinned host inputs -> device arena -> proofs -> host transcripts
    e2e = None
    if args.fs:
        tail = fs_ev[-steps:]
        out["fs_phases"] = {"commit_ms": sum(e[0].elapsed_time(e[1]) for e in tail) / steps,
                            "prove_ms": sum(e[1].elapsed_time(e[2]) for e in tail) / steps,
                            "committed_bytes": committed_bytes}
        if args.cached_weights:
            out["fs_phases"].update({"weights_cached": True, "weight_commit_ms_once": weight_commit_ms,
                                     "weight_bytes": sum(k * n for (m, k, n) in shapes)})
    if args.batched or args.fs or args.verify:
        e2e = {"value": None, "unit": UNIT, "skipped": "the host-buffer entry point proves interactively, proof by proof"}
    elif not args.no_e2e:
        need = algo_bytes
        if mem_available_bytes() < int(1.25 * need * (world if world > 1 else 1)):
            e2e = {"value": None, "unit": UNIT, "skipped": "not enough host memory for pinned inputs"}
        else:
            host = []
            for p in problems:
                host.append(tuple(torch.empty(t.shape, dtype=t.dtype, pin_memory=True).copy_(t)
                                  for t in (p.A, p.B, p.C)) + (p.proof_id,))
            torch.cuda.synchronize()
            hp = imm.HostProver(host, device=dev)
            hp.prove(SEED)                                   # warm-up (page-locks, first touch of the arena)
            barrier()
            k2 = max(1, args.e2e_steps)
            w0 = time.perf_counter()
            for _ in range(k2):
                hp.prove(SEED)                               # synchronous: returns after the D2H copy
            e2e_s = (time.perf_counter() - w0) / k2
            e2e_s = rep.max_over_ranks(e2e_s)
            same = bool((hp.transcripts == host_t).all())
            e2e = {"value": macs * world / e2e_s, "unit": UNIT, "ms_per_step": e2e_s * 1e3, "steps": k2,
                   "h2d_bytes_per_step": hp.h2d_bytes, "d2h_bytes_per_step": hp.d2h_bytes,
                   "matches_device_path": same}
            del hp, host
    out["e2e"] = e2e

    # ---- the oracle beside it (rank 0, single GPU): first two layers' proofs, one per thread
    if not args.no_cpu_baseline and world == 1 and not (args.batched or args.fs or args.verify):
        nsample = min(len(problems), 8)
        sample = sample_to_host(problems[:nsample])
        threads = min(os.cpu_count() or 1, nsample)
        secs, want = oracle_time_sample(sample, threads)
        ok = all([int(v) & 0xFFFFFFFFFFFFFFFF for v in host_t[i, :len(w)]] == [int(x) for x in w]
                 for i, w in enumerate(want))
        out["cpu_baseline"] = {"value": field_macs(shapes[:nsample]) / secs, "unit": UNIT, "cores": threads,
                               "nproc": os.cpu_count(), "compiler": oracle_build_line(),
                               "kind": "oracle", "seconds": secs,
                               "sample": f"the first {nsample} of the {len(problems)} proofs, "
                                         f"one proof per thread, same inputs as the GPU run",
                               "gpu_transcripts_match": ok}
        if not ok:
            raise SystemExit("GPU transcripts differ from the oracle on the sampled proofs")
    if rank == 0:
        print(json.dumps(out))
    rep.close()


# ------------------------------------------------------------------------ logit distance distribution


def ldd_oracle_rows(dep, ref, topk, rows):
    """The float64 oracle on the given rows: (tv, kl, top-K distance) lists."""
    from oracle import ldd
    tv, kl, dist = [], [], []
    for i in rows:
        tv.append(ldd.tv_distance(dep[i], ref[i]))
        kl.append(ldd.kl_divergence(dep[i], ref[i]))
        dist.append(ldd.topk_distance(ref[i], topk[i]))
    return tv, kl, dist


def run_ldd(args):
    """One step = every decision step's TV and KL distance, its Top-K distance, and the per-request
    tail statistic.  Not the headline workload: a second data-parallel path of the same audit."""
    from paper_2602_22700_b200 import imm, synth
    from paper_2602_22700_b200.replicas import Replicas
    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    rep = Replicas("nccl", dev)
    imm.lib()
    warmup, steps = max(args.warmup, 3), max(args.steps, 1)
    T, n, K = args.tokens, args.vocab, args.topk
    ref = synth.reference_logits(rep.seed(SEED), T, n, device=dev)
    dep = synth.deployed_logits(ref, rep.seed(SEED), synth.NOISE_QUANTISED)
    topk = torch.topk(dep, K, dim=1).indices.to(torch.int32).contiguous()      # what the server committed to
    offsets = synth.request_offsets(rep.seed(SEED), T, max(1, T // 256), device=dev)
    t1, t2 = 0.1, 0.02
    bytes_tvkl, bytes_topk = 8 * T * n, 4 * T * n

    barrier = rep.barrier

    def one_pass(ev=None):
        if ev:
            ev[0].record()
        tv, kl = imm.ldd_tv_kl(dep, ref)
        if ev:
            ev[1].record()
        d, st = imm.ldd_topk_distance(ref, topk)
        if ev:
            ev[2].record()
        p, flag = imm.ldd_tail_fraction(tv, offsets, t1, t2)
        if ev:
            ev[3].record()
        return tv, kl, d, st, p, flag

    for _ in range(warmup):
        one_pass()
    barrier()
    sampler = ClockSampler(local_rank if "CUDA_VISIBLE_DEVICES" not in os.environ else
                           int(os.environ["CUDA_VISIBLE_DEVICES"].split(",")[local_rank]))
    sampler.start()
    time.sleep(0.25)
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(steps)]
    t0 = time.time()
    for e in evs:
        out = one_pass(e)
    barrier()
    t1w = time.time()
    clocks = sampler.stop(t0, t1w)
    elapsed_ms = evs[0][0].elapsed_time(evs[-1][3])
    elapsed_ms = rep.max_over_ranks(elapsed_ms)
    ms_per_step = elapsed_ms / steps
    ph = [sum(e[i].elapsed_time(e[i + 1]) for e in evs) / steps for i in range(3)]
    tv, kl, d, st, p, flag = out
    assert int(st.abs().max()) == 0
    peak, peak_kind = measured_peaks()
    tvkl_gbs = bytes_tvkl / (ph[0] * 1e-3) / 1e9
    res = {
        "metric": "LDD decision steps/sec", "value": T * world / (ms_per_step * 1e-3), "unit": "steps/s",
        "n_gpus": world, "steps": steps, "warmup": warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": workload_name("ldd", 0, T, n, K), "tokens": T, "vocab": n, "topk": K,
                   "requests": int(offsets.numel()) - 1, "input_bytes_per_gpu": bytes_tvkl + 4 * T * K,
                   "l2": f"inputs ({bytes_tvkl / 2**30:.2f} GiB) exceed the 126 MB L2 many times over; no flush",
                   "parallelism": "1 GPU" if world == 1 else f"{world} independent replicas, no collective"},
        "hbm_gbs_whole_step": (bytes_tvkl + bytes_topk) / (ms_per_step * 1e-3) / 1e9,
        "phases": {"tv_kl": {"ms": ph[0], "gbs": tvkl_gbs},
                   "topk_distance": {"ms": ph[1], "gbs": bytes_topk / (ph[1] * 1e-3) / 1e9},
                   "tail_fraction": {"ms": ph[2], "gbs": None}},
        "roofline": {"kernel": "tv_kl_kernel (two logit rows read once from HBM, second pass from L2)", "bound": "hbm",
                     "achieved": tvkl_gbs, "peak": peak, "peak_kind": peak_kind, "unit": "GB/s", "frac": tvkl_gbs / peak,
                     "frac_of_8tbs": tvkl_gbs / 8000.0,
                     "gbs_per_sm_mhz": (tvkl_gbs / clocks["sm_mhz"]) if clocks and clocks.get("sm_mhz") else None,
                     "traffic": (LDD_TVKL_TRAFFIC_RATIO * bytes_tvkl) if LDD_TVKL_TRAFFIC_RATIO else None},
        "gpu_launches": 3 * steps,
        "clocks": clocks,
        "flagged_requests": int(flag.sum()),
    }
    e2e = None
    if not args.no_e2e:
        hd = torch.empty(dep.shape, dtype=dep.dtype, pin_memory=True).copy_(dep)
        hr = torch.empty(ref.shape, dtype=ref.dtype, pin_memory=True).copy_(ref)
        hk = torch.empty(topk.shape, dtype=topk.dtype, pin_memory=True).copy_(topk)
        dd, dr, dk = torch.empty_like(dep), torch.empty_like(ref), torch.empty_like(topk)
        outs = [torch.empty(T, dtype=torch.float64, pin_memory=True) for _ in range(3)]
        torch.cuda.synchronize()

        def e2e_pass():
            dd.copy_(hd, non_blocking=True); dr.copy_(hr, non_blocking=True); dk.copy_(hk, non_blocking=True)
            a, b = imm.ldd_tv_kl(dd, dr)
            c, _ = imm.ldd_topk_distance(dr, dk)
            imm.ldd_tail_fraction(a, offsets, t1, t2)
            outs[0].copy_(a, non_blocking=True); outs[1].copy_(b, non_blocking=True); outs[2].copy_(c, non_blocking=True)
            torch.cuda.synchronize()

        e2e_pass()
        barrier()
        k2 = max(1, args.e2e_steps)
        w0 = time.perf_counter()
        for _ in range(k2):
            e2e_pass()
        e2e_s = (time.perf_counter() - w0) / k2
        e2e_s = rep.max_over_ranks(e2e_s)
        e2e = {"value": T * world / e2e_s, "unit": "steps/s", "ms_per_step": e2e_s * 1e3, "steps": k2,
               "h2d_bytes_per_step": hd.numel() * 4 + hr.numel() * 4 + hk.numel() * 4, "d2h_bytes_per_step": 3 * T * 8,
               "matches_device_path": bool((outs[0].to(dev) == tv).all() and (outs[2].to(dev) == d).all())}
        del hd, hr, hk, dd, dr, dk
    res["e2e"] = e2e
    if not args.no_cpu_baseline and world == 1:
        rows = list(range(0, T, max(1, T // 48)))[:48]
        hdep, href, htop = dep[rows].cpu().numpy(), ref[rows].cpu().numpy(), topk[rows].cpu().numpy()
        w0 = time.perf_counter()
        otv, okl, odist = ldd_oracle_rows(hdep, href, htop, range(len(rows)))
        secs = time.perf_counter() - w0
        gtv, gkl, gd = tv[rows].cpu().numpy(), kl[rows].cpu().numpy(), d[rows].cpu().numpy()
        ok = (max(abs(a - b) for a, b in zip(gtv, otv)) <= 2e-5 and
              all(abs(a - b) <= 2e-5 + 2e-4 * abs(b) for a, b in zip(gkl, okl)) and
              all(abs(a - b) <= 1e-9 * max(1.0, abs(b)) for a, b in zip(gd, odist)))
        res["cpu_baseline"] = {"value": len(rows) / secs, "unit": "steps/s", "cores": 1, "nproc": os.cpu_count(),
                               "kind": "oracle", "seconds": secs,
                               "sample": f"{len(rows)} of the {T} decision steps, evenly spaced, same inputs as the GPU run",
                               "gpu_matches_oracle_within_tolerance": ok}
        if not ok:
            raise SystemExit("GPU distances differ from the oracle beyond the tolerance")
    if rank == 0:
        print(json.dumps(res))
    rep.close()


# ------------------------------------------------------------------------ links between products


def run_glue(args):
    """One step = the element-wise check that the down projection's int8 input is the requantised int32
    output of the up projection (every entry of a tokens x 14336 hidden matrix)."""
    from paper_2602_22700_b200 import imm, synth
    from paper_2602_22700_b200.replicas import Replicas
    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    rep = Replicas("nccl", dev)
    imm.lib()
    warmup, steps = max(args.warmup, 3), max(args.steps, 1)
    T, d_model, d_ff = args.tokens, 4096, 14336
    seed = rep.seed(SEED)
    A = synth.gauss_i8(seed, synth.tid(0, synth.ROLE_ACT), T, d_model, synth.Q_SIGMA20, dev)
    W = synth.gauss_i8(seed, synth.tid(0, synth.ROLE_W), d_model, d_ff, synth.Q_SIGMA8, dev)
    C = synth.exact_matmul_i32(A, W)
    gated = bool(args.gated)
    if gated:
        # gate = C; up = a second product of the same activations; H manufactured with torch integer ops
        W2 = synth.gauss_i8(seed, synth.tid(1, synth.ROLE_W), d_model, d_ff, synth.Q_SIGMA8, dev)
        U = synth.exact_matmul_i32(A, W2)
        del W2
        act_host = [int(round(v / (1.0 + math.exp(-v / 16.0)))) for v in range(-128, 128)]
        act_dev = torch.tensor(act_host, dtype=torch.int32, device=dev)
        H = torch.empty((T, d_ff), dtype=torch.int8, device=dev)
        for r0 in range(0, T, 1024):                           # in slabs: the intermediates are 64-bit
            q = lambda X: torch.clamp((X >> 9) + (((X & 511) + 256) >> 9), -128, 127)
            pr = act_dev[(q(C[r0:r0 + 1024]) + 128).long()] * q(U[r0:r0 + 1024])
            H[r0:r0 + 1024] = torch.clamp((pr >> 7) + (((pr & 127) + 64) >> 7), -127, 127).to(torch.int8)
        del pr, act_dev

        def check(G_, U_, H_, out_):
            return imm.gated_link_check(G_, U_, H_, act_host, 9, 256, 7, 64, -127, 127, out=out_)
    else:
        U = None
        H = synth.requantize_i8(C)

        def check(G_, U_, H_, out_):
            return imm.requant_check(G_, H_, out=out_)
    del A, W
    nbytes = (9 if gated else 5) * T * d_ff
    out = torch.empty(2, dtype=torch.int64, device=dev)
    barrier = rep.barrier
    for _ in range(warmup):
        check(C, U, H, out)
    barrier()
    sampler = ClockSampler(local_rank if "CUDA_VISIBLE_DEVICES" not in os.environ else
                           int(os.environ["CUDA_VISIBLE_DEVICES"].split(",")[local_rank]))
    sampler.start()
    time.sleep(0.25)
    flush = nbytes < 2 * L2_BYTES
    scrub = torch.empty(512 << 20, dtype=torch.uint8, device=dev) if flush else None
    pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    t0 = time.time()
    for a, b in pairs:
        if flush:
            scrub.fill_(1)
        a.record()
        check(C, U, H, out)
        b.record()
    barrier()
    t1w = time.time()
    clocks = sampler.stop(t0, t1w)
    elapsed_ms = rep.max_over_ranks(sum(a.elapsed_time(b) for a, b in pairs))
    ms_per_step = elapsed_ms / steps
    got = [int(v) for v in out.cpu()]
    if got != [0, -1]:
        raise SystemExit(f"the honest link does not hold: {got}")
    peak, peak_kind = measured_peaks()
    gbs = nbytes / (ms_per_step * 1e-3) / 1e9
    res = {
        "metric": "checked entries/sec", "value": T * d_ff * world / (ms_per_step * 1e-3), "unit": "entries/s",
        "n_gpus": world, "steps": steps, "warmup": warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "i32", "data": "synthetic",
        "config": {"workload": workload_name("glue", 0, T) + (" -- gated: activation table of the gate times the up "
                                                                  "projection" if gated else ""),
                   "tokens": T, "input_bytes_per_gpu": nbytes,
                   "map": ("clamp((act[q(G)] * q(U) + 64) >> 7, -127, 127), q(X) = clamp((X + 256) >> 9, -128, 127), act = "
                           "round(x * sigmoid(x / 16))" if gated else "clamp((C + 256) >> 9, -127, 127)"),
                   "l2": ("L2 flushed between steps (512 MB overwritten outside the timed event pairs)" if flush else
                          f"inputs ({nbytes / 2**30:.2f} GiB) exceed the 126 MB L2 several times over; no flush"),
                   "parallelism": "1 GPU" if world == 1 else f"{world} independent replicas, no collective"},
        "hbm_gbs_whole_step": gbs,
        "roofline": {"kernel": ("gated_link_kernel (4 bytes of G + 4 of U + 1 of H per entry, read once); timed as the whole "
                                "imm_gated_link_check call (two 8-byte memsets + the kernel)" if gated else
                                "requant_check_kernel (4 bytes of C + 1 byte of H per entry, read once); timed as the whole "
                                "imm_requant_check call (two 8-byte memsets + the kernel)"), "bound": "hbm", "achieved": gbs,
                     "peak": peak, "peak_kind": peak_kind, "unit": "GB/s", "frac": gbs / peak, "frac_of_8tbs": gbs / 8000.0,
                     "gbs_per_sm_mhz": (gbs / clocks["sm_mhz"]) if clocks and clocks.get("sm_mhz") else None,
                     "traffic": (GATED_TRAFFIC_RATIO if gated else GLUE_TRAFFIC_RATIO) * nbytes},
        "gpu_launches": steps,
        "clocks": clocks,
    }
    e2e = None
    if not args.no_e2e:
        hC = torch.empty(C.shape, dtype=C.dtype, pin_memory=True).copy_(C)
        hH = torch.empty(H.shape, dtype=H.dtype, pin_memory=True).copy_(H)
        dC, dH = torch.empty_like(C), torch.empty_like(H)
        hU = torch.empty(U.shape, dtype=U.dtype, pin_memory=True).copy_(U) if gated else None
        dU = torch.empty_like(U) if gated else None
        hout = torch.empty(2, dtype=torch.int64, pin_memory=True)
        torch.cuda.synchronize()

        def e2e_pass():
            dC.copy_(hC, non_blocking=True); dH.copy_(hH, non_blocking=True)
            if gated:
                dU.copy_(hU, non_blocking=True)
            hout.copy_(check(dC, dU, dH, out), non_blocking=True)
            torch.cuda.synchronize()

        e2e_pass()
        barrier()
        k2 = max(1, args.e2e_steps)
        w0 = time.perf_counter()
        for _ in range(k2):
            e2e_pass()
        e2e_s = rep.max_over_ranks((time.perf_counter() - w0) / k2)
        e2e = {"value": T * d_ff * world / e2e_s, "unit": "entries/s", "ms_per_step": e2e_s * 1e3, "steps": k2,
               "h2d_bytes_per_step": nbytes, "d2h_bytes_per_step": 16,
               "matches_device_path": [int(v) for v in hout] == got}
        del hC, hH, dC, dH, hU, dU
    res["e2e"] = e2e
    if not args.no_cpu_baseline and world == 1:
        from oracle import glue
        rows = min(T, 512)
        Ch, Hh = C[:rows].cpu().numpy(), H[:rows].cpu().numpy()
        Hh[rows // 2, 77] ^= 1                               # one planted difference, found by both sides
        Hd = H[:rows].clone()
        Hd[rows // 2, 77] ^= 1
        Uh = U[:rows].cpu().numpy() if gated else None
        w0 = time.perf_counter()
        if gated:
            want = glue.gated_link_check(Ch, Uh, Hh, np.array(act_host, dtype=np.int8), 9, 256, 7, 64, -127, 127)
        else:
            want = glue.requant_check(Ch, Hh, 9, 256, -127, 127)
        secs = time.perf_counter() - w0
        ok = [int(v) for v in check(C[:rows], U[:rows] if gated else None, Hd, out).cpu()] == list(want) and want[0] == 1
        res["cpu_baseline"] = {"value": rows * d_ff / secs, "unit": "entries/s", "cores": 1, "nproc": os.cpu_count(),
                               "kind": "oracle", "seconds": secs,
                               "sample": f"the first {rows} of the {T} rows, one planted difference, same inputs as the GPU run",
                               "gpu_matches_oracle": ok}
        if not ok:
            raise SystemExit("GPU link check differs from the oracle")
    if rank == 0:
        print(json.dumps(res))
    rep.close()


# ------------------------------------------------------------------------ hash commitments


def commit_workload(imm, synth, seed, T, n, dev):
    """Deployed logits of T decision steps cut into requests; one message and one 32-byte r per request."""
    ref = synth.reference_logits(seed, T, n, device=dev)
    dep = synth.deployed_logits(ref, seed, synth.NOISE_BENIGN)
    del ref
    requests = max(1, T // 128)
    off = synth.request_offsets(seed, T, requests, device="cpu").tolist()
    msgs = [dep[off[i]:off[i + 1]] for i in range(requests)]
    rs = [bytes((7 * i + j) & 255 for j in range(32)) for i in range(requests)]
    return dep, off, msgs, rs


def run_commit(args):
    """One step = the commitment psi = Hash(r, logits) of every request of the batch."""
    from paper_2602_22700_b200 import imm, synth
    from paper_2602_22700_b200.replicas import Replicas
    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    rep = Replicas("nccl", dev)
    imm.lib()
    warmup, steps = max(args.warmup, 3), max(args.steps, 1)
    T, n = args.tokens, args.vocab
    dep, off, msgs, rs = commit_workload(imm, synth, rep.seed(SEED), T, n, dev)
    nbytes = dep.numel() * 4
    com = imm.Committer(msgs, rs, device=dev)
    barrier = rep.barrier
    for _ in range(warmup):
        com.commit()
    barrier()
    sampler = ClockSampler(local_rank if "CUDA_VISIBLE_DEVICES" not in os.environ else
                           int(os.environ["CUDA_VISIBLE_DEVICES"].split(",")[local_rank]))
    sampler.start()
    time.sleep(0.25)
    flush = nbytes < 2 * L2_BYTES
    scrub = torch.empty(512 << 20, dtype=torch.uint8, device=dev) if flush else None
    pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    t0 = time.time()
    for a, b in pairs:
        if flush:
            scrub.fill_(1)
        a.record()
        com.commit()
        b.record()
    barrier()
    t1w = time.time()
    clocks = sampler.stop(t0, t1w)
    elapsed_ms = rep.max_over_ranks(sum(a.elapsed_time(b) for a, b in pairs))
    ms_per_step = elapsed_ms / steps
    digests = com.digests.cpu().numpy()
    gbs = nbytes / (ms_per_step * 1e-3) / 1e9
    sm_mhz = clocks.get("sm_mhz") or 1965.0
    alu_peak = COMMIT_ALU_PEAK_GBS_AT_1965 * sm_mhz / 1965.0
    res = {
        "metric": "committed bytes/sec", "value": nbytes * world / (ms_per_step * 1e-3), "unit": "B/s",
        "n_gpus": world, "steps": steps, "warmup": warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "u32", "data": "synthetic",
        "config": {"workload": workload_name("commit", 0, T, n), "tokens": T, "vocab": n, "requests": len(msgs),
                   "hash": "SHA-256, RFC 6962 tree over 4096-byte leaves, length-bound final hash with 32-byte r",
                   "input_bytes_per_gpu": nbytes,
                   "l2": ("L2 flushed between steps (512 MB overwritten outside the timed event pairs)" if flush else
                          f"inputs ({nbytes / 2**30:.2f} GiB) exceed the 126 MB L2 many times over; no flush"),
                   "parallelism": "1 GPU" if world == 1 else f"{world} independent replicas, no collective"},
        "hbm_gbs_whole_step": gbs,
        "roofline": {"kernel": "commit_leaf_kernel (SHA-256 of 4096-byte leaves, one per thread); timed as the whole imm_commit "
                               "call, of which the leaf kernel is 97 % in the launch list", "bound": "alu",
                     "achieved": gbs, "peak": alu_peak, "unit": "GB/s", "frac": gbs / alu_peak,
                     "peak_kind": "integer ALU pipe: 148 SMs x 64 lanes x sampled SM clock / 17.18 ALU instructions per hashed byte",
                     "traffic": (COMMIT_TRAFFIC_RATIO * nbytes) if COMMIT_TRAFFIC_RATIO else None},
        "gpu_launches": com.launches * steps,
        "clocks": clocks,
    }
    e2e = None
    if not args.no_e2e:
        host = torch.empty(dep.shape, dtype=dep.dtype, pin_memory=True).copy_(dep)
        stage = torch.empty_like(dep)
        smsgs = [stage[off[i]:off[i + 1]] for i in range(len(msgs))]
        com2 = imm.Committer(smsgs, rs, device=dev)
        out = torch.empty((len(msgs), 32), dtype=torch.uint8, pin_memory=True)
        torch.cuda.synchronize()

        def e2e_pass():
            stage.copy_(host, non_blocking=True)
            out.copy_(com2.commit(), non_blocking=True)
            torch.cuda.synchronize()

        e2e_pass()
        barrier()
        k2 = max(1, args.e2e_steps)
        w0 = time.perf_counter()
        for _ in range(k2):
            e2e_pass()
        e2e_s = rep.max_over_ranks((time.perf_counter() - w0) / k2)
        e2e = {"value": nbytes * world / e2e_s, "unit": "B/s", "ms_per_step": e2e_s * 1e3, "steps": k2,
               "h2d_bytes_per_step": nbytes, "d2h_bytes_per_step": out.numel(),
               "matches_device_path": bool((out.numpy() == digests).all())}
        del host, stage, com2
    res["e2e"] = e2e
    if not args.no_cpu_baseline and world == 1:
        from oracle import commitment
        pick, total = [], 0
        for i in sorted(range(len(msgs)), key=lambda i: msgs[i].numel()):
            if total + msgs[i].numel() * 4 > (6 << 30) and pick:
                break
            pick.append(i)
            total += msgs[i].numel() * 4
        data = {i: msgs[i].cpu().numpy().tobytes() for i in pick}
        w0 = time.perf_counter()
        want = {i: commitment.commit(data[i], rs[i]) for i in pick}
        secs = time.perf_counter() - w0
        ok = all(bytes(digests[i]) == want[i] for i in pick)
        res["cpu_baseline"] = {"value": total / secs, "unit": "B/s", "cores": 1, "nproc": os.cpu_count(),
                               "kind": "oracle", "seconds": secs,
                               "sample": f"{len(pick)} of the {len(msgs)} requests ({total} bytes), same inputs as the GPU run",
                               "gpu_matches_oracle": ok}
        if not ok:
            raise SystemExit("GPU commitments differ from the oracle")
    if rank == 0:
        print(json.dumps(res))
    rep.close()


# ------------------------------------------------------------------------ reference arm (CPU oracle)


def run_reference(args):
    rank, _, world = dist_env()
    if rank != 0:
        return
    from paper_2602_22700_b200 import synth
    device = "cuda" if torch.cuda.is_available() else "cpu"
    if args.config == "ldd":
        rows = 48
        ref = synth.reference_logits(SEED, rows, args.vocab, device=device)
        dep = synth.deployed_logits(ref, SEED, synth.NOISE_QUANTISED)
        topk = torch.topk(dep, args.topk, dim=1).indices.to(torch.int32)
        hdep, href, htop = dep.cpu().numpy(), ref.cpu().numpy(), topk.cpu().numpy()
        warmup, steps = max(args.warmup, 1), max(args.steps, 1)
        for _ in range(warmup):
            ldd_oracle_rows(hdep, href, htop, range(4))
        w0 = time.perf_counter()
        for _ in range(steps):
            ldd_oracle_rows(hdep, href, htop, range(rows))
        per = (time.perf_counter() - w0) / steps
        desc = f"{rows} decision steps of the workload per step, one thread"
        print(json.dumps({
            "impl": "reference", "metric": "LDD decision steps/sec", "value": rows / per, "unit": "steps/s",
            "n_gpus": world, "steps": steps, "warmup": warmup, "ms_per_step": per * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": workload_name("ldd", 0, args.tokens, args.vocab, args.topk), "tokens": args.tokens,
                       "vocab": args.vocab, "topk": args.topk, "sampled": desc},
            "cpu_baseline": {"value": rows / per, "unit": "steps/s", "cores": 1, "kind": "oracle", "sample": desc},
            "e2e": {"value": rows / per, "unit": "steps/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        }))
        return
    if args.config == "commit":
        from oracle import commitment
        rows = 256
        ref = synth.reference_logits(SEED, rows, args.vocab, device=device)
        data = synth.deployed_logits(ref, SEED, synth.NOISE_BENIGN).cpu().numpy().tobytes()
        r = bytes(range(32))
        warmup, steps = max(args.warmup, 1), max(args.steps, 1)
        for _ in range(warmup):
            commitment.commit(data[:1 << 20], r)
        w0 = time.perf_counter()
        for _ in range(steps):
            commitment.commit(data, r)
        per = (time.perf_counter() - w0) / steps
        desc = f"one request of {rows} decision steps ({len(data)} bytes) per step, one thread"
        print(json.dumps({
            "impl": "reference", "metric": "committed bytes/sec", "value": len(data) / per, "unit": "B/s",
            "n_gpus": world, "steps": steps, "warmup": warmup, "ms_per_step": per * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "u32", "data": "synthetic",
            "config": {"workload": workload_name("commit", 0, args.tokens, args.vocab), "tokens": args.tokens,
                       "vocab": args.vocab, "sampled": desc},
            "cpu_baseline": {"value": len(data) / per, "unit": "B/s", "cores": 1, "kind": "oracle", "sample": desc},
            "e2e": {"value": len(data) / per, "unit": "B/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        }))
        return
    if args.config == "glue":
        from oracle import glue
        rows = 512
        rng = np.random.default_rng(SEED)
        Ch = rng.integers(-70000, 70000, size=(rows, 14336)).astype(np.int32)
        Hh = glue.requantize(Ch, 9, 256, -127, 127)
        warmup, steps = max(args.warmup, 1), max(args.steps, 1)
        for _ in range(warmup):
            glue.requant_check(Ch[:32], Hh[:32], 9, 256, -127, 127)
        w0 = time.perf_counter()
        for _ in range(steps):
            glue.requant_check(Ch, Hh, 9, 256, -127, 127)
        per = (time.perf_counter() - w0) / steps
        desc = f"{rows} rows of 14336 entries per step, one thread"
        print(json.dumps({
            "impl": "reference", "metric": "checked entries/sec", "value": rows * 14336 / per, "unit": "entries/s",
            "n_gpus": world, "steps": steps, "warmup": warmup, "ms_per_step": per * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "i64", "data": "synthetic",
            "config": {"workload": workload_name("glue", 0, args.tokens), "tokens": args.tokens, "sampled": desc},
            "cpu_baseline": {"value": rows * 14336 / per, "unit": "entries/s", "cores": 1, "nproc": os.cpu_count(),
                             "kind": "oracle", "sample": desc},
            "e2e": {"value": rows * 14336 / per, "unit": "entries/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        }))
        return
    layers = min(args.layers, 2)
    tokens = args.tokens if device == "cuda" else min(args.tokens, 256)
    problems = make_problems(args.config, SEED, layers, tokens, device)[:8]
    sample = sample_to_host(problems)
    shapes = [p.mkn for p in problems]
    del problems
    threads = min(os.cpu_count() or 1, len(sample))
    macs = field_macs(shapes)
    warmup, steps = max(args.warmup, 1), max(args.steps, 1)
    for _ in range(warmup):
        oracle_time_sample(sample, threads)
    total = 0.0
    for _ in range(steps):
        secs, _ = oracle_time_sample(sample, threads)
        total += secs
    per = total / steps
    value = macs / per
    desc = f"the first {len(sample)} proofs of the workload at {tokens} tokens per step, one proof per thread"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world,
        "steps": steps, "warmup": warmup, "ms_per_step": per * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "u64", "data": "synthetic",
        "config": {"workload": workload_name(args.config, args.layers, args.tokens),
                   "layers": args.layers if args.config == "decoder" else None,
                   "tokens": args.tokens, "sampled": desc,
                   "note": None if tokens == args.tokens else "no CUDA device for input generation: token count reduced"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "nproc": os.cpu_count(),
                         "compiler": oracle_build_line(), "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    args = parse_args()
    if args.tokens is None:
        args.tokens = WORKLOADS[args.config][0]
    if args.impl == "reference":
        run_reference(args)
    elif args.config == "ldd":
        run_ldd(args)
    elif args.config == "commit":
        run_commit(args)
    elif args.config == "glue":
        run_glue(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
