#!/usr/bin/env python
"""Benchmark of the decode hot path (append/evict + progressive encode + decode attention).

One "step" = one decode step of the whole batch over all L layers, through ptenc_decode_step(layer=-1), in
steady state: every ring full, every sequence evicting one token per step.  Workload at 1 GPU = the
Qwen2.5-7B-shaped configuration the metric is quoted on; other workloads with --workload.

    python bench.py --gpus N --steps K --warmup W            (N > 1: under torch.distributed.run, or run directly,
                                                              in which case the script starts the N ranks itself)
    python bench.py --impl reference ...                     (times the CPU oracle on a bounded sample)

Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _oracle_worker(path: str) -> None:
    """One process of the CPU-oracle timing: loads its inputs (numpy arrays written by the parent), builds the
    oracle's cache for one layer, fills the window, says "ready", waits for "go" on stdin, runs the timed steps and
    prints the seconds they took.  Imports numpy and the oracle only, so that many of these start quickly."""
    import numpy as np
    from oracle.ptenc_oracle import OracleCache
    d = np.load(path, allow_pickle=False)
    n_seq, W, E, n_prompt = int(d["n_seq"]), int(d["window"]), int(d["evict_chunk"]), int(d["n_prompt"])
    orc = OracleCache(n_layers=1, batch=n_seq, n_q_heads=int(d["n_q_heads"]), n_kv_heads=int(d["n_kv_heads"]),
                      head_dim=int(d["head_dim"]), window=W, evict_chunk=E, n_global=int(d["n_global"]),
                      rank=int(d["rank"]), policy="score" if int(d["score_policy"]) else "fifo",
                      recent=int(d["recent"]) if int(d["score_policy"]) else 0)
    orc.set_encoder(0, **{k: d["enc_" + k] for k in ("Wq_a", "Wk_a", "Wv_a", "q_g", "k_g", "v_g")})
    q, k, v = d["q"], d["k"], d["v"]                      # [R, n_seq, H, D] each
    R = q.shape[0]
    if n_prompt > 0:
        orc.prefill(0, d["Kp"], d["Vp"], [n_prompt] * n_seq)
    for t in range(W - n_prompt):                         # fill (not timed)
        orc.append_evict(0, k[t % R], v[t % R])
    for t in range(int(d["warm"])):
        orc.decode_step(0, q[t % R], k[t % R], v[t % R])
    print("ready", flush=True)
    sys.stdin.readline()
    n_steps = int(d["n_steps"])
    w0, c0 = time.perf_counter(), time.process_time()
    for t in range(n_steps):
        orc.decode_step(0, q[t % R], k[t % R], v[t % R])
    print(json.dumps({"wall": time.perf_counter() - w0, "cpu": time.process_time() - c0}), flush=True)


if __name__ == "__main__" and len(sys.argv) == 3 and sys.argv[1] == "--oracle-worker":
    _oracle_worker(sys.argv[2])
    sys.exit(0)

import numpy as np  # noqa: E402
import torch  # noqa: E402

from ptenc_inputs import CONFIGS, make_inputs, stress_config  # noqa: E402

METRIC = "decode_tokens_per_s"
UNIT = "tokens/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
# DRAM bytes moved (read + written, ncu counters) per algorithmic byte of the tensor-core attention kernel, keyed by
# window: each ratio was measured on a launch with a smaller batch of the same head shape and window (tile loads
# without the L2 hint, as in the launches it is scaled to; the profiler flushes the caches before every pass, so the
# hinted build reads the same), and DRAM traffic grows in proportion to the K/V tiles a launch reads.  Windows with no
# capture report no traffic figure.
ATTN_DRAM_BYTES_PER_ALGORITHMIC_BYTE = {512: 1.0036, 2048: 1.0040}


def workload_cfg(name: str) -> dict:
    if name.startswith("stress"):
        _, w, b = name.split("-")          # e.g. stress-w512-b16
        c = stress_config(int(w[1:]), int(b[1:]))
    else:
        c = dict(CONFIGS[name])
    c.pop("ragged", None)
    return c


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def live_after(t: int, W: int, E: int, P: int = 0) -> int:
    """Tokens a sequence holds after its t-th decoded token (0-based) arrived: P pinned prompt tokens plus the sliding
    part, which fills its W - P slots and then, on every E-th arrival, is found full and evicts E tokens."""
    cap = W - P
    E = min(E, cap)
    return P + (t + 1 if t < cap else cap - E + 1 + (t - cap) % E)


def evicts_at(t: int, W: int, E: int, P: int = 0) -> bool:
    cap = W - P
    return t >= cap and (t - cap) % min(E, cap) == 0


def bytes_model(c: dict, E: int = 1, steps=None, P: int = 0, score_policy: bool = False) -> dict:
    """Algorithmic bytes (all layers, all sequences active) summed over the given steps (token indices); one
    full-window evicting step when `steps` is None.  Per layer and sequence: the live K and V rows + q + o for the
    attention, the arriving K/V rows for the append, and on an evicting step the E evicted K/V rows + the state read
    and written."""
    L, B, Hq, Hkv, D, W = c["n_layers"], c["batch"], c["n_q_heads"], c["n_kv_heads"], c["head_dim"], c["window"]
    elt = 2 if c["dtype"] == "bf16" else 4
    d_q, d_kv = Hq * D, Hkv * D
    if steps is None:
        steps = [W]
        live = [W]
        ev = [True]
    else:
        live = [live_after(t, W, E, P) for t in steps]
        ev = [evicts_at(t, W, E, P) for t in steps]
    attn = sum(L * B * (2 * n * d_kv * elt + 2 * d_q * elt) for n in live)          # K,V window + q + o
    append = len(live) * L * B * 2 * d_kv * elt
    enc = sum(L * B * (2 * min(E, W - P) * d_kv * elt + 2 * c["n_global"] * c["rank"] * 4) for e in ev if e)
    if score_policy:
        # importance-aware eviction: the per-slot scores are read and written once per step (fp32).  The logits that
        # carry the attention mass from the attention kernel to the scores are this implementation's traffic, not the
        # method's, and count against the achieved figure.
        append += sum(L * B * 2 * (n - P) * 4 for n in live)
    return {"attn": attn, "step": attn + append + enc, "attn_per_step": [L * B * (2 * n * d_kv * elt + 2 * d_q * elt)
                                                                          for n in live]}


# ======================================================================================== clocks sampling
class ClockSampler:
    COLS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
            "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
            "clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.proc = None
        self.path = f"/tmp/ptenc_clocks_{os.getpid()}.csv"
        try:
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            sel = uuid if uuid.startswith("GPU-") else "GPU-" + uuid
        except Exception:
            sel = str(device_index)
        self.cmd = ["nvidia-smi", "-i", sel, f"--query-gpu={self.COLS}", "--format=csv,noheader,nounits", "-lms", "50"]

    def start(self):
        try:
            self.f = open(self.path, "w")
            self.proc = subprocess.Popen(self.cmd, stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.f.close()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        try:
            for line in open(self.path):
                parts = [x.strip() for x in line.split(",")]
                if len(parts) < 7:
                    continue
                try:
                    sm.append(float(parts[0]))
                    mx.append(float(parts[1]))
                except ValueError:
                    continue
                for nm, val in zip(names, parts[3:7]):
                    if val.lower() == "active":
                        reasons.add(nm)
            os.remove(self.path)
        except Exception:
            pass
        if sm:
            hi = [x for x in sm if x >= 0.5 * max(sm)]       # samples taken under load
            out.update(sm_mhz=statistics.median(hi), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


# ======================================================================================== CPU oracle legs
def host_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except Exception:
        return os.cpu_count() or 1


def oracle_sample(c: dict, n_seq: int, n_steps: int, warm: int = 1, E: int = 1, n_prompt: int = 0, workers: int = 1,
                  policy: str = "fifo", recent: int = 0):
    """Times the CPU oracle, as it stands, on `workers` processes at once, each holding 1 layer x n_seq sequences of
    its own at the full window (sequences are independent, so this is how the oracle uses many cores).  Every
    process runs single-threaded; all start their timed steps together.  Returns (seconds per sampled step = the
    slowest process's, processes, cpu-seconds used per wall-second)."""
    tmp = f"/tmp/ptenc_oracle_{os.getpid()}"
    os.makedirs(tmp, exist_ok=True)
    cc = {**c, "n_layers": 1, "batch": n_seq}
    env = {**os.environ, "OMP_NUM_THREADS": "1", "OPENBLAS_NUM_THREADS": "1", "MKL_NUM_THREADS": "1"}
    procs, paths = [], []
    for w in range(workers):
        gen = make_inputs(cc, seed=1000 + w, device="cpu")          # every process decodes its own sequences
        P = gen.encoder_params(0)
        R = 4
        q = np.stack([gen.step_q(t)[0].double().numpy() for t in range(R)])
        kv = [gen.step_kv(t) for t in range(R)]
        arrays = dict(n_seq=n_seq, window=c["window"], evict_chunk=E, n_prompt=n_prompt, n_q_heads=c["n_q_heads"],
                      n_kv_heads=c["n_kv_heads"], head_dim=c["head_dim"], n_global=c["n_global"], rank=c["rank"],
                      warm=warm, n_steps=n_steps, score_policy=int(policy == "score"), recent=recent, q=q, k=np.stack([x[0][0].double().numpy() for x in kv]),
                      v=np.stack([x[1][0].double().numpy() for x in kv]),
                      **{"enc_" + k: v.double().numpy() for k, v in P.items()})
        if n_prompt > 0:
            shape = (1, n_seq, n_prompt, c["n_kv_heads"], c["head_dim"])
            arrays["Kp"] = gen.generic(50, 0, shape, 1.0)[0].double().numpy()
            arrays["Vp"] = gen.generic(51, 0, shape, 1.0)[0].double().numpy()
        path = os.path.join(tmp, f"w{w}.npz")
        np.savez(path, **arrays)
        paths.append(path)
        procs.append(subprocess.Popen([sys.executable, os.path.join(ROOT, "bench.py"), "--oracle-worker", path],
                                      stdin=subprocess.PIPE, stdout=subprocess.PIPE, text=True, env=env, cwd=ROOT))
    try:
        for p in procs:
            if p.stdout.readline().strip() != "ready":
                raise RuntimeError("oracle worker failed to start")
        for p in procs:
            p.stdin.write("go\n")
            p.stdin.flush()
        res = [json.loads(p.stdout.readline()) for p in procs]
    finally:
        for p in procs:
            try:
                p.stdin.close()
            except Exception:
                pass
            p.wait(timeout=60)
        for path in paths:
            try:
                os.remove(path)
            except OSError:
                pass
        try:
            os.rmdir(tmp)
        except OSError:
            pass
    wall = max(r["wall"] for r in res)
    return wall / n_steps, workers, sum(r["cpu"] for r in res) / wall


def oracle_baseline(c: dict, n_steps: int, E: int, n_prompt: int, warm: int = 1, policy: str = "fifo",
                    recent: int = 0) -> dict:
    """The oracle on one core and on all host cores; tokens/s normalised to all L layers."""
    L, B, W = c["n_layers"], c["batch"], c["window"]
    nproc = host_cores()
    n1 = min(8, B)
    kw = dict(warm=warm, E=E, n_prompt=n_prompt, policy=policy, recent=recent)
    sec1, _, busy1 = oracle_sample(c, n1, n_steps, workers=1, **kw)
    nw = 2                                                   # sequences per process on the all-cores leg
    secN, P, busyN = oracle_sample(c, nw, n_steps, workers=nproc, **kw)
    return {
        "value": P * nw / (secN * L), "unit": UNIT, "cores": P, "nproc": nproc, "kind": "oracle",
        "cpu_seconds_per_wall_second": busyN,
        "one_core": {"value": n1 / (sec1 * L), "unit": UNIT, "cores": 1, "cpu_seconds_per_wall_second": busy1,
                     "seconds_per_sampled_step": sec1,
                     "sample": f"1 process x {n1} of {B} sequences x 1 of {L} layers x {n_steps} steps"},
        "seconds_per_sampled_step": secN,
        "sample": (f"oracle decode_step, as it stands: {P} single-threaded processes (one per host core) x {nw} sequences "
                   f"each x 1 of {L} layers x {n_steps} steps at window {W} (full, evicting), timed together; "
                   f"tokens/s = sequences / (step time x {L} layers)"),
    }


def run_reference(args, c: dict):
    """--impl reference: the oracle on a bounded sample; tokens/s normalised to all L layers."""
    if rank_env()[0] != 0:
        return
    base = oracle_baseline(c, max(1, args.steps), args.evict_chunk, args.prompt_len, warm=max(1, args.warmup),
                           policy=args.policy, recent=args.recent)
    L, B = c["n_layers"], c["batch"]
    seqs = base["cores"] * 2
    line = {
        "impl": "reference", "metric": METRIC, "value": base["value"], "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup,
        # measured: one sampled step = every process decoding one token for its sequences in one layer
        "ms_per_step": base["seconds_per_sampled_step"] * 1e3,
        "ms_per_full_step_extrapolated": base["seconds_per_sampled_step"] * 1e3 * L * B / seqs,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_block(args, c),
        "cpu_baseline": base,
        "e2e": {"value": base["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def l2_note(c: dict) -> str:
    elt = 2 if c["dtype"] == "bf16" else 4
    ring = 2 * c["n_layers"] * c["batch"] * c["n_kv_heads"] * c["head_dim"] * c["window"] * elt
    if ring > 4 * 126e6:
        return f"K/V rings read per step ({ring / 2**30:.2f} GiB) exceed the 126 MB L2 by {ring / 126e6:.0f}x; no flush needed"
    return (f"K/V rings ({ring / 2**20:.2f} MiB) fit the 126 MB L2 and are not flushed: this workload is latency-bound and "
            "carries no roofline claim")


def config_block(args, c: dict) -> dict:
    return {"workload": args.workload, "n_layers": c["n_layers"], "batch_per_gpu": c["batch"],
            "n_q_heads": c["n_q_heads"], "n_kv_heads": c["n_kv_heads"], "head_dim": c["head_dim"],
            "window": c["window"], "evict_chunk": args.evict_chunk, "pinned_prompt": args.prompt_len,
            "policy": args.policy + (f" (recent {args.recent})" if args.policy == "score" else ""), "n_global": c["n_global"], "rank": c["rank"],
            "phase": ("steady state: rings full, one eviction + encode per sequence per step" if args.evict_chunk == 1
                      else f"steady state: rings between {c['window'] - args.evict_chunk + 1} and {c['window']} tokens, "
                           f"every {args.evict_chunk}-th step evicts and encodes {args.evict_chunk} tokens per sequence"),
            "launch_mode": "all layers per call (layer = -1)",
            "l2": l2_note(c),
            "parallelism": f"dp{args.gpus} (batch shards, no collective on the path)"}


# ======================================================================================== rank plumbing
def rank_env():
    """(rank, world size, local rank) from the launcher's environment; (0, 1, 0) when run directly."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def launcher_argv(n_gpus: int, argv) -> list:
    """The command that runs this script as n_gpus ranks on one node (one process per GPU, rendezvous on the loopback
    address)."""
    import socket
    sock = socket.socket()
    sock.bind(("127.0.0.1", 0))
    port = sock.getsockname()[1]
    sock.close()
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n_gpus}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.join(ROOT, "bench.py"), *argv]


def ensure_ranks(args) -> None:
    """`--gpus N` with N > 1 needs N ranks.  Started by a launcher (WORLD_SIZE set) the two must agree; started
    directly, the script starts the ranks itself and this process becomes the launcher."""
    world = os.environ.get("WORLD_SIZE")
    if world is not None:
        if int(world) != args.gpus:
            sys.exit(f"bench.py: --gpus {args.gpus} but the launcher started {world} ranks")
        return
    if args.gpus > 1:
        cmd = launcher_argv(args.gpus, sys.argv[1:])
        os.execv(cmd[0], cmd)


def run_dry(args, c: dict):
    """--dry-run: the rank plumbing alone (process group on gloo, barrier, max over ranks, one line from rank 0), no
    GPU and no kernels.  Not a measurement."""
    rank, world, local = rank_env()
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("gloo")
        dist.barrier()
    ms = max_over_ranks([float(rank + 1)], dist, "cpu")[0]
    if rank == 0:
        print(json.dumps({"dry_run": True, "n_gpus": world, "ranks_seen_max_ms": ms,
                          "config": config_block(args, c)}), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def shard_seed(rank: int) -> int:
    """Each rank decodes its own batch shard: same shapes, its own synthetic stream.  Sequences are independent on
    this path (own ring, own state), so the shards never exchange data."""
    return int(rank)


def max_over_ranks(values, dist, device):
    """Element-wise maximum of a list of per-rank timings over all ranks (the slowest rank sets the job's time)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def job_tokens_per_s(world: int, batch_per_rank: int, steps: int, ms_total: float) -> float:
    """Whole-job throughput: every rank decodes batch_per_rank tokens per step (weak scaling)."""
    return world * batch_per_rank * steps / (ms_total * 1e-3)


# ======================================================================================== GPU leg
def run_gpu(args, c: dict):
    import paper_2602_16839_b200 as pt

    rank, world, local = rank_env()
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)

    L, B, Hq, Hkv, D, W = c["n_layers"], c["batch"], c["n_q_heads"], c["n_kv_heads"], c["head_dim"], c["window"]
    gen = make_inputs(c, seed=shard_seed(rank), device=dev)
    E = args.evict_chunk
    score_policy = args.policy == "score"
    cfg = pt.make_config(n_layers=L, batch=B, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=D, window=W, evict_chunk=E,
                         n_global=c["n_global"], rank=c["rank"], dtype=c["dtype"], device=local,
                         policy=pt.binding.POLICY_SCORE if score_policy else pt.binding.POLICY_FIFO,
                         recent=args.recent if score_policy else 0)
    cache = pt.Cache(cfg)
    for l in range(L):
        P = gen.encoder_params(l)
        cache.set_encoder(l, P["Wq_a"], P["Wk_a"], P["Wv_a"], P["q_g"], P["k_g"], P["v_g"])

    # input pool: R distinct steps' worth of q/k/v, resident in HBM and mirrored in pinned host memory
    R = 4
    pool = []
    for t in range(R):
        k, v = gen.step_kv(t)
        pool.append((gen.step_q(t), k, v))
    out = torch.empty_like(pool[0][0])

    # pinned prompt (Sec. 3.3 / 4.1 policy), then fill the rings (untimed): the sliding part reaches its capacity;
    # warm-up steps then run in steady state
    P = args.prompt_len
    if P > 0:
        Kp = gen.generic(50, 0, (L, B, P, Hkv, D), 1.0)
        Vp = gen.generic(51, 0, (L, B, P, Hkv, D), 1.0)
        cache.prefill(-1, Kp, Vp, torch.full((B,), P, dtype=torch.int32, device=dev), P)
        del Kp, Vp
    for t in range(W - P):
        q, k, v = pool[t % R]
        cache.append_evict(-1, k, v)
    torch.cuda.synchronize()

    def sync_all():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    # ---- device-resident timing -----------------------------------------------------------------------
    K, Wm = args.steps, args.warmup
    for t in range(Wm):
        cache.decode_step(-1, *pool[t % R], out)
    ev_a = [torch.cuda.Event(enable_timing=True) for _ in range(K)]
    ev_b = [torch.cuda.Event(enable_timing=True) for _ in range(K)]
    for e in ev_a + ev_b:
        e.record()                                   # creates the CUDA handles
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local) if rank == 0 else None
    sync_all()
    launches0 = cache.launch_count()
    if sampler:
        sampler.start()
        time.sleep(0.12)
    torch.cuda.nvtx.range_push("ptenc_timed")
    e0.record()
    for t in range(K):
        cache.decode_step(-1, *pool[t % R], out)
    e1.record()
    sync_all()
    ms_total = e0.elapsed_time(e1)
    launches = cache.launch_count() - launches0
    # the same K steps once more with an event pair around every attention launch (for the roofline of that kernel);
    # an event in front of the launch makes it an ordinary serialised launch, so these steps are a little slower than
    # the ones timed above and are not part of `value`
    e2, e3 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e2.record()
    for t in range(K):
        cache.time_next_attn(ev_a[t], ev_b[t])
        cache.decode_step(-1, *pool[(K + t) % R], out)
    e3.record()
    sync_all()
    torch.cuda.nvtx.range_pop()
    ms_total_events = e2.elapsed_time(e3)
    attn_ms = [a.elapsed_time(b) for a, b in zip(ev_a, ev_b)]
    clocks = sampler.stop() if sampler else None
    status = cache.status()
    cache_info = cache.info()

    # ---- end to end: host buffers in, host buffer out, through ptenc_decode_step_host ------------------------
    hpool = [tuple(x.cpu().pin_memory() for x in p) for p in pool]
    hout = torch.empty(out.shape, dtype=out.dtype).pin_memory()
    staging = torch.empty(cache.host_staging_bytes(-1), dtype=torch.uint8, device=dev)
    Ke = max(3, min(K, 100)) if E == 1 else E          # chunked eviction: one whole period of E steps
    for t in range(3):
        cache.decode_step_host(-1, *hpool[t % R], hout, staging)
    sync_all()
    h0, h1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    h0.record()
    for t in range(Ke):
        cache.decode_step_host(-1, *hpool[t % R], hout, staging)
    h1.record()
    sync_all()
    ms_e2e = h0.elapsed_time(h1)
    h2d = sum(x.numel() * x.element_size() for x in hpool[0])
    d2h = hout.numel() * hout.element_size()

    # ---- side measurements of the two kernels that the step average hides (rank 0, on request) -------------------------
    extras = {}
    if rank == 0 and args.extras:
        def timed(fn, n=20, flush=None):
            ts = []
            for _ in range(n):
                if flush is not None:
                    flush.zero_()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(); fn(); b.record()
                torch.cuda.synchronize()
                ts.append(a.elapsed_time(b))
            ts.sort()
            return ts[len(ts) // 2]
        elt = 2 if c["dtype"] == "bf16" else 4
        G, r, d_kv, d_q = c["n_global"], c["rank"], Hkv * D, Hq * D
        if E > 1:
            # the encoder's burst: every sequence folds a chunk of E staged rows (the rows staged by the last evicting
            # step are folded again on each call; the arithmetic and the traffic are those of a real burst)
            n_done = (W - P) + Wm + 2 * K + 3 + Ke                # decoded tokens so far (fill, warm-up, the timed loops)
            t = n_done
            while not evicts_at(t, W, E, P):
                t += 1
            for i in range(n_done, t + 1):                        # run on to the next evicting step
                cache.append_evict(-1, pool[i % R][1], pool[i % R][2])
            Ee = min(E, W - P)
            torch.cuda.nvtx.range_push("ptenc_extras_encode")
            ms = timed(lambda: cache.encode(-1))
            torch.cuda.nvtx.range_pop()
            by = L * B * (2 * Ee * d_kv * elt + 2 * G * r * 4)
            fl = L * B * Ee * (4 * d_kv * r + 4 * r * r) + L * B * 2 * G * r * r
            extras["encode_burst"] = {"ms": ms, "algorithmic_gbs": by / ms / 1e6, "tflops": fl / ms / 1e9,
                                      "rows_per_sequence": Ee, "tensor_core_encode": cache.info()["tensor_core_encode"],
                                      "how": "median of 20 ptenc_encode(layer=-1) calls on the staged chunk, CUDA events"}
        # the dynamic weight update on a d_q x d_q projection, L2 flushed before each call
        Am = gen.generic(60, 0, (L, d_q, G), G ** -0.5)
        Bw = gen.generic(61, 0, (L, r, d_q), d_q ** -0.5)
        xin = gen.generic(62, 0, (L, B, d_q), 1.0)
        yio = gen.generic(63, 0, (L, B, d_q), 1.0)
        flush = torch.empty(256 * 2 ** 20, dtype=torch.uint8, device=dev)
        torch.cuda.nvtx.range_push("ptenc_extras_lora")
        ms = timed(lambda: cache.lora_apply(-1, Am, Bw, xin, yio), flush=flush)
        torch.cuda.nvtx.range_pop()
        by = L * (2 * G * d_q * elt + B * (3 * d_q * elt + G * r * 4))
        extras["lora_apply"] = {"ms": ms, "algorithmic_gbs": by / ms / 1e6, "d_in": d_q, "d_out": d_q,
                                "how": "median of 20 ptenc_lora_apply(layer=-1) calls, L2 flushed, CUDA events"}
        del Am, Bw, xin, yio, flush

    # ---- max over ranks -------------------------------------------------------------------------------------
    ms_total, ms_e2e = max_over_ranks([ms_total, ms_e2e], dist, dev)

    if rank == 0:
        timed_tokens = list(range(W - P + Wm, W - P + Wm + K))  # decoded-token index arriving at each timed step
        bm = bytes_model(c, E, timed_tokens, P, score_policy)
        bm_ev = bytes_model(c, E, [t + K for t in timed_tokens], P, score_policy)     # the pass with events
        peak, peak_kind = measured_peak()
        ms_step = ms_total / K
        attn_avg_ms = sum(attn_ms) / len(attn_ms)
        attn_gbs = bm_ev["attn"] / (sum(attn_ms) * 1e-3) / 1e9
        step_gbs = bm["step"] / (ms_total * 1e-3) / 1e9
        bm["attn"] /= K                                          # per launch / per step averages from here on
        bm["step"] /= K
        counted = cache_info["tensor_core_attn"] and P == 0 and E == 1 and not score_policy   # the captured launch shape
        ratio = ATTN_DRAM_BYTES_PER_ALGORITHMIC_BYTE.get(W) if counted else None
        traffic = ratio * bm["attn"] if ratio is not None else None
        bm.pop("attn_per_step")
        line = {
            "metric": METRIC, "value": job_tokens_per_s(world, B, K, ms_total), "unit": UNIT, "n_gpus": world,
            "steps": K, "warmup": Wm, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": c["dtype"], "data": "synthetic",
            "config": config_block(args, c),
            "clocks": clocks,
            "e2e": {"value": job_tokens_per_s(world, B, Ke, ms_e2e), "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e / Ke, "steps": Ke,
                    "call": "ptenc_decode_step_host (pinned host q/k/v in, host out)"},
            "gpu_launches": launches,
            "roofline": {"bound": "hbm", "kernel": ("decode attention (k_attn_bf16)" if cache_info["tensor_core_attn"]
                                                     else "decode attention (k_attn_generic)"), "achieved": attn_gbs,
                         "peak": peak, "peak_kind": f"of {peak_kind} copy bandwidth", "unit": "GB/s",
                         "frac": attn_gbs / peak, "frac_of_8tbs": attn_gbs / NOMINAL_HBM_GBS,
                         "traffic": traffic, "algorithmic_bytes_per_launch": bm["attn"],
                         "avg_launch_ms": attn_avg_ms, "share_of_step": attn_avg_ms / (ms_total_events / K),
                         "timed": f"{K} launches with an event pair each, in a second pass over the same steps "
                                  f"({ms_total_events / K:.4f} ms per step with the events in place)"},
            "hbm": {"step_algorithmic_gbs": step_gbs, "frac_of_8tbs": step_gbs / NOMINAL_HBM_GBS,
                    "frac_of_measured": step_gbs / peak, "algorithmic_bytes_per_step": bm["step"]},
            "device_status": status,
            **({"extras": extras} if extras else {}),
        }
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = oracle_baseline(c, args.cpu_steps, E, P, policy=args.policy, recent=args.recent)
        print(json.dumps(line), flush=True)
    cache.close()
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="qwen7b",
                    help="tiny | qwen3b | qwen7b | llama8b | stress-w<W>-b<B>")
    ap.add_argument("--evict-chunk", type=int, default=1,
                    help="tokens evicted at once when a ring is full (1 = ring per step, the timed configuration; "
                         "window/4 is the setting of the paper's runs, Sec. 4.1)")
    ap.add_argument("--n-global", type=int, default=0,
                    help="number of state vectors G (0 = the workload's own, 32; the paper's ablation uses 16/32/48/64)")
    ap.add_argument("--prompt-len", type=int, default=0,
                    help="tokens of a pinned prompt per sequence (kept for the whole rollout; the window slides over "
                         "the remaining slots)")
    ap.add_argument("--policy", default="fifo", choices=["fifo", "score"],
                    help="which tokens leave a full cache: the oldest (sliding window, the timed configuration) or the "
                         "ones that received the least attention so far (Sec. 4.3, token dropping)")
    ap.add_argument("--recent", type=int, default=256,
                    help="--policy score: the newest RECENT tokens are never evicted")
    ap.add_argument("--cpu-steps", type=int, default=96, help="steps of the CPU-oracle sample")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--dry-run", action="store_true",
                    help="exercise the launch and rank plumbing only (gloo, no GPU, no kernels); prints a line marked "
                         "dry_run")
    ap.add_argument("--extras", action="store_true",
                    help="also time the encoder's burst on a staged chunk (with --evict-chunk > 1) and the dynamic "
                         "weight update, each alone")
    args = ap.parse_args()
    c = workload_cfg(args.workload)
    if args.n_global > 0:
        c["n_global"] = args.n_global
    if args.impl == "reference":
        run_reference(args, c)
        return
    ensure_ranks(args)
    if args.dry_run:
        run_dry(args, c)
        return
    if args.warmup < 3:
        args.warmup = 3
    run_gpu(args, c)


if __name__ == "__main__":
    main()
