"""Benchmark of the FastMTP draft / verify hot path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--batch B] [--subset N] [--ctx L | --ctx-min A --ctx-max B] [--draft-steps K]
                    [--subset-kind uniform|zipf] [--no-cpu-baseline]
    python bench.py --sweep                      subset x batch x K table (one JSON line per point)
    python bench.py --target-layers L [--batch B]  fastmtp_target_step on a random L-layer target
    python bench.py --e2e-loop                   greedy vs speculative decoding loops at full depth, oracle-checked

One step = one pass of the hot path over one batch of synthetic input: fastmtp_draft (the K
recursive MTP steps with the compressed-vocabulary head, one kernel launch) followed by
fastmtp_verify_accept on target logits [B, K+1, V]. The default workload is the 7B-class head at
batch 1 (d=3584, 28/4 heads of 128, ffn 18944, V=152064, subset 32768, 2048 cached tokens, K=3).

Prints one JSON line (rank 0). `value` is draft tokens per second with every input resident in
HBM; `e2e` is the same through the *_host entry points (pinned host buffers in, results out).
With --gpus N > 1 (launched under torch.distributed.run) every rank runs an independent replica
on its own sequences: sequences are the unit the path shards by, and no data crosses GPUs.
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

import numpy as np


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--batch", type=int, default=1)
    ap.add_argument("--subset", type=int, default=32768, help="compressed vocabulary size (0 = full vocabulary)")
    ap.add_argument("--subset-kind", default="uniform", choices=["uniform", "zipf"])
    ap.add_argument("--ctx", type=int, default=2048, help="cached context tokens per sequence")
    ap.add_argument("--ctx-min", type=int, default=0, help="with --ctx-max: ragged contexts, uniform integers in [min, max]")
    ap.add_argument("--ctx-max", type=int, default=0)
    ap.add_argument("--draft-steps", type=int, default=3)
    ap.add_argument("--shape", default="7b", choices=["7b", "tiny"])
    ap.add_argument("--seed", type=int, default=1234)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--target-layers", type=int, default=0,
                    help="instead of the draft path, time fastmtp_target_step on a random target of this many layers "
                         "(1 row and draft-steps+1 rows per sequence); one JSON line per row count")
    ap.add_argument("--e2e-loop", action="store_true",
                    help="the end-to-end configuration: random 28-layer target of the 7B-class shape + the MTP layer, 512-token "
                         "prompt, 256 generated tokens, draft-steps=3, subset 32768; greedy and speculative decoding by the library "
                         "(token-identical), the oracle on the first 16 tokens; one JSON line")
    ap.add_argument("--loop-layers", type=int, default=28)
    ap.add_argument("--loop-prompt", type=int, default=512)
    ap.add_argument("--loop-tokens", type=int, default=256)
    ap.add_argument("--loop-oracle-tokens", type=int, default=16)
    ap.add_argument("--sweep", action="store_true",
                    help="vocabulary-compression sweep on one GPU: subset size x batch x draft steps, one JSON line each")
    return ap.parse_args()


def algorithmic_bytes_per_draft_step(s, B, N, ctx_lens, k):
    """Bytes one MTP draft step must move: every weight of the head once (projection, decoder
    layer, the N gathered output-head rows), the cached K/V of every sequence up to the current
    position, the embedding rows and the norm gains (bf16 = 2 bytes)."""
    qd, kvd = s.n_q_heads * s.head_dim, s.n_kv_heads * s.head_dim
    weights = 2 * s.d * s.d + s.d * (qd + 2 * kvd) + qd * s.d + 3 * s.d * s.ffn + N * s.d
    kv = sum(2 * kvd * (int(L) + k) for L in ctx_lens)          # K and V entries
    return 2 * weights + 2 * kv + B * 2 * s.d + 10 * s.d


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.rows = []
        self.proc = None
        self.index = index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), line.strip()))

    def stop(self, t0, t1):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        rows = [r for t, r in self.rows if t0 - 0.05 <= t <= t1 + 0.15] or [r for _, r in self.rows]
        for r in rows:
            f = [x.strip() for x in r.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# DRAM traffic of one mega_kernel launch on the default workload, from the ncu capture summarised in
# profiles/mega_kernel_7b_batch1_ncu.md (dram__bytes_read.sum + dram__bytes_write.sum). It is only
# reported while the kernel sources are the ones the counters were taken from.
NCU_TRAFFIC = {"bytes_per_launch": 2261864960 + 4352000, "sources_sha256": "a1f7629c6b7ad52b9c2a1297dd01150a4472d763b732ac45c7092491a3c4fcda"}
def kernel_sources_sha256():
    """Hash of every source the library is compiled from (all of csrc/ and the public header)."""
    import hashlib
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2509_18362_b200", "csrc")
    files = sorted(os.path.join(csrc, f) for f in os.listdir(csrc) if f.endswith((".cu", ".cuh")))
    for f in files + [os.path.join(ROOT, "include", "fastmtp.h")]:
        with open(f, "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def make_inputs(a, rank):
    from paper_2509_18362_b200 import inputs as I
    s = I.QWEN7B if a.shape == "7b" else I.TINY
    seed = a.seed + 1000 * rank
    N = a.subset if 0 < a.subset < s.vocab else s.vocab
    K = a.draft_steps
    W = I.mtp_weights(s, a.seed)                     # same model on every replica
    if a.ctx_max > 0:
        ctx_lens = [int(x) for x in I.context_lengths(a.batch, a.ctx_min, a.ctx_max, seed + 6)]
    else:
        ctx_lens = [a.ctx] * a.batch
    kv = I.paged_kv(s, ctx_lens, K + 1, seed + 1)
    h = I.hidden_bf16(seed + 2, (a.batch, s.d))
    tok = I.token_ids(seed + 3, (a.batch,), s.vocab)
    if N >= s.vocab:
        ids = None
    elif a.subset_kind == "uniform":
        ids = I.subset_uniform(s.vocab, N, a.seed + 4)
    else:
        ids = I.subset_zipf(s.vocab, N, a.seed + 4)
    vcase = I.verify_case(a.batch, K, s.vocab, seed + 5)
    return s, N, K, W, kv, h, tok, ids, vcase, ctx_lens


def workload_name(a, s, N):
    return (f"{a.shape} MTP head draft+verify: d={s.d} Hq/Hkv={s.n_q_heads}/{s.n_kv_heads} dh={s.head_dim} "
            f"ffn={s.ffn} V={s.vocab} subset={N}({a.subset_kind}) "
            + (f"ctx=uniform[{a.ctx_min},{a.ctx_max}]" if a.ctx_max > 0 else f"ctx={a.ctx}") + f" page={s.page_size}")


def cpu_oracle_sample(s, W, kv, h, tok, ids, vcase, K, seconds=12.0, max_calls=6):
    """Times the oracle as it stands on sequence 0 of the workload: repeated K-step drafts plus
    verification. Returns (draft tokens/s, cores, description)."""
    from oracle import fastmtp_oracle as O
    cores = os.cpu_count() or 1
    try:
        from threadpoolctl import threadpool_info
        nt = [p.get("num_threads", 1) for p in threadpool_info()]
        if nt:
            cores = max(nt)
    except Exception:
        pass
    kv1 = {k: (v.copy() if isinstance(v, np.ndarray) else v) for k, v in kv.items()}
    kv1["block_table"] = kv1["block_table"][:1]
    kv1["seq_lens"] = kv1["seq_lens"][:1]
    times = []
    t_begin = time.perf_counter()
    for _ in range(max_calls):
        t0 = time.perf_counter()
        O.draft(s, W, h[:1], tok[:1], kv1, K, ids)
        O.verify_accept(vcase["logits"][:1], vcase["drafts"][:1])
        times.append(time.perf_counter() - t0)
        if time.perf_counter() - t_begin > seconds:
            break
    best = min(times)
    return K / best, cores, f"{len(times)} calls of draft(K={K})+verify on sequence 0 of the workload, best call {best:.3f} s"


def run_reference(a):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    s, N, K, W, kv, h, tok, ids, vcase, _ = make_inputs(a, 0)
    from oracle import fastmtp_oracle as O
    kv1 = {k: (v.copy() if isinstance(v, np.ndarray) else v) for k, v in kv.items()}
    kv1["block_table"], kv1["seq_lens"] = kv1["block_table"][:1], kv1["seq_lens"][:1]
    cores = os.cpu_count() or 1

    def step():
        O.draft(s, W, h[:1], tok[:1], kv1, K, ids)
        O.verify_accept(vcase["logits"][:1, :K + 1], vcase["drafts"][:1, :K])

    for _ in range(a.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(a.steps):
        step()
    dt = time.perf_counter() - t0
    value = K * a.steps / dt
    sample = (f"each step: oracle draft(K={K}) + verify of {K + 1} logit rows on sequence 0 (batch 1) of the workload "
              f"(the repo arm's K; about 2 s of host time per step)")
    print(json.dumps({
        "impl": "reference", "metric": "draft_tokens_per_s", "value": value, "unit": "tokens/s", "n_gpus": a.gpus,
        "steps": a.steps, "warmup": a.warmup, "ms_per_step": dt / a.steps * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_name(a, s, N), "batch": 1, "draft_steps": K},
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def run_ours(a):
    import torch
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    import __graft_entry__ as G
    G.build()
    from paper_2509_18362_b200 import binding as Bd

    s, N, K, W, kv, h, tok, ids, vcase, ctx_lens = make_inputs(a, rank)
    B = a.batch
    ctx = Bd.Context(s, max_rows=max(8, B), max_K=max(8, K), max_ctx=max(ctx_lens) + K + 1)
    dW = Bd.to_device(W)
    w = Bd.mtp_w(dW)
    dkv = Bd.to_device(kv)
    ckv = Bd.kv(dkv)
    dh, dtok = Bd.bf16_tensor(h), torch.from_numpy(tok).cuda()
    dids = None if ids is None else torch.from_numpy(ids).cuda()
    dlogits, ddrafts_v = Bd.bf16_tensor(vcase["logits"]), torch.from_numpy(vcase["drafts"]).cuda()
    out_d = torch.zeros((B, K), dtype=torch.int32, device="cuda")
    acc = torch.zeros(B, dtype=torch.int32, device="cuda")
    bon = torch.zeros(B, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    # host-side buffers of the end-to-end leg (pinned)
    hh = Bd.bf16_tensor(h, "cpu").pin_memory()
    htok = torch.from_numpy(tok).pin_memory()
    hlog = Bd.bf16_tensor(vcase["logits"], "cpu").pin_memory()
    hdv = torch.from_numpy(vcase["drafts"]).pin_memory()
    hout = torch.zeros((B, K), dtype=torch.int32).pin_memory()
    hacc = torch.zeros(B, dtype=torch.int32).pin_memory()
    hbon = torch.zeros(B, dtype=torch.int32).pin_memory()

    def step_dev():
        ctx.fastmtp_draft(w, dh, dtok, ckv, B, K, dids, out_d, None, None, status)
        ctx.fastmtp_verify_accept(dlogits, ddrafts_v, B, K, s.vocab, acc, bon, None, status)

    def step_host():
        ctx.fastmtp_draft_host(w, hh, htok, ckv, B, K, dids, hout)
        ctx.fastmtp_verify_accept_host(hlog, hdv, B, K, s.vocab, hacc, hbon)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    from paper_2509_18362_b200 import replicas

    def max_over_ranks(ms):
        return replicas.max_over_ranks(ms, dist, device="cuda")

    sampler = ClockSampler(local)
    for _ in range(max(a.warmup, 3)):
        step_dev()
    barrier()
    sampler.start()
    time.sleep(0.25)
    # ---- timed region 1: inputs resident in HBM; one event pair around the whole region and one
    # around every draft call (the dominant kernel), all on the launching stream
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    kev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
           for _ in range(a.steps)]
    launches0 = ctx.launch_count
    barrier()
    t_wall0 = time.time()
    ev[0].record()
    for i in range(a.steps):
        kev[i][0].record()
        ctx.fastmtp_draft(w, dh, dtok, ckv, B, K, dids, out_d, None, None, status)
        kev[i][1].record()
        ctx.fastmtp_verify_accept(dlogits, ddrafts_v, B, K, s.vocab, acc, bon, None, status)
        kev[i][2].record()
    ev[1].record()
    barrier()
    t_wall1 = time.time()
    launches = ctx.launch_count - launches0
    clocks = sampler.stop(t_wall0, t_wall1)
    ms_total = max_over_ranks(ev[0].elapsed_time(ev[1]))
    draft_all = np.array([e0.elapsed_time(e1) for e0, e1, _ in kev])
    verify_all = np.array([e1.elapsed_time(e2) for _, e1, e2 in kev])
    draft_ms = float(np.mean(draft_all))
    assert int(status.item()) == 0, f"device status {int(status.item()):#x}"
    assert np.array_equal(acc.cpu().numpy(), vcase["length"]), "verify_accept result changed"

    # ---- timed region 2: end to end through the host-buffer entry points
    for _ in range(3):
        step_host()
    barrier()
    e2 = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    n_e2e = max(10, a.steps // 4)
    e2[0].record()
    for _ in range(n_e2e):
        step_host()
    e2[1].record()
    barrier()
    ms_e2e = max_over_ranks(e2[0].elapsed_time(e2[1]))
    assert np.array_equal(hout.numpy(), out_d.cpu().numpy()), "host and device entry points disagree"

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    ms_per_step = ms_total / a.steps
    value = replicas.job_throughput(B * K, world, a.steps, ms_total)
    e2e_value = replicas.job_throughput(B * K, world, n_e2e, ms_e2e)
    bytes_launch = sum(algorithmic_bytes_per_draft_step(s, B, N, ctx_lens, k) for k in range(K))
    peak, peak_kind = load_peaks()
    achieved = bytes_launch / (draft_ms * 1e-3) / 1e9
    # which path the draft call took: one persistent launch per group of sequences, or (more sequences than one
    # launch takes) the batched path, a sequence of tensor-core GEMM and row-wise kernels per step
    per_call = (launches / a.steps) - 1                      # kernels of one fastmtp_draft call (verify is the other one)
    kernel_name = ("mega_kernel (fastmtp_draft, K steps per launch)" if per_call <= 2 else
                   "batched path: all %d kernels of one fastmtp_draft call (skinny_gemm_kernel x %d, attn_kernel, row-wise)"
                   % (per_call, 6 * K))
    out = {
        "metric": "draft_tokens_per_s", "value": value, "unit": "tokens/s", "n_gpus": world, "steps": a.steps,
        "warmup": max(a.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16 storage, f32 accumulate", "data": "synthetic",
        "config": {"workload": workload_name(a, s, N), "batch": B, "draft_steps": K,
                   "l2": "inputs larger than L2: every step re-streams %.0f MB of weights" % (bytes_launch / K / 1e6),
                   "parallelism": "replicas" if world > 1 else "single GPU"},
        "us_per_draft_step": draft_ms * 1e3 / K,
        "gpu_launches": int(launches),
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": "tokens/s",
                "h2d_bytes_per_step": int(hh.numel() * 2 + htok.numel() * 4 + hlog.numel() * 2 + hdv.numel() * 4),
                "d2h_bytes_per_step": int(hout.numel() * 4 + hacc.numel() * 4 + hbon.numel() * 4 + 8),
                "steps": n_e2e},
        "roofline": {"bound": "hbm", "kernel": kernel_name,
                     "achieved": achieved, "peak": peak, "peak_kind": peak_kind, "unit": "GB/s",
                     "frac": achieved / peak, "frac_of_nominal_8TBs": achieved / 8000.0,
                     "algorithmic_bytes_per_launch": int(bytes_launch), "launch_ms": draft_ms,
                     "launch_ms_median": float(np.median(draft_all)), "launch_ms_min": float(draft_all.min()),
                     "launch_ms_max": float(draft_all.max()),
                     "traffic": (NCU_TRAFFIC["bytes_per_launch"]
                                 if (a.shape == "7b" and B == 1 and N == 32768 and a.ctx == 2048 and a.ctx_max == 0 and K == 3
                                     and kernel_sources_sha256() == NCU_TRAFFIC["sources_sha256"]) else None)},
    }
    # the verification kernel (a read-once scan of the [B, K+1, V] bf16 logits) timed by its own event pairs; at
    # batch 1 it moves 1.2 MB and is bound by its launch, from a few dozen sequences on by HBM
    vbytes = B * (K + 1) * s.vocab * 2
    vms = float(np.mean(verify_all))
    out["verify"] = {"kernel": "verify_kernel (fastmtp_verify_accept)", "bound": "hbm" if vbytes > (64 << 20) else "launch",
                     "algorithmic_bytes_per_launch": int(vbytes), "launch_ms": vms, "launch_ms_median": float(np.median(verify_all)),
                     "launch_ms_min": float(verify_all.min()), "achieved": vbytes / (vms * 1e-3) / 1e9, "peak": peak, "unit": "GB/s",
                     "frac": vbytes / (vms * 1e-3) / 1e9 / peak}
    if world == 1 and not a.no_cpu_baseline:
        v, cores, sample = cpu_oracle_sample(s, W, kv, h, tok, ids, vcase, K)
        out["cpu_baseline"] = {"value": v, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample}
    print(json.dumps(out))
    ctx.close()
    if dist is not None:
        dist.destroy_process_group()


def run_sweep(a):
    """Subset size {8192 .. full} (Zipf-weighted draws) x batch {1, 4, 16, 32, 64} x K {1, 3, 5} on the 7B-class head at
    context 2048: device-timed draft calls only, one JSON line per point."""
    import torch
    import __graft_entry__ as G
    G.build()
    from paper_2509_18362_b200 import binding as Bd
    from paper_2509_18362_b200 import inputs as I
    torch.cuda.set_device(0)
    s = I.QWEN7B if a.shape == "7b" else I.TINY
    W = I.mtp_weights(s, a.seed)
    dW = Bd.to_device(W)
    w = Bd.mtp_w(dW)
    peak, peak_kind = load_peaks()
    sizes = [8192, 16384, 32768, 65536, s.vocab] if a.shape == "7b" else [256, 1024, s.vocab]
    for B in (1, 4, 16, 32, 64):
        ctx_lens = [a.ctx] * B
        kv = I.paged_kv(s, ctx_lens, 6, a.seed + 1)
        dkv = Bd.to_device(kv)
        ckv = Bd.kv(dkv)
        dh = Bd.bf16_tensor(I.hidden_bf16(a.seed + 2, (B, s.d)))
        dtok = torch.from_numpy(I.token_ids(a.seed + 3, (B,), s.vocab)).cuda()
        ctx = Bd.Context(s, max_rows=max(8, B), max_K=8, max_ctx=a.ctx + 8)
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        for N in sizes:
            ids = None if N >= s.vocab else torch.from_numpy(I.subset_zipf(s.vocab, N, a.seed + 4)).cuda()
            for K in (1, 3, 5):
                out_d = torch.zeros((B, K), dtype=torch.int32, device="cuda")
                for _ in range(5):
                    ctx.fastmtp_draft(w, dh, dtok, ckv, B, K, ids, out_d, None, None, status)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                torch.cuda.synchronize()
                n = 50 if B <= 4 else 10
                e0.record()
                for _ in range(n):
                    ctx.fastmtp_draft(w, dh, dtok, ckv, B, K, ids, out_d, None, None, status)
                e1.record()
                torch.cuda.synchronize()
                ms = e0.elapsed_time(e1) / n
                nbytes = sum(algorithmic_bytes_per_draft_step(s, B, N, ctx_lens, k) for k in range(K))
                print(json.dumps({"sweep": True, "subset": N, "batch": B, "draft_steps": K, "ctx": a.ctx,
                                  "us_per_draft_step": ms * 1e3 / K, "draft_tokens_per_s": B * K / (ms * 1e-3),
                                  "mb_per_step": nbytes / K / 1e6, "gbs": nbytes / (ms * 1e-3) / 1e9,
                                  "frac_of_" + peak_kind: nbytes / (ms * 1e-3) / 1e9 / peak}), flush=True)
        assert int(status.item()) == 0
        ctx.close()


def run_target(a):
    """Device-timed fastmtp_target_step on a random target model of --target-layers layers at the
    chosen width: M = 1 (plain decode) and M = draft-steps + 1 (verification rows), batch --batch,
    --ctx cached tokens per layer. The bytes counted are every layer weight and the full output
    head once, the cached K/V of every layer, and the logits written."""
    import torch
    import __graft_entry__ as G
    G.build()
    from paper_2509_18362_b200 import binding as Bd
    from paper_2509_18362_b200 import inputs as I
    torch.cuda.set_device(0)
    nl, B = a.target_layers, a.batch
    s = (I.QWEN7B if a.shape == "7b" else I.TINY).with_layers(nl)
    Wt = I.target_weights(s, a.seed)
    dW = Bd.to_device(Wt)
    w, keep = Bd.target_w(dW)
    peak, peak_kind = load_peaks()
    qd, kvd = s.n_q_heads * s.head_dim, s.n_kv_heads * s.head_dim
    layer_w = s.d * (qd + 2 * kvd) + qd * s.d + 3 * s.d * s.ffn
    for M in (1, a.draft_steps + 1):
        kvs = [I.paged_kv(s, [a.ctx] * B, M + 1, a.seed + 10 + l, tag="tkv%d" % l) for l in range(nl)]
        dkvs = [Bd.to_device(kv) for kv in kvs]
        ckvs = [Bd.kv(k) for k in dkvs]
        ctx = Bd.Context(s, max_rows=max(8, B * M), max_K=8, max_ctx=a.ctx + M + 1)
        tok = torch.from_numpy(I.token_ids(a.seed + 3, (B, M), s.vocab)).cuda()
        out_l = torch.zeros((B, M, s.vocab), dtype=torch.bfloat16, device="cuda")
        out_a = torch.zeros((B, M), dtype=torch.int32, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        for _ in range(5):
            ctx.fastmtp_target_step(w, tok, ckvs, B, M, None, out_l, out_a, status)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        n, l0 = 30, ctx.launch_count
        e0.record()
        for _ in range(n):
            ctx.fastmtp_target_step(w, tok, ckvs, B, M, None, out_l, out_a, status)
        e1.record()
        torch.cuda.synchronize()
        assert int(status.item()) == 0, f"device status {int(status.item()):#x}"
        ms = e0.elapsed_time(e1) / n
        nbytes = 2 * (nl * layer_w + s.vocab * s.d) + nl * B * 2 * 2 * kvd * (a.ctx + M) + 2 * B * M * (s.vocab + s.d)
        print(json.dumps({"target_step": True, "layers": nl, "batch": B, "rows_per_seq": M, "ctx": a.ctx, "ms": ms,
                          "launches_per_call": (ctx.launch_count - l0) // n,
                          "us_per_layer_incl_head": ms * 1e3 / nl, "mb": nbytes / 1e6, "gbs": nbytes / (ms * 1e-3) / 1e9,
                          "frac_of_" + peak_kind: nbytes / (ms * 1e-3) / 1e9 / peak}), flush=True)
        ctx.close()


def run_e2e_loop(a):
    """Greedy and speculative decoding of one sequence through the C ABI on a random target + MTP head; checks that the
    two emit the same tokens and that the first tokens agree with the oracle (teacher-forced, near ties exempt)."""
    import torch
    import __graft_entry__ as G
    G.build()
    from paper_2509_18362_b200 import binding as Bd, inputs as I, loop
    torch.cuda.set_device(0)
    s = (I.QWEN7B if a.shape == "7b" else I.TINY).with_layers(a.loop_layers)
    P, n_new, K, n_or = a.loop_prompt, a.loop_tokens, a.draft_steps, a.loop_oracle_tokens
    N = a.subset if 0 < a.subset < s.vocab else s.vocab
    max_ctx = P + n_new + K + 3
    t0 = time.time()
    dWt, Wt = I.target_weights_cuda(s, a.seed)
    Wm = I.mtp_weights(s, a.seed + 1, embed=Wt["embed"], lm_head=Wt["lm_head"])
    prompt = [int(t) for t in I.token_ids(a.seed + 2, (P,), s.vocab)]
    ids = None if N >= s.vocab else I.subset_uniform(s.vocab, N, a.seed + 3)
    mk = lambda: [I.empty_paged_kv(s, 1, max_ctx, a.seed + 10 + l) for l in range(s.n_layers)]
    ctx = Bd.Context(s, max_rows=64, max_K=max(8, K), max_ctx=max_ctx)
    t_gen = time.time() - t0

    def timed(fn):
        torch.cuda.synchronize()
        t = time.time()
        r = fn()
        torch.cuda.synchronize()
        return r, time.time() - t

    ref, t_greedy = timed(lambda: loop.greedy_decode(loop.Target(ctx, s, dWt, [Bd.to_device(kv) for kv in mk()]), prompt, n_new + K + 1))
    dWm = dict(Bd.to_device({k: v for k, v in Wm.items() if k not in ("embed", "lm_head")}), embed=dWt["embed"], lm_head=dWt["lm_head"])
    dids = None if ids is None else torch.from_numpy(ids).cuda()

    def spec(inject):
        tgt = loop.Target(ctx, s, dWt, [Bd.to_device(kv) for kv in mk()])
        mkv = Bd.to_device(I.empty_paged_kv(s, 1, max_ctx, a.seed + 20))
        return loop.speculative_decode(tgt, Bd.mtp_w(dWm), mkv, dids, prompt, n_new, K, inject)

    def inject(rnd, K_, emitted):          # every other round: drafts right for a planted number of positions
        if rnd % 2 == 0:
            return None
        n_ok = (rnd // 2) % (K_ + 1)
        good = ref[emitted:emitted + K_]
        return list(good[:n_ok]) + [(t + 1) % s.vocab for t in good[n_ok:]]

    (out_mtp, st_mtp), t_mtp = timed(lambda: spec(None))
    (out_inj, st_inj), t_inj = timed(lambda: spec(inject))
    lossless = out_mtp == ref[:n_new] and out_inj == ref[:n_new]

    from oracle import fastmtp_oracle as O
    t0 = time.time()
    rows = list(range(P - 1, P - 1 + n_or))
    _, logits = O.target_forward_block(s, Wt, prompt + [int(t) for t in ref[:n_or - 1]], mk(), logit_rows=rows)
    t_oracle = time.time() - t0
    exempt, wrong = 0, 0
    for i, r in enumerate(rows):
        t, _ = O.argmax_token(O.round_bf16(logits[r]))
        if t != ref[i]:
            top2 = np.partition(logits[r], logits[r].shape[0] - 2)[-2:]
            ulp = 2.0 ** (np.floor(np.log2(max(abs(top2[1]), 1e-30))) - 7)
            if top2[1] - top2[0] - ulp < 1e-2:
                exempt += 1
            else:
                wrong += 1
    print(json.dumps({
        "e2e_loop": True, "layers": s.n_layers, "prompt": P, "generated": n_new, "draft_steps": K, "subset": N,
        "token_identical_to_greedy": bool(lossless),
        "greedy": {"seconds": t_greedy, "tokens_per_s": (n_new + K + 1) / t_greedy, "note": "prefill of the prompt included"},
        "speculative_mtp_drafts": {"seconds": t_mtp, "tokens_per_s": n_new / t_mtp, "tau": st_mtp["tau"],
                                   "accept_rate_by_position": st_mtp["accept_rate_by_position"], "target_calls": st_mtp["target_calls"],
                                   "note": "random weights: the head's drafts are almost never accepted"},
        "speculative_injected_drafts": {"seconds": t_inj, "tokens_per_s": n_new / t_inj, "tau": st_inj["tau"],
                                        "accept_rate_by_position": st_inj["accept_rate_by_position"],
                                        "target_calls": st_inj["target_calls"],
                                        "note": "every other round drafts right for 0..K positions in turn"},
        "oracle": {"tokens_checked": n_or, "mismatches_outside_near_ties": wrong, "near_tie_exemptions": exempt,
                   "seconds": t_oracle, "cores": os.cpu_count(), "how": "prompt + tokens teacher-forced in one layer-grouped pass"},
        "weights_seconds": t_gen, "data": "synthetic (weights drawn on the device, seeded)"}))
    ctx.close()
    if not lossless or wrong:
        raise SystemExit(1)


def main():
    a = parse_args()
    if a.e2e_loop:
        return run_e2e_loop(a)
    if a.target_layers > 0:
        return run_target(a)
    if a.sweep:
        return run_sweep(a)
    if a.impl == "reference":
        run_reference(a)
    else:
        run_ours(a)


if __name__ == "__main__":
    main()
