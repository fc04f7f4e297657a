#!/usr/bin/env python
"""Benchmark of the SAGE decode-round hot path on B200.

One step = one tree-verify round of the 16k-context video workload
(configuration 4): fused entropy + top-10 over the draft logits [60 x 152064],
entropy -> template for the next round (handed over on the device), tree-masked
attention of the 60-node tree against a 16384-token paged bf16 cache for 80
stacked layers, target argmax, greedy acceptance and KV compaction.

  python bench.py --gpus N --steps K --warmup W            CUDA path (this repo)
  python bench.py --impl reference --steps K --warmup W    the fp64 CPU oracle on the host cores

Prints ONE JSON line.  With N > 1 (torchrun) every rank runs an independent
replica of the round on its own GPU (the path has no exchange step); the time is
the max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from workloads import make_logits, make_target_logits, make_template, markov_entropy_states  # noqa: E402
from workloads.gen import _rng  # noqa: E402

CFG = 4
HQ, HKV, D, P, V = 64, 8, 128, 64, 152064
N_LAYERS, L_PREFIX, N_NODES, N_VISUAL = 80, 16384, 60, 32 * 196
K_TOP, K_ENT, MAX_PATH, ROUNDS = 10, 10, 9, 8
TEMPLATE_SHAPES = [(8, 2, N_NODES), (3, 10, N_NODES)]      # deep-narrow / shallow-wide, 60 nodes each
THRESHOLDS = [0.5]
WORKLOAD = "config4: qwen2.5-vl-72b layer shape 64/8/128 bf16, 16384-token prefix (6272 visual + 10112 text), " \
           "page 64 shuffled, 60-node tree, 80 layers, logits 60x152064 fp32"


# DRAM bytes per layer of the benchmark's attention launch (split schedule, 60-node tree) as counted by
# ncu: dram__bytes_read.sum + dram__bytes_write.sum = 615.30 MB + 3.81 MB over 9 layers
# (profiles/tree_attention_split_kernel_config4_9layers.md).  Traffic grows in proportion to the layer
# count: every layer streams its own K/V once.  Set to None whenever that kernel changes until the
# counters are taken again.
ATTN_DRAM_BYTES_PER_LAYER = 619.11e6 / 9


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def round_states():
    for tid in range(5, 30):
        states = markov_entropy_states(_rng(CFG, 50 + tid), ROUNDS, 0.8)
        if len(set(states)) == 2:
            return states
    raise RuntimeError("no chain")


def template_schedule(states, steps):
    """Template used at step i: chosen from the confidence of the previous step's draft
    logits (look-ahead); step 0 starts from alpha = 0.5 -> template 0."""
    out = []
    for i in range(steps):
        out.append(0 if i == 0 else (0 if states[(i - 1) % ROUNDS] == 0 else 1))
    return out


class ClockSampler:
    """SM clock, power and clock-event reasons of one GPU while a timed region runs: read-only NVML
    queries from a thread every ~2 ms (nvidia-smi's loop mode cannot sample a 50 ms region)."""

    def __init__(self, uuid=None, index=0):
        self.rows, self.thread, self.stop_flag, self.h, self.nv = [], None, False, None, None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            if uuid is not None:
                try:
                    self.h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + str(uuid)).encode())
                except Exception:
                    self.h = None
            if self.h is None:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.sm_max = float(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.h = None

    def _loop(self):
        nv, h = self.nv, self.h
        while not self.stop_flag:
            try:
                self.rows.append((time.time(), float(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM)),
                                  int(nv.nvmlDeviceGetCurrentClocksEventReasons(h)),
                                  nv.nvmlDeviceGetPowerUsage(h) / 1000.0))
            except Exception:
                pass
            time.sleep(0.002)

    def start(self):
        if self.h is None:
            return
        self.stop_flag = False
        self.thread = threading.Thread(target=self._loop, daemon=True)
        self.thread.start()

    def stop(self, t0, t1):
        if self.h is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["NVML unavailable"], "samples": 0}
        self.stop_flag = True
        self.thread.join()
        rows = [r for r in self.rows if t0 <= r[0] <= t1] or self.rows
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": self.sm_max, "reasons": ["no samples"], "samples": 0}
        nv = self.nv
        names = {nv.nvmlClocksEventReasonHwSlowdown: "hw_slowdown",
                 nv.nvmlClocksEventReasonHwThermalSlowdown: "hw_thermal_slowdown",
                 nv.nvmlClocksEventReasonSwThermalSlowdown: "sw_thermal_slowdown",
                 nv.nvmlClocksEventReasonSwPowerCap: "sw_power_cap"}
        reasons = sorted({name for r in rows for bit, name in names.items() if r[2] & bit})
        sm = sorted(r[1] for r in rows)
        return {"sm_mhz": sm[len(sm) // 2], "sm_min_mhz": sm[0], "sm_max_mhz": self.sm_max, "reasons": reasons,
                "samples": len(rows), "power_w_max": max(r[3] for r in rows)}


# ----------------------------------------------------------------------------------------------
# CPU oracle timing (cpu_baseline leg and --impl reference)
# ----------------------------------------------------------------------------------------------
def oracle_sample_seconds(rows_sample=6, heads_sample=1):
    """Times the oracle, as it stands, on a bounded sample of one round: the logits side on
    `rows_sample` of the 60 draft rows and as many target rows, attention of one layer for
    `heads_sample` of the 8 KV heads, acceptance and compaction of one layer.  Returns the
    seconds for that sample and the seconds of a full round extrapolated from it."""
    import oracle
    from workloads import make_kv_cache, make_q
    tree = make_template(*TEMPLATE_SHAPES[1])
    r = _rng(CFG, 900)
    lg = make_logits(r, rows_sample, V, "high")["logits"]
    kv = make_kv_cache(r, [L_PREFIX], [N_NODES], [N_VISUAL], heads_sample, shuffle=True, spare_frac=0.125)
    G = HQ // HKV
    q = make_q(r, N_NODES, heads_sample * G)[0]
    offs = np.array([0, N_NODES], np.int32)
    t0 = time.perf_counter()
    _, lse = oracle.softmax_entropy(lg)
    idx = oracle.topk(lg, K_TOP)
    oracle.topk_logprob(lg, idx, lse)
    _, alpha = oracle.confidence(lg, K_ENT)
    oracle.select_tree(alpha[:1].astype(np.float32), THRESHOLDS)
    oracle.topk(lg, 1)                                    # target argmax on as many rows
    oracle.softmax_entropy(lg)
    t_logits = time.perf_counter() - t0
    t0 = time.perf_counter()
    oracle.tree_attention(q, kv["k_pool"][0], kv["v_pool"][0], kv["page_table"], kv["seq_len"], tree["parent"], offs,
                          heads_sample * G, heads_sample, D, P, 1.0 / np.sqrt(D))
    t_attn = time.perf_counter() - t0
    t0 = time.perf_counter()
    rr = _rng(CFG, 901)
    draft = rr.integers(0, 3, N_NODES).astype(np.int32)
    target = rr.integers(0, 3, N_NODES).astype(np.int32)
    path, plen, _ = oracle.accept(tree["parent"], draft, target, offs, MAX_PATH)
    oracle.compact_kv(kv["k_pool"], kv["v_pool"], kv["page_table"], kv["seq_len"], path, plen, P)
    t_tail = time.perf_counter() - t0
    full = t_logits * (N_NODES / rows_sample) + t_attn * (HKV / heads_sample) * N_LAYERS \
        + t_tail * (HKV / heads_sample) * N_LAYERS
    return t_logits + t_attn + t_tail, full


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cores = len(os.sched_getaffinity(0))
    for _ in range(args.warmup):
        oracle_sample_seconds()
    t0 = time.perf_counter()
    fulls = []
    for _ in range(args.steps):
        _, full = oracle_sample_seconds()
        fulls.append(full)
    wall = time.perf_counter() - t0
    full = float(np.mean(fulls))
    value = 1.0 / full
    sample = "per step: logits side on 6 of 60 rows (x10), attention + compaction of 1 of 8 KV heads of 1 of 80 " \
             "layers (x640); a full round is extrapolated from the sample"
    # ms_per_step is the measured time of one sampled step (steps x ms_per_step = the timed wall clock);
    # the round the metric is quoted on is the extrapolation from it, given separately.
    line = {"impl": "reference", "metric": "tree-verify rounds/s", "value": value, "unit": "rounds/s", "n_gpus": 1,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": wall / args.steps * 1e3,
            "extrapolated_round_ms": full * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD, "l2": "n/a (CPU)"},
            "cpu_baseline": {"value": value, "unit": "rounds/s", "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "rounds/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "sample_wall_s": wall}
    print(json.dumps(line))


# ----------------------------------------------------------------------------------------------
# CUDA path
# ----------------------------------------------------------------------------------------------
def max_over_ranks(value, world, device):
    """The slowest rank's device time: every rank runs an independent replica of the round (the
    path has no exchange step), so the job's time is the maximum."""
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def run_cuda(args):
    import torch
    import torch.distributed as dist
    import paper_2602_00523_b200 as sage

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    peaks = load_peaks()
    gen = torch.Generator(device=dev)
    gen.manual_seed(523000 + 1000 * CFG + 11 + rank)

    # ---- resident state: paged K/V for 80 layers (generated on the device; perf-only data)
    tot = L_PREFIX + N_NODES
    used_pages = (tot + P - 1) // P
    n_pages = int(np.ceil(used_pages * 1.125))
    perm = _rng(CFG, 1).permutation(n_pages)[:used_pages]
    page_table = torch.from_numpy(perm.astype(np.int32)).to(dev).view(1, -1)
    k_pool = torch.empty((N_LAYERS, n_pages, HKV, P, D), dtype=torch.bfloat16, device=dev)
    v_pool = torch.empty_like(k_pool)
    vis_pages = torch.from_numpy(perm[:N_VISUAL // P].astype(np.int64)).to(dev)
    for pool in (k_pool, v_pool):
        for layer in range(N_LAYERS):
            pool[layer].normal_(generator=gen)
            pool[layer, vis_pages] *= 1.5
    seq_len0 = torch.tensor([L_PREFIX], dtype=torch.int32, device=dev)
    seq_len = seq_len0.clone()

    # ---- templates and per-round inputs
    tmpl = [make_template(*t) for t in TEMPLATE_SHAPES]
    bank_p = np.full((2, 64), -1, np.int32)
    bank_r = np.zeros((2, 64), np.int32)
    for i, t in enumerate(tmpl):
        bank_p[i, :N_NODES], bank_r[i, :N_NODES] = t["parent"], t["rank"]
    bank_parent = torch.from_numpy(bank_p).to(dev)
    bank_rank = torch.from_numpy(bank_r).to(dev)
    bank_n = torch.tensor([N_NODES, N_NODES], dtype=torch.int32, device=dev)
    policy = sage.make_policy(THRESHOLDS)
    states = round_states()
    total_steps = args.warmup + args.steps
    sched = template_schedule(states, total_steps + 1)

    node_offsets = torch.tensor([0, N_NODES], dtype=torch.int32, device=dev)
    root_token = torch.tensor([int(_rng(CFG, 6).integers(0, V))], dtype=torch.int32, device=dev)
    alpha_row = torch.zeros(1, dtype=torch.int32, device=dev)
    status = sage.new_status(dev)

    draft_host = [torch.from_numpy(make_logits(_rng(CFG, 100 + r), N_NODES, V, "low" if s == 0 else "high")["logits"])
                  .pin_memory() for r, s in enumerate(states)]
    draft_dev = [t.to(dev) for t in draft_host]
    # target logits need the draft tokens of (round, template): one untimed expansion each
    target_host, target_dev = {}, {}
    for i in range(total_steps + 1):                  # one more: the copy pipeline stages one step ahead
        key = (i % ROUNDS, sched[i])
        if key in target_host:
            continue
        t = tmpl[key[1]]
        o = sage.sage_expand_topk(draft_dev[key[0]], K_TOP, K_ENT, parent=torch.from_numpy(t["parent"]).to(dev),
                                  rank=torch.from_numpy(t["rank"]).to(dev), node_offsets=node_offsets,
                                  root_token=root_token, status=status)
        tok = o["draft_token"].cpu().numpy()
        rr = _rng(CFG, 200 + key[0] * 2 + key[1])
        leaf = int(rr.integers(N_NODES // 2, N_NODES))
        tl = make_target_logits(rr, t, tok, leaf, V)["logits"]
        target_host[key] = torch.from_numpy(tl).pin_memory()
        target_dev[key] = target_host[key].to(dev)
    q_host = torch.empty((N_LAYERS, N_NODES, HQ, D), dtype=torch.bfloat16).normal_().pin_memory()
    q_dev = q_host.to(dev)
    tree_kv_host = torch.empty((2, N_LAYERS, HKV, N_NODES, D), dtype=torch.bfloat16).normal_().pin_memory()
    tree_page = int(perm[L_PREFIX // P])
    assert L_PREFIX % P == 0 and N_NODES <= P

    # ---- preallocated outputs / workspaces (no allocation inside the timed region)
    ws_topk = torch.empty(sage.sage_expand_topk_workspace_size(N_NODES, V), dtype=torch.uint8, device=dev)
    ws_attn = torch.empty(max(16, sage.sage_tree_attention_workspace_size(N_LAYERS, 1, N_NODES, HQ, HKV, D,
                                                                          used_pages)), dtype=torch.uint8, device=dev)
    out_draft, out_target, out_accept = {}, {}, {}
    tree_buf = [{"next_parent": bank_parent[0].clone(), "next_rank": bank_rank[0].clone(),
                 "next_node_offsets": node_offsets.clone()} for _ in range(2)]
    sel_out = [dict(tb) for tb in tree_buf]
    attn_out = torch.empty_like(q_dev)
    result_host = torch.empty(MAX_PATH + 3, dtype=torch.int32).pin_memory()
    result_dev = torch.empty(MAX_PATH + 3, dtype=torch.int32, device=dev)
    attn_events = []
    other_events = {"expand_draft": [], "expand_target": [], "accept_compact": []}

    def timed_call(name, on, fn):
        if not on:
            return fn()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        r = fn()
        e1.record()
        other_events[name].append((e0, e1))
        return r

    def one_round(i, from_host, time_attn):
        r = i % ROUNDS
        cur, nxt = tree_buf[i % 2], sel_out[(i + 1) % 2]
        key = (r, sched[i])
        if from_host:
            # this step's inputs were copied from pinned host memory on the copy stream while the
            # previous step computed (two staging slots); the tree's K/V rows go from the staging
            # slot into their cache page on the device
            slot = staging[i % 2]
            torch.cuda.current_stream().wait_event(ev_copied[i % 2])
            draft, target, q = slot["draft"], slot["target"], slot["q"]
            k_pool[:, tree_page, :, :N_NODES, :].copy_(slot["tree_kv"][0])
            v_pool[:, tree_page, :, :N_NODES, :].copy_(slot["tree_kv"][1])
        else:
            draft, target, q = draft_dev[r], target_dev[key], q_dev
        d = timed_call("expand_draft", time_attn and not from_host, lambda: sage.sage_expand_topk(
            draft, K_TOP, K_ENT, parent=cur["next_parent"], rank=cur["next_rank"], node_offsets=node_offsets,
            root_token=root_token, out=out_draft, ws=ws_topk, status=status))
        sage.sage_select_tree(d["alpha"], policy, alpha_row=alpha_row, bank_parent=bank_parent, bank_rank=bank_rank,
                              bank_n_nodes=bank_n, handover=True, out=nxt, status=status)
        if time_attn:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
        sage.sage_tree_attention(q, k_pool, v_pool, page_table, seq_len, cur["next_parent"], node_offsets,
                                 1.0 / np.sqrt(D), out=attn_out, ws=ws_attn, status=status)
        if time_attn:
            e1.record()
            attn_events.append((e0, e1))
        t = timed_call("expand_target", time_attn and not from_host, lambda: sage.sage_expand_topk(
            target, 1, 1, out=out_target, ws=ws_topk, status=status))

        def tail():
            acc = sage.sage_accept(cur["next_parent"], d["draft_token"], t["topk_idx"], node_offsets, MAX_PATH,
                                   out=out_accept, status=status)
            sage.sage_compact_kv(k_pool, v_pool, page_table, seq_len, acc["path"], acc["path_len"], status=status)
            return acc
        a = timed_call("accept_compact", time_attn and not from_host, tail)
        seq_len.copy_(seq_len0)                       # the next round starts from the same prefix length
        if from_host:
            result_dev[:MAX_PATH].copy_(a["path"][0])
            result_dev[MAX_PATH:MAX_PATH + 1].copy_(a["path_len"])
            result_dev[MAX_PATH + 1:MAX_PATH + 2].copy_(a["bonus_token"])
            result_dev[MAX_PATH + 2:].copy_(nxt["template_id"])
            result_host.copy_(result_dev, non_blocking=True)
            ev_consumed[i % 2].record()               # the staging slot may be refilled from here on
        return a, nxt

    copy_stream = torch.cuda.Stream(device=dev)
    staging = [{"draft": torch.empty_like(draft_dev[0]), "target": torch.empty_like(draft_dev[0]),
                "q": torch.empty_like(q_dev), "tree_kv": torch.empty(tree_kv_host.shape, dtype=torch.bfloat16,
                                                                      device=dev)} for _ in range(2)]
    ev_copied = [torch.cuda.Event() for _ in range(2)]
    ev_consumed = [torch.cuda.Event() for _ in range(2)]

    def stage_inputs(i):
        """Host -> device copies of step i's inputs (draft and target logits, q, the tree's K/V rows),
        enqueued on the copy stream so that they overlap the previous step's kernels."""
        slot, r = staging[i % 2], i % ROUNDS
        with torch.cuda.stream(copy_stream):
            copy_stream.wait_event(ev_consumed[i % 2])        # step i-2 is done with this slot
            slot["draft"].copy_(draft_host[r], non_blocking=True)
            slot["target"].copy_(target_host[(r, sched[i])], non_blocking=True)
            slot["q"].copy_(q_host, non_blocking=True)
            slot["tree_kv"].copy_(tree_kv_host, non_blocking=True)
            ev_copied[i % 2].record(copy_stream)
    # tree buffers alternate: sel_out[j] writes into tree_buf[j]'s tensors
    for j in range(2):
        sel_out[j]["template_id"] = torch.zeros(1, dtype=torch.int32, device=dev)
        sel_out[j]["depth_cont"] = torch.zeros(1, dtype=torch.float32, device=dev)
        sel_out[j]["width_cont"] = torch.zeros(1, dtype=torch.float32, device=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(from_host):
        attn_events.clear()
        if not from_host:
            for v in other_events.values():
                v.clear()
        for j in range(2):                            # both tree buffers restart from template 0
            tree_buf[j]["next_parent"].copy_(bank_parent[0])
            tree_buf[j]["next_rank"].copy_(bank_rank[0])
        seen = []
        if from_host:
            stage_inputs(0)
        for i in range(args.warmup):
            if from_host:
                stage_inputs(i + 1)                   # the next step's copies overlap this step's kernels
            one_round(i, from_host, False)
        barrier()
        sampler = ClockSampler(getattr(torch.cuda.get_device_properties(dev), "uuid", None), local)
        sampler.start()
        t0 = time.time()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(args.warmup, total_steps):
            if from_host:
                # Every timed step issues one full set of host -> device copies (those of the step
                # after it; the first timed step's own copies ran during the last warm-up step).
                stage_inputs(i + 1)
            _, nxt = one_round(i, from_host, True)
            if from_host:
                torch.cuda.current_stream().synchronize()     # the host consumes the result every step
                seen.append(int(result_host[MAX_PATH + 2]))
        if from_host:
            torch.cuda.current_stream().wait_stream(copy_stream)      # the last staged copies end inside the timed region
        e1.record()
        barrier()
        t1 = time.time()
        clocks = sampler.stop(t0, t1)
        ms = e0.elapsed_time(e1)
        attn_ms = float(np.mean([a.elapsed_time(b) for a, b in attn_events]))
        ms = max_over_ranks(ms, world, dev)
        return ms, attn_ms, clocks, seen

    ws_cache = {"buf": ws_attn}

    def ws_for(n_layers, n_nodes_cap):
        """Attention workspace large enough for this shape (grown on demand, outside any timed region)."""
        need = sage.sage_tree_attention_workspace_size(n_layers, 1, n_nodes_cap, HQ, HKV, D, used_pages)
        if ws_cache["buf"].numel() < need:
            ws_cache["buf"] = torch.empty(need, dtype=torch.uint8, device=dev)
        return ws_cache["buf"]

    def graph_time_us(fn, passes=3):
        """GPU time of one call of fn(): its launches are captured in a CUDA graph once and replayed, so that
        the host's per-call cost (Python, ctypes, tensor views) does not sit between the kernels."""
        fn()                                          # first call outside the capture (per-device set-up, tensor maps)
        torch.cuda.synchronize()
        side = torch.cuda.Stream(device=dev)
        side.wait_stream(torch.cuda.current_stream())
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                fn()
        torch.cuda.current_stream().wait_stream(side)
        g.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(passes):
            g.replay()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e3 / passes

    def per_layer_attention_us(passes=3):
        """Attention launched layer by layer, as a model's forward does (other layers' work would sit
        in between): 80 single-layer calls walk over the 80 layers' K/V (5.5 GB), so no layer's K/V is
        still in L2 when its turn comes.  Returns the mean GPU microseconds per call (attention + merge kernel;
        the 80 calls are replayed as one CUDA graph)."""
        tree_parent = bank_parent[1, :N_NODES].contiguous()
        ws1 = torch.empty(max(16, sage.sage_tree_attention_workspace_size(1, 1, N_NODES, HQ, HKV, D, used_pages)),
                          dtype=torch.uint8, device=dev)

        def sweep():
            for layer in range(N_LAYERS):
                sage.sage_tree_attention(q_dev[layer:layer + 1], k_pool[layer:layer + 1], v_pool[layer:layer + 1],
                                         page_table, seq_len, tree_parent, node_offsets, 1.0 / np.sqrt(D),
                                         out=attn_out[layer:layer + 1], ws=ws1, status=status)
        return graph_time_us(sweep, passes) / N_LAYERS

    def attention_by_tree_size(reps=5):
        """The 80-layer attention launch alone for trees of 16 ... 60 nodes at the same 16k context
        (M = nodes x 8 query rows per KV head decides which roof binds: HBM up to about 200 rows, the
        tensor pipe above).  CUDA events around `reps` launches after two warm-up launches; every launch
        streams all layers' K/V (far larger than L2)."""
        from workloads import make_template as mk
        rows = []
        for depth, width, n in ((8, 2, 16), (8, 2, 24), (8, 2, 32), (6, 3, 36), (4, 6, 48), (3, 10, 60)):
            tp = torch.from_numpy(mk(depth, width, n)["parent"]).to(dev)
            offs = torch.tensor([0, n], dtype=torch.int32, device=dev)
            qn = q_dev[:, :n].contiguous()
            on = torch.empty_like(qn)
            wsn = ws_for(N_LAYERS, n)
            call = lambda: sage.sage_tree_attention(qn, k_pool, v_pool, page_table, seq_len, tp, offs, 1.0 / np.sqrt(D),
                                                    out=on, ws=wsn, status=status)
            call(); call()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(reps):
                call()
            e1.record()
            torch.cuda.synchronize()
            t_ms = e0.elapsed_time(e1) / reps
            T = L_PREFIX + n
            byts = (2.0 * T * HKV * D * 2 + 2.0 * n * HQ * D * 2) * N_LAYERS
            flop = 4.0 * n * (HQ // HKV) * T * D * HKV * N_LAYERS
            rows.append({"template": [depth, width, n], "rows_per_kv_head": n * (HQ // HKV), "ms_per_launch": t_ms,
                         "gbs": byts / (t_ms * 1e-3) / 1e9, "tflops": flop / (t_ms * 1e-3) / 1e12,
                         "algorithmic_bytes": byts, "flops": flop})
        return rows

    def attention_latency(passes=2):
        """Single-layer calls in the latency regime (draft-side attention, level-by-level growth, plain
        decode): contexts of 2048 and 16384 tokens, trees of 1 / 10 / 60 nodes.  Each pass walks over all
        layers' K/V, so no call finds its K/V in L2.  GPU microseconds per call (CUDA-graph replay of the 80
        calls: kernel time and the gaps between kernels, without the host's per-call cost)."""
        from workloads import chain_tree, make_template as mk
        rows = []
        for ctx in (2048, 16384):
            sl = torch.tensor([ctx], dtype=torch.int32, device=dev)
            for n, tree in ((1, chain_tree(1)), (10, mk(4, 3, 10)), (60, mk(3, 10, 60))):
                tp = torch.from_numpy(tree["parent"]).to(dev)
                offs = torch.tensor([0, n], dtype=torch.int32, device=dev)
                qs = [q_dev[layer:layer + 1, :n].contiguous() for layer in range(N_LAYERS)]
                on = torch.empty_like(qs[0])
                wsn = ws_for(1, n)

                def sweep():
                    for layer in range(N_LAYERS):
                        sage.sage_tree_attention(qs[layer], k_pool[layer:layer + 1], v_pool[layer:layer + 1], page_table, sl,
                                                 tp, offs, 1.0 / np.sqrt(D), out=on, ws=wsn, status=status)
                rows.append({"context": ctx, "nodes": n, "us_per_call": graph_time_us(sweep, passes) / N_LAYERS})
        return rows

    def policy_comparison(rounds=12, p_acc=0.8, gamma=0.9):
        """Algorithm 1 as a device-side loop (no host round trip between rounds) under a synthetic acceptance
        process (level l of the greedy path agrees with probability p * gamma^(l-1); lower-ranked candidates
        geometrically less often), for four tree policies on this workload's shapes: SD-Chain, a static
        SD-Tree, entropy-selected templates (look-ahead) and trees grown level by level with the depth
        steered by the acceptance history.  Rounds/s and accepted tokens/s; the stand-in target's few
        torch indexing kernels per round are inside the timing."""
        from paper_2602_00523_b200.decode_loop import DecodeLoop, SyntheticTarget
        from workloads import TEMPLATES, acceptance_picks, chain_tree, make_loop_logits
        cap = sage.SAGE_MAX_NODES
        grow = cap + (rounds + 3) * MAX_PATH
        pages_loop = (L_PREFIX + grow + P - 1) // P
        assert pages_loop <= n_pages
        pt_loop = torch.from_numpy(_rng(CFG, 1).permutation(n_pages)[:pages_loop].astype(np.int32)).to(dev).view(1, -1)
        rr = _rng(CFG, 700)
        # draft distributions with a clear first choice and plausible alternatives, sharper or flatter per round
        draft = [torch.from_numpy(make_loop_logits(rr, cap, V, kd)).to(dev) for kd in ("steps:9.5", "low", "steps:8", "steps:10.5")]
        picks = acceptance_picks(rr, 64, cap, 8, K_TOP, p_acc, gamma)
        noise = torch.empty((cap, V), dtype=torch.float32, device=dev).normal_(generator=gen)
        q64 = torch.empty((N_LAYERS, cap, HQ, D), dtype=torch.bfloat16, device=dev).normal_(generator=gen)
        specs = [("sd_chain_depth8", "chain", dict(trees=[chain_tree(9)])),
                 ("sd_tree_static_4x6", "static", dict(trees=[make_template(4, 6, N_NODES)])),
                 ("sage_templates", "templates", dict(trees=[make_template(d_, w_, N_NODES) for d_, w_, _ in TEMPLATES],
                                                      thresholds=[0.8, 0.4, 0.1])),
                 ("sage_dynamic_history", "dynamic", dict())]
        rows = []
        for name, pol, kw in specs:
            loop = DecodeLoop(policy=pol, draft_logits=draft, target=SyntheticTarget(noise, picks, K_TOP), k=K_TOP,
                              k_entropy=K_ENT, q=q64, k_pool=k_pool, v_pool=v_pool, page_table=pt_loop, prefix_len=L_PREFIX,
                              max_path=MAX_PATH, n_budget=N_NODES, rounds_capacity=rounds + 3, **kw)
            loop.run(3)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            loop.run(rounds)
            e1.record()
            torch.cuda.synchronize()
            if int(loop.status.item()) != 0:
                raise RuntimeError("device status in the policy loop: " + sage.status_string(int(loop.status.item())))
            t_ms = e0.elapsed_time(e1)
            plen = loop.rec["path_len"][3:3 + rounds].float()
            rows.append({"policy": name, "rounds_per_s": rounds / (t_ms * 1e-3), "accepted_tokens_per_s": float(plen.sum()) / (t_ms * 1e-3),
                         "mean_tokens_per_round": float(plen.mean()), "mean_tree_nodes": float(loop.rec["n_nodes"][3:3 + rounds].float().mean()),
                         "rounds": rounds})
        return {"acceptance_process": {"p": p_acc, "gamma": gamma}, "node_budget": N_NODES, "layers": N_LAYERS, "results": rows}

    ms, attn_ms, clocks, _ = timed(False)
    other_us = {k: (float(np.mean([a.elapsed_time(b) for a, b in v])) * 1e3 if v else None) for k, v in other_events.items()}
    layer_us = None if args.no_per_layer else per_layer_attention_us()
    by_tree = None if args.no_sweeps else attention_by_tree_size()
    latency = None if args.no_sweeps else attention_latency()
    policies = None if args.no_policies else policy_comparison()
    if int(status.item()) != 0:
        raise RuntimeError("device status: " + sage.status_string(int(status.item())))
    e2e_ms, _, _, seen = timed(True)
    expect = [sched[i + 1] for i in range(args.warmup, total_steps)]
    if seen != expect:
        raise RuntimeError(f"template sequence {seen} differs from the schedule {expect}")
    if int(status.item()) != 0:
        raise RuntimeError("device status: " + sage.status_string(int(status.item())))

    if rank == 0:
        steps = args.steps
        value = world * steps / (ms * 1e-3)
        e2e_value = world * steps / (e2e_ms * 1e-3)
        M = N_NODES * (HQ // HKV)
        flops = 4.0 * M * tot * D * HKV * N_LAYERS
        kv_bytes = 2.0 * tot * HKV * D * 2 * N_LAYERS + 2.0 * N_NODES * HQ * D * 2 * N_LAYERS
        ach_tf = flops / (attn_ms * 1e-3) / 1e12
        ach_gb = kv_bytes / (attn_ms * 1e-3) / 1e9
        h2d = draft_host[0].numel() * 4 * 2 + q_host.numel() * 2 + tree_kv_host.numel() * 2
        if args.no_cpu_baseline:
            cpu_baseline = None
        else:
            sample_s, full_s = oracle_sample_seconds(rows_sample=N_NODES, heads_sample=HKV)
            cpu_baseline = {"value": 1.0 / full_s, "unit": "rounds/s", "cores": len(os.sched_getaffinity(0)),
                            "kind": "oracle",
                            "sample": f"{sample_s:.1f} s of oracle work: the whole logits side (60 draft + 60 target "
                                      f"rows), attention, acceptance and compaction of 1 of the {N_LAYERS} layers; "
                                      "the other layers are extrapolated"}
        # expand (3), select + hand-over (2), attention (5: the library starts the kernels for trees of one row
        # tile (+ merge), two row tiles (+ merge) and more, and the tree size found on the device leaves the last
        # one running; at this shape it has one context slice per CTA, so no merge of its own), target top-1 (2),
        # accept (1), compact + advance (2).  With --layers below 9 the launch is short and only one kernel starts.
        launches = 3 + 2 + 5 + 2 + 1 + 2
        # Which tensor peak applies: the burst figure when the SM clock stayed at its maximum through the
        # timed region, the sustained one when the power cap pulled it down.  Both fractions are printed.
        sm, sm_max = clocks.get("sm_mhz"), clocks.get("sm_max_mhz")
        burst = bool(sm and sm_max and sm >= 0.97 * sm_max and "sw_power_cap" not in clocks.get("reasons", []))
        peak_tf = peaks["bf16_tflops"] if burst else peaks["bf16_tflops_sustained"]
        hbm_entry = None
        if by_tree is not None:
            for row in by_tree:
                row["frac_hbm"] = row["gbs"] / peaks["hbm_gbs"]
                row["frac_bf16_burst"] = row["tflops"] / peaks["bf16_tflops"]
                row["bound"] = "hbm" if row["rows_per_kv_head"] * 1.0 < peaks["bf16_tflops"] * 1e3 / peaks["hbm_gbs"] else "tensor"
            r24 = by_tree[1]
            hbm_entry = {"kernel": f"tree_attention, 24-node (8,2) tree, {N_LAYERS} stacked layers, 16k context",
                         "bound": "hbm", "achieved": r24["gbs"], "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": r24["frac_hbm"], "traffic": None, "ms_per_launch": r24["ms_per_launch"],
                         "algorithmic_bytes": r24["algorithmic_bytes"], "target_frac": 0.70,
                         "target_met": bool(r24["frac_hbm"] >= 0.70), "peak_source": peaks["source"] + " (copy bandwidth)",
                         "one_row_tile": {"kernel": f"tree_attention, 16-node (8,2) tree (128 query rows per KV head), "
                                                    f"{N_LAYERS} stacked layers, 16k context",
                                          "achieved": by_tree[0]["gbs"], "frac": by_tree[0]["frac_hbm"],
                                          "ms_per_launch": by_tree[0]["ms_per_launch"],
                                          "target_met": bool(by_tree[0]["frac_hbm"] >= 0.70)}}
        logits_bytes = float(N_NODES) * V * 4
        line = {
            "metric": "tree-verify rounds/s", "value": value, "unit": "rounds/s", "n_gpus": world, "steps": steps,
            "warmup": args.warmup, "ms_per_step": ms / steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": WORKLOAD, "parallelism": f"replicas x{world}",
                       "l2": f"inputs larger than L2: {kv_bytes / 1e9:.2f} GB of K/V streamed per step"},
            "e2e": {"value": e2e_value, "unit": "rounds/s", "h2d_bytes_per_step": int(h2d),
                    "d2h_bytes_per_step": int(result_host.numel() * 4), "ms_per_step": e2e_ms / steps,
                    "pipeline": "the inputs of step i+1 are copied from pinned host memory on a second stream "
                                "while step i computes (two staging slots); the host reads every step's result"},
            "gpu_launches": launches * steps,
            "clocks": clocks,
            "roofline": {"kernel": f"tree_attention, 60-node tree ({N_LAYERS} stacked layers per launch)", "bound": "tensor",
                         "achieved": ach_tf, "peak": peak_tf, "unit": "TFLOP/s", "frac": ach_tf / peak_tf,
                         "frac_of_burst_peak": ach_tf / peaks["bf16_tflops"],
                         "frac_of_sustained_peak": ach_tf / peaks["bf16_tflops_sustained"],
                         "peak_regime": "burst (SM clock at maximum during the timed region)" if burst else
                                        "sustained (SM clock below maximum / power cap active during the timed region)",
                         "ms_x_sm_mhz": None if not sm else attn_ms * sm,
                         "traffic": None if ATTN_DRAM_BYTES_PER_LAYER is None else ATTN_DRAM_BYTES_PER_LAYER * N_LAYERS,
                         "traffic_unit": "bytes per launch (ncu DRAM read+write on a 9-layer capture, scaled by layers)",
                         "algorithmic_bytes": kv_bytes,
                         "peak_source": peaks["source"], "ms_per_launch": attn_ms,
                         "hbm": {"achieved": ach_gb, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                 "frac": ach_gb / peaks["hbm_gbs"],
                                 "note": "480 query rows per KV head: above the ridge, the tensor roof binds; the "
                                         "70 % HBM target applies to the HBM-bound trees (roofline_hbm_bound)"}},
            "roofline_hbm_bound": hbm_entry,
            "attention_by_tree_size": by_tree,
            "attention_latency": latency,
            "policies": policies,
            "other_launches": {
                "expand_topk_draft_k10": None if not other_us["expand_draft"] else {
                    "us": other_us["expand_draft"], "gbs": logits_bytes / (other_us["expand_draft"] * 1e-6) / 1e9,
                    "frac_hbm": logits_bytes / (other_us["expand_draft"] * 1e-6) / 1e9 / peaks["hbm_gbs"],
                    "algorithmic_bytes": logits_bytes, "launches": 3},
                "expand_topk_target_k1": None if not other_us["expand_target"] else {
                    "us": other_us["expand_target"], "gbs": logits_bytes / (other_us["expand_target"] * 1e-6) / 1e9,
                    "frac_hbm": logits_bytes / (other_us["expand_target"] * 1e-6) / 1e9 / peaks["hbm_gbs"],
                    "algorithmic_bytes": logits_bytes, "launches": 2},
                "accept_compact": None if not other_us["accept_compact"] else {
                    "us": other_us["accept_compact"], "launches": 3,
                    "note": f"{N_LAYERS} layers; at most 9 rows x 8 heads x 256 B x 2 pools moved per layer: latency-bound"}},
            "attention_per_layer": None if layer_us is None else {
                "us_per_call": layer_us, "tflops": flops / N_LAYERS / (layer_us * 1e-6) / 1e12,
                "gbs": kv_bytes / N_LAYERS / (layer_us * 1e-6) / 1e9,
                "note": "80 single-layer calls walking over all layers' K/V (attention + merge kernels), replayed as "
                        "one CUDA graph"},
            "cpu_baseline": cpu_baseline,
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    global N_LAYERS, WORKLOAD
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--layers", type=int, default=N_LAYERS,
                    help="stacked layers per round (the workload has 80; fewer only for small profiler captures)")
    ap.add_argument("--no-per-layer", action="store_true",
                    help="skip the layer-by-layer attention timing (profiler launch lists of the round alone)")
    ap.add_argument("--no-sweeps", action="store_true",
                    help="skip the tree-size sweep and the latency sweep of the attention call")
    ap.add_argument("--no-policies", action="store_true",
                    help="skip the device-side decode loop under the four tree policies")
    ap.add_argument("--no-cpu-baseline", action="store_true",
                    help="skip timing the CPU oracle (profiler captures)")
    args = ap.parse_args()
    if args.layers != N_LAYERS:
        WORKLOAD = WORKLOAD.replace(f"{N_LAYERS} layers", f"{args.layers} layers (reduced: not the benchmark workload)")
        N_LAYERS = args.layers
    if args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
