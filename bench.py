#!/usr/bin/env python
"""Benchmark of the KV restore/save hot path on B200.

One *step* = one pass of the whole path over one batch: for every layer, build the
I/O contexts on the GPU and restore the prefix KV from the object store into the paged
pool; then, for every layer, build and save it back; then poll every completion.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

N > 1 (under torchrun) runs N independent replicas, one per GPU, with no data-path
collective (the path does not shard: "replicas only"); the time is the max over ranks.
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

import numpy as np

GIB = 1 << 30
METRIC = ("per-layer KV restore+save payload GB/s (HBM object store <-> paged pool), descriptor "
          "build included; restore_gbs / restore_hbm_frac / blocks_per_s: the restore direction")
NOMINAL_HBM_GBS = 7700.0          # HBM3e datasheet figure of the HGX B200 (context, not a ceiling)
STREAM_STORE = 0x100
STREAM_POOL = 0x200


# ----------------------------------------------------------------------------
# ranks
# ----------------------------------------------------------------------------
def rank_env():
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init_dist(backend: str):
    import torch.distributed as dist
    rank, local_rank, world = rank_env()
    if world > 1 and not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29511")
        dist.init_process_group(backend=backend, rank=rank, world_size=world)
    return rank, local_rank, world


def barrier(world: int):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


def max_over_ranks(x: float, world: int, device) -> float:
    """Slowest rank's value (the whole job is done when the last replica is)."""
    if world == 1:
        return x
    import torch
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(x: float, world: int, device) -> float:
    if world == 1:
        return x
    import torch
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


# ----------------------------------------------------------------------------
# clocks
# ----------------------------------------------------------------------------
class ClockSampler:
    """nvidia-smi clock / throttle-reason samples while the timed region runs."""
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
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-i", str(self.index), "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "samples": len(sm),
                "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------
# workload on the device
# ----------------------------------------------------------------------------
def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) per payload byte of one launch of
# copy_bulk_kernel on all SMs, from an ncu capture of one config-2 layer (1 GiB payload, 32,768
# entries of 32 KiB; traffic is proportional to the payload because every entry is an
# independent copy).  A constant of the kernel version it was captured on: it has to be
# re-captured on that small case whenever copy_bulk_kernel changes.
NCU_DRAM_BYTES_PER_PAYLOAD_BYTE = {"restore_copy": 1.955, "save_copy": 1.952}


def ncu_traffic(kernel: str):
    return NCU_DRAM_BYTES_PER_PAYLOAD_BYTE.get(kernel)


class Replica:
    """Config-2-shaped workload resident on one GPU, registered with the library."""

    def __init__(self, args, device_index: int, host_store: bool = False, n_layers=None,
                 hit_tokens=None, ring_depth=None, shared_prefix_frac=0.0):
        import torch
        from paper_2605_03375_b200 import tutti as T
        from paper_2605_03375_b200 import workload as wl
        self.torch, self.T, self.wl = torch, T, wl
        self.dev = torch.device("cuda", device_index)
        torch.cuda.set_device(self.dev)
        over = {}
        if getattr(args, "pool_hnd", False):
            over["pool_hnd"] = True
        for kv in getattr(args, "set", None) or []:
            k, v = kv.split("=")
            over[k] = int(v)
        if n_layers is None and getattr(args, "layers", 0):
            n_layers = args.layers
        if n_layers is not None:
            over["n_layers"] = n_layers
        if hit_tokens is not None:
            over["hit_tokens"] = hit_tokens
        if shared_prefix_frac:
            over["shared_prefix_frac"] = shared_prefix_frac
        self.w = w = wl.config(args.config, args.scale, **over)
        self.geom = T.geom_of(w)
        self.ctx = T.Context(self.geom, device_index)
        if w.pool_hnd:
            self.ctx.tutti_set_option(T.OPT_POOL_LAYOUT, T.POOL_HND)
        lo = self.lo = self.ctx.layout
        self.block_bytes = int(lo.block_bytes)
        self.payload_per_layer = w.total_tokens * 2 * int(lo.token_bytes)
        self.blocks_per_layer = len(w.block_ids)
        # object store (every layer resident)
        self.host_store = host_store
        self.store = []
        for d in range(w.n_devices):
            n = int(lo.dev_bytes)
            if host_store:
                t = torch.empty(n, dtype=torch.uint8, pin_memory=True)
                step = 1 << 28
                for o in range(0, n, step):
                    m = min(step, n - o)
                    tmp = wl.fill_u16_torch(w.seed, STREAM_STORE + d, o // 2, m // 2, self.dev)
                    t[o:o + m].copy_(tmp.view(torch.uint8))
                kind = T.STORE_HOST_PINNED
            else:
                t = torch.empty(n, dtype=torch.uint8, device=self.dev)
                wl.fill_u16_torch(w.seed, STREAM_STORE + d, 0, n // 2, self.dev, out=t)
                kind = T.STORE_HBM
            self.store.append(t)
            self.ctx.tutti_store_register(d, t.data_ptr(), n, kind)
        # pool: R resident layers; layer l uses buffer l mod R
        pool_bytes = 2 * w.n_pool_blocks * self.block_bytes
        free, _ = torch.cuda.mem_get_info(self.dev)
        fit = int((free * 0.85) // pool_bytes)
        R = args.resident_layers if args.resident_layers else w.n_layers
        self.R = max(1, min(R, fit, w.n_layers))
        self.pool = []
        for i in range(self.R):
            t = torch.empty(pool_bytes, dtype=torch.uint8, device=self.dev)
            wl.fill_u16_torch(w.seed, STREAM_POOL + i, 0, pool_bytes // 2, self.dev, out=t)
            self.pool.append(t)
        self.v_off = w.n_pool_blocks * self.block_bytes
        for l in range(w.n_layers):
            t = self.pool[l % self.R]
            self.ctx.tutti_pool_register(l, t.data_ptr(), t.data_ptr() + self.v_off,
                                         self.block_bytes, w.n_pool_blocks)
        # batch tables: pinned host copies (e2e uploads them every step) and device copies
        def host(a, dt):
            return torch.from_numpy(np.ascontiguousarray(a).astype(dt).view(np.int32)).pin_memory()
        self.tables_host = (host(w.hit_tokens, np.uint32), host(w.obj_start, np.uint32),
                            host(w.obj_slot, np.uint32), host(w.blk_start, np.uint32),
                            host(w.block_ids, np.int32))
        self.tables_dev = tuple(t.to(self.dev) for t in self.tables_host)
        self.batch = T.make_batch(*self.tables_dev)
        self.table_bytes = sum(t.numel() * 4 for t in self.tables_host)
        n_iocb_layer = max(1, -(-2 * len(w.obj_slot) // args.ioctx_per_iocb))
        depth = 1
        passes_in_flight = 2 if host_store else 1           # the duplex e2e leg polls one pass late
        while depth < 2 * passes_in_flight * w.n_layers * n_iocb_layer:
            depth *= 2
        iocb_mib = getattr(args, "iocb_mib", 0)
        if iocb_mib:
            # IOCBs cut by bytes: a layer takes ceil(entries * block_bytes / bytes) of them
            n_iocb_layer = max(1, -(-2 * len(w.block_ids) * self.block_bytes // (iocb_mib << 20)))
            depth = 1
            while depth < 2 * passes_in_flight * w.n_layers * n_iocb_layer:
                depth *= 2
        if ring_depth:
            depth = ring_depth            # a small ring: builds meet TUTTI_EAGAIN and the ring wraps
        self.ring = T.Ring(self.ctx, depth, args.ioctx_per_iocb,
                           2 * len(w.block_ids) * (2 * passes_in_flight * w.n_layers + 1),
                           2 * len(w.obj_slot))
        if iocb_mib:
            self.ring.tutti_ring_set_iocb_bytes(iocb_mib << 20)
        self.n_iocb_layer = n_iocb_layer
        self.ring_depth = depth
        self.stream = torch.cuda.Stream(self.dev)
        self.build_stream = torch.cuda.Stream(self.dev)
        self.write_stream = torch.cuda.Stream(self.dev)
        self.saved_ev = {}          # duplex mode: last save of every layer
        self.stage_build = torch.cuda.Stream(self.dev)
        self.stage_bufs = None      # staged mode: two staging buffers per direction
        self.stage_ev = {}
        # staged mode: contexts below this size stay on the zero-copy path
        self.stage_min_bytes = int(getattr(args, "stage_min_mib", 2.0) * 2**20)
        # duplex mode: each direction on a few SMs, so that both kernels are resident at once
        # (the host link, not the SM count, bounds them)
        self.duplex_sms = getattr(args, "e2e_sms", 12)
        self.duplex_save_sms = getattr(args, "e2e_save_sms", 8) or self.duplex_sms
        self.unpolled = []          # duplex mode: IOCBs of the previous pass
        # descriptors on their own stream pay off when a pass is long (the build of the next
        # direction runs beside the copy); for a short pass the event round trip between the
        # two streams costs more than it hides, and one stream lets the copy kernel start
        # behind the emit kernel as a dependent launch
        self.two_streams = (not getattr(args, "one_stream", False) and
                            self.payload_per_layer * w.n_layers >= 8 * GIB)
        G = getattr(args, "layers_per_launch", 0)
        if not G:
            # one build launch and one copy launch span the whole pass (measured on config 2:
            # 0.978 of the copy peak with one layer per launch, 1.014 with 4, 1.024 with 32;
            # for short prefixes the launches are the cost).  Every layer keeps its own IOCBs
            # and completion entries, so a layer still completes as soon as its bytes landed.
            G = w.n_layers
        G = min(G, w.n_layers, max(1, depth // (2 * n_iocb_layer)))
        self.layers_per_launch = max(1, G)
        self.epoch = 1
        if args.engine:
            self.ctx.tutti_set_option(T.OPT_COPY_ENGINE, args.engine)
        for opt, val in ((T.OPT_CTAS_PER_SM, args.ctas_per_sm), (T.OPT_BULK_WARPS, args.bulk_warps),
                         (T.OPT_BULK_STAGES, args.bulk_stages), (T.OPT_CLAIM_CHUNKS, args.claim),
                         (T.OPT_BULK_CHUNK_BYTES, getattr(args, "bulk_chunk", 0))):
            if val:
                self.ctx.tutti_set_option(opt, val)

    def close(self):
        self.torch.cuda.synchronize()
        self.ring.close()
        self.ctx.close()

    def step(self, sm_count=0, upload_tables=False, events=None, directions=(0, 1)):
        """One pass: all layers restored, all layers saved, all completions polled."""
        T, torch = self.T, self.torch
        s = self.stream
        self.epoch += 1
        self.batch.plan_epoch = self.epoch
        issued = []
        polled = 0
        sb = self.build_stream if self.two_streams else s
        with torch.cuda.stream(s):
            if upload_tables:
                for h, d in zip(self.tables_host, self.tables_dev):
                    d.copy_(h, non_blocking=True)
            if self.two_streams:
                fork = torch.cuda.Event()
                fork.record(s)
                sb.wait_event(fork)
            for op in directions:
                if events is not None:
                    ev = torch.cuda.Event(enable_timing=True)
                    ev.record(s)
                    events["pass"].append(ev)
                G = max(1, self.layers_per_launch)
                for l0 in range(0, self.w.n_layers, G):
                    # descriptors are built on their own stream, ahead of the copies; one
                    # copy launch then executes the IOCBs of G consecutive layers (each
                    # layer keeps its own IOCBs and completion entries)
                    g = min(G, self.w.n_layers - l0)
                    if events is not None:
                        ba = torch.cuda.Event(enable_timing=True)
                        bb_ = torch.cuda.Event(enable_timing=True)
                        ba.record(sb)
                    h0 = time.perf_counter()
                    rc, first, per = self.ring.tutti_build_sqes_layers(self.batch, l0, g, op, stream=sb,
                                                                       allow=(T.EAGAIN,))
                    if events is not None:
                        events["host_s"]["build"] += time.perf_counter() - h0
                        events["host_s"]["n_build"] += 1
                    if rc == T.EAGAIN:
                        # the ring is full: consume the completions of what was issued, retry
                        polled += self.poll_list(issued)
                        issued = []
                        rc, first, per = self.ring.tutti_build_sqes_layers(self.batch, l0, g, op,
                                                                           stream=sb)
                    if events is not None:
                        bb_.record(sb)
                        events["build"].append((ba, bb_, g))
                    n = g * per
                    if self.two_streams:
                        built = torch.cuda.Event()
                        built.record(sb)
                        s.wait_event(built)
                    if events is not None:
                        a = torch.cuda.Event(enable_timing=True)
                        b = torch.cuda.Event(enable_timing=True)
                        a.record(s)
                    h0 = time.perf_counter()
                    if op == T.OP_READ:
                        self.ring.tutti_kv_restore_layer(first, n, sm_count, stream=s)
                    else:
                        self.ring.tutti_kv_save_layer(first, n, sm_count, stream=s)
                    if events is not None:
                        events["host_s"]["issue"] += time.perf_counter() - h0
                        events["host_s"]["n_issue"] += 1
                        b.record(s)
                        events["copy"][op].append((a, b, min(G, self.w.n_layers - l0)))
                    issued.append((first, n))
            if events is not None:
                ev = torch.cuda.Event(enable_timing=True)
                ev.record(s)
                events["pass"].append(ev)
        return polled + self.poll_list(issued)

    def poll_list(self, issued):
        T = self.T
        total = 0
        for first, n in issued:
            rc, nbytes, err, done = self.ring.tutti_ring_poll_range(first, n, 20_000_000_000)
            if rc != T.OK or err != 0:
                raise RuntimeError(f"IOCBs {first}+{n}: poll rc {rc}, status {err}, {done} done")
            total += nbytes
        return total

    def step_duplex(self, upload_tables=False, group=2, times=None):
        """One pass with both directions of the host link busy: a group of layers is saved on
        its own stream as soon as it has been restored, while the next group is being restored.
        The READ and the WRITE descriptors of the whole pass are built with one call each; a
        copy launch executes the IOCBs of `group` consecutive layers.  Ordering is by events: a
        save waits for the restore of its layers, a restore waits for the previous pass's save
        of its layers (same objects, same pool buffers).  Completions of a pass are polled
        after the next pass has been issued, so the streams never run dry."""
        T, torch = self.T, self.torch
        sR, sW, sb = self.stream, self.write_stream, self.build_stream
        L = self.w.n_layers
        assert self.R == L, "duplex mode needs one pool buffer per layer"
        self.epoch += 1
        self.batch.plan_epoch = self.epoch
        if upload_tables:
            # the tables are read only by the build kernels, which run on this same stream:
            # stream order alone keeps the upload behind the previous pass's builds
            with torch.cuda.stream(sb):
                for h, d in zip(self.tables_host, self.tables_dev):
                    d.copy_(h, non_blocking=True)
        rc, fr, per_r = self.ring.tutti_build_sqes_layers(self.batch, 0, L, T.OP_READ, stream=sb)
        rc, fw, per_w = self.ring.tutti_build_sqes_layers(self.batch, 0, L, T.OP_WRITE, stream=sb)
        built = torch.cuda.Event()
        built.record(sb)
        sR.wait_event(built)
        sW.wait_event(built)
        if times is not None:
            for key, st in (("r0", sR), ("w0", sW)):
                ev = torch.cuda.Event(enable_timing=True)
                ev.record(st)
                times.setdefault(key, []).append(ev)
        for l0 in range(0, L, group):
            g = min(group, L - l0)
            if l0 in self.saved_ev:
                sR.wait_event(self.saved_ev[l0])
            self.ring.tutti_kv_restore_layer(fr + l0 * per_r, g * per_r, self.duplex_sms, stream=sR)
            restored = torch.cuda.Event()
            restored.record(sR)
            sW.wait_event(restored)
            self.ring.tutti_kv_save_layer(fw + l0 * per_w, g * per_w, self.duplex_save_sms, stream=sW)
            saved = torch.cuda.Event()
            saved.record(sW)
            self.saved_ev[l0] = saved
        if times is not None:
            for key, st in (("r1", sR), ("w1", sW)):
                ev = torch.cuda.Event(enable_timing=True)
                ev.record(st)
                times.setdefault(key, []).append(ev)
        total = self.poll_list(self.unpolled)
        self.unpolled = [(fr, L * per_r), (fw, L * per_w)]
        return total

    def step_staged(self, upload_tables=False, directions=(0, 1)):
        """One pass of staged transfers with both directions of the host link busy: the copy
        engines carry every layer's contexts between the pinned-host store and two pairs of
        staging buffers in HBM (tutti_stage_copy_layer: one copy per context), the kernels
        scatter staging -> pool and gather pool -> staging on all SMs in between.  Per layer:
        copy in -> restore kernel -> save kernel -> copy out; the copy-in of layer l+1 and the
        copy-out of layer l-1 run beside them on their own streams.  Completions of a pass are
        polled after the next pass has been issued.  `directions` may name one direction only."""
        T, torch = self.T, self.torch
        sK, sIn, sOut, sb = self.stream, self.build_stream, self.write_stream, self.stage_build
        L = self.w.n_layers
        do_r, do_w = T.OP_READ in directions, T.OP_WRITE in directions
        self.epoch += 1
        self.batch.plan_epoch = self.epoch
        if upload_tables:
            with torch.cuda.stream(sb):
                for h, d in zip(self.tables_host, self.tables_dev):
                    d.copy_(h, non_blocking=True)
        rc, n_ctx, n_st, need = self.ring.tutti_stage_plan(self.batch, self.stage_min_bytes,
                                                           stream=sb)         # once per batch
        self.stage_ctx_mib = need / max(n_st, 1) / 2**20
        self.stage_frac = need / self.payload_per_layer      # no shared objects in these legs
        need = max(need, 16)
        if self.stage_bufs is None or self.stage_bufs[0].numel() < need:
            self.stage_bufs = [torch.empty(need, dtype=torch.uint8, device=self.dev) for _ in range(4)]
        in_bufs, out_bufs = self.stage_bufs[:2], self.stage_bufs[2:]
        issued = []
        prev, cur = self.stage_ev, {}
        def last(kind, l):
            """Events that free the staging buffer layer l + 2 is about to use: `kind` of layer
            l of this pass, or, before layer 0, of the last two layers of the previous pass
            (either may have used that buffer, depending on the parity of L)."""
            if l >= 0:
                return [cur.get((kind, l))]
            return [prev.get((kind, L - 1)), prev.get((kind, L - 2))]
        for l in range(L):
            si, so = in_bufs[l % 2], out_bufs[l % 2]
            if do_r:
                # copy in: the staging buffer is free once the restore kernel two layers back is
                # done, and the store's bytes of this layer are final once its last copy-out
                # has landed
                for ev in last("restored", l - 2) + [prev.get(("out", l))]:
                    if ev is not None:
                        sIn.wait_event(ev)
                self.ring.tutti_stage_copy_layer(l, T.OP_READ, si.data_ptr(), need, stream=sIn)
                ev_in = torch.cuda.Event()
                ev_in.record(sIn)
                rc, fr, nr = self.ring.tutti_build_sqes_staged(self.batch, l, T.OP_READ, si.data_ptr(),
                                                               need, stream=sb)
                issued.append((fr, nr))
            if do_w:
                rc, fw, nw = self.ring.tutti_build_sqes_staged(self.batch, l, T.OP_WRITE, so.data_ptr(),
                                                               need, stream=sb)
                issued.append((fw, nw))
            built = torch.cuda.Event()
            built.record(sb)
            sK.wait_event(built)
            if do_r:
                sK.wait_event(ev_in)
                self.ring.tutti_kv_restore_layer(fr, nr, 0, stream=sK)
                ev_r = torch.cuda.Event()
                ev_r.record(sK)
                cur[("restored", l)] = ev_r
            if do_w:
                for ev in last("out", l - 2):
                    if ev is not None:
                        sK.wait_event(ev)              # the out buffer has been copied out
                self.ring.tutti_kv_save_layer(fw, nw, 0, stream=sK)
                ev_g = torch.cuda.Event()
                ev_g.record(sK)
                sOut.wait_event(ev_g)
                self.ring.tutti_stage_copy_layer(l, T.OP_WRITE, so.data_ptr(), need, stream=sOut)
                ev_o = torch.cuda.Event()
                ev_o.record(sOut)
                cur[("out", l)] = ev_o
        for key, ev in prev.items():
            cur.setdefault(key, ev)                     # a direction this pass did not run
        self.stage_ev = cur
        total = self.poll_list(self.unpolled)
        self.unpolled = issued
        return total

    def finish_staged(self):
        """Join the copy-out stream into the kernel stream and poll what is outstanding."""
        for key, ev in self.stage_ev.items():
            if ev is not None:
                self.stream.wait_event(ev)
        total = self.poll_list(self.unpolled)
        self.unpolled = []
        return total

    def finish_duplex(self):
        """Join the save stream into the restore stream and poll what is outstanding."""
        for ev in self.saved_ev.values():
            self.stream.wait_event(ev)
        total = self.poll_list(self.unpolled)
        self.unpolled = []
        return total

    def spot_check(self, n_samples=256, original=False):
        """Guard against timing a kernel that did no work: for random (token, head) rows the
        bytes in the pool must equal the bytes in the store, located with the library's own
        layout (tutti_obj_layout strides) and the host copies of the tables.  This is a
        self-check of the run, not the parity test (tests/ compare with the CPU oracle)."""
        torch = self.torch
        w, lo = self.w, self.lo
        rng = np.random.default_rng(1234)
        row = w.head_dim * w.elem_bytes
        for _ in range(n_samples):
            l = int(rng.integers(w.n_layers - self.R, w.n_layers))   # layers whose pool buffer is still theirs
            r = int(rng.integers(0, w.n_req))
            t = int(rng.integers(0, int(w.hit_tokens[r])))
            kv = int(rng.integers(0, 2))
            hd = int(rng.integers(0, w.n_kv_heads))
            slot = int(w.obj_slot[int(w.obj_start[r]) + t // w.obj_tokens])
            d = slot % w.n_devices
            so = ((slot // w.n_devices) * int(lo.stride_slot) + l * int(lo.stride_layer) +
                  kv * int(lo.stride_kv) + (t % w.obj_tokens) * int(lo.token_bytes) + hd * row)
            blk = int(w.block_ids[int(w.blk_start[r]) + t // w.block_tokens])
            tok = t % w.block_tokens
            bo = (hd * w.block_tokens + tok) * row if w.pool_hnd else tok * int(lo.token_bytes) + hd * row
            po = kv * self.v_off + blk * self.block_bytes + bo
            a = self.store[d][so:so + row].to(self.dev)
            b = self.pool[l % self.R][po:po + row]
            if not torch.equal(a, b):
                return False
            if original:
                # restore-then-save passes leave the store as it was generated
                g = self.wl.fill_u16_torch(w.seed, STREAM_STORE + d, so // 2, row // 2, self.dev)
                if not torch.equal(a, g.view(torch.uint8)):
                    return False
        return True


def cpu_baseline(rep, seconds_hint=10.0):
    """The oracle, as it stands, on the host cores: restore + save of whole layers of the
    same batch, on host copies of the same inputs.  Two figures: the plain token-by-token
    loop on one thread (the parity reference), and the same map taken a block at a time with
    the batch's blocks dealt out over every host core."""
    import oracle
    w = rep.w
    lo = rep.lo
    og = oracle.geom(1, w.n_kv_heads, w.head_dim, w.elem_bytes, w.block_tokens, w.obj_tokens,
                     w.n_devices, w.layout, w.n_slots)       # one layer's slice of the store
    ob = (w.hit_tokens, w.obj_start, w.obj_slot, w.blk_start, w.block_ids)
    layer_bytes = int(lo.stride_layer)
    if w.layout != rep.wl.LAYOUT_LAYER_MAJOR:
        raise RuntimeError("cpu_baseline expects the layer-major store of the bench workloads")
    cores = os.cpu_count() or 1

    # host copies of two layers, fetched once and used in turn (3.75 GiB each, far beyond any
    # host cache; fetching a fresh copy for every timed layer would cost more than the timing)
    host_layers = []
    for l in range(min(2, w.n_layers)):
        store = [s[l * layer_bytes:(l + 1) * layer_bytes].cpu().numpy() for s in rep.store]
        host_layers.append((store, rep.pool[l % rep.R].cpu().numpy().copy()))

    def run(move, budget):
        done_bytes, t_total, layers = 0, 0.0, 0
        while t_total < budget:
            store, pool = host_layers[layers % len(host_layers)]
            t0 = time.perf_counter()
            rc1 = move(store, pool, True)
            rc2 = move(store, pool, False)
            t_total += time.perf_counter() - t0
            assert rc1 == 0 and rc2 == 0
            done_bytes += 2 * rep.payload_per_layer
            layers += 1
        return done_bytes, t_total, layers

    def single(store, pool, to_pool):
        fn = oracle.restore_layer if to_pool else oracle.save_layer
        return fn(og, 0, ob, store, pool, 0, rep.v_off, rep.block_bytes, w.n_pool_blocks, w.pool_hnd)

    def all_cores(store, pool, to_pool):
        return oracle.move_layer_blocks_mt(og, 0, ob, store, pool, 0, rep.v_off, rep.block_bytes,
                                           w.n_pool_blocks, to_pool, cores, w.pool_hnd)

    b1, t1, n1 = run(single, seconds_hint)
    bN, tN, nN = run(all_cores, seconds_hint * 0.6)
    return {"value": round(b1 / t1 / 1e9, 3), "unit": "GB/s", "cores": 1,
            "host_cores": cores, "kind": "oracle", "seconds": round(t1 + tN, 2),
            "sample": f"restore+save of a full layer of the same batch, {n1} times over host copies "
                      f"of {len(host_layers)} layers ({b1 / GIB:.1f} GiB payload), token-by-token "
                      f"loop, single thread",
            "blocks_per_s": round(n1 * 2 * rep.blocks_per_layer / t1),
            "all_cores": {"value": round(bN / tN / 1e9, 3), "unit": "GB/s", "cores": cores,
                          "blocks_per_s": round(nN * 2 * rep.blocks_per_layer / tN),
                          "sample": f"restore+save of a full layer, {nN} times, one memcpy per "
                                    f"block and K/V half, blocks dealt out over {cores} threads"}}


# ----------------------------------------------------------------------------
# arms
# ----------------------------------------------------------------------------
def workload_name(w):
    return (f"cfg{w.name[3:]}: {w.n_layers} layers x {w.n_req} requests x "
            f"{int(w.hit_tokens.mean())} tokens, {w.n_kv_heads} KV heads x {w.head_dim} x "
            f"{ {1: 'fp8', 2: 'bf16', 4: 'fp32'}.get(w.elem_bytes, str(w.elem_bytes) + ' B') }, "
            f"block {w.block_tokens}, "
            f"objects of {w.obj_tokens} tokens, pool {w.n_pool_blocks} blocks 60% occupied")


_T0 = time.perf_counter()


def phase(name):
    """Progress note on stderr (the JSON line on stdout stays the only output there)."""
    print(f"[bench +{time.perf_counter() - _T0:6.1f}s] {name}", file=sys.stderr, flush=True)


def run_ours(args):
    import torch
    phase("start")
    rank, local_rank, world = init_dist("nccl")
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (no CPU fallback)"
    from paper_2605_03375_b200 import tutti as T
    rep = Replica(args, local_rank)
    w = rep.w
    peak, peak_kind = measured_peak()
    phase("workload resident")

    for _ in range(args.warmup):
        rep.step(sm_count=args.sm_count)
    torch.cuda.synchronize()
    k0, _ = rep.ring.tutti_ring_stats()
    sampler = ClockSampler(local_rank)
    sampler.start()
    events = {"pass": [], "build": [], "copy": {T.OP_READ: [], T.OP_WRITE: []},
              "host_s": {"build": 0.0, "n_build": 0, "issue": 0.0, "n_issue": 0}}
    barrier(world)
    torch.cuda.synchronize()
    e0 = torch.cuda.Event(enable_timing=True)
    e1 = torch.cuda.Event(enable_timing=True)
    e0.record(rep.stream)
    moved = 0
    for _ in range(args.steps):
        moved += rep.step(events=events, sm_count=args.sm_count)
    e1.record(rep.stream)
    torch.cuda.synchronize()
    barrier(world)
    clocks = sampler.stop()
    k1, _ = rep.ring.tutti_ring_stats()
    ms_total = max_over_ranks(e0.elapsed_time(e1), world, rep.dev)
    ms_step = ms_total / args.steps
    payload_step = 2 * w.n_layers * rep.payload_per_layer
    assert moved == payload_step * args.steps
    all_payload = sum_over_ranks(float(payload_step), world, rep.dev)
    value = all_payload / (ms_step * 1e-3) / 1e9

    # per-direction figures from the events inside the timed region
    def dir_stats(op):
        pairs = events["copy"][op]
        ms = [a.elapsed_time(b) / g for a, b, g in pairs]     # per layer of the launch
        passes = events["pass"]
        idx = 0 if op == T.OP_READ else 1
        pass_ms = [passes[3 * s + idx].elapsed_time(passes[3 * s + idx + 1])
                   for s in range(args.steps)]
        per_layer = statistics.mean(pass_ms) / w.n_layers
        gbs = rep.payload_per_layer / (per_layer * 1e-3) / 1e9
        return {"payload_gbs": round(gbs, 1), "hbm_traffic_gbs": round(2 * gbs, 1),
                "hbm_frac": round(2 * gbs / peak, 4), "ms_per_layer": round(per_layer, 4),
                "blocks_per_s": round(rep.blocks_per_layer / (per_layer * 1e-3)),
                "copy_kernel_ms": round(statistics.mean(ms), 4),
                "copy_kernel_ms_min": round(min(ms), 4)}
    restore, save = dir_stats(T.OP_READ), dir_stats(T.OP_WRITE)
    # descriptor build (plan once per step + emit), per layer, on the build stream
    build_ms = statistics.mean(a.elapsed_time(b) / g for a, b, g in events["build"])
    verified = rep.spot_check()
    phase("main leg timed and checked")

    out = None
    if rank == 0:
        # roofline of the dominant kernel (the restore copy kernel): algorithmic bytes per
        # launch = payload read + payload written + SGL entry and object address per block
        n_entries = 2 * rep.blocks_per_layer
        alg_bytes = 2 * rep.payload_per_layer + n_entries * 24
        achieved = alg_bytes / (restore["copy_kernel_ms"] * 1e-3) / 1e9
        traffic = ncu_traffic("restore_copy")
        out = {
            "metric": METRIC, "value": round(value, 1), "unit": "GB/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(ms_step, 3),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u8",
            "data": "synthetic (seeded bf16 N(0,1) KV bytes, seeded block tables and object map)",
            "config": {"workload": workload_name(w), "layers": w.n_layers,
                       "payload_gib_per_layer": round(rep.payload_per_layer / GIB, 3),
                       "store": "hbm, all layers resident",
                       "resident_pool_layers": rep.R,
                       "parallelism": "replicas only" if world > 1 else "1 gpu",
                       "l2": "inputs larger than L2 (each layer moves >= 2 GiB of HBM traffic)",
                       "copy_engine": args.engine or "auto",
                       "streams": "copy + descriptor-build stream, event-ordered"
                       if rep.two_streams else "one stream",
                       "layers_per_launch": rep.layers_per_launch,
                       "ioctx_per_iocb": args.ioctx_per_iocb},
            "restore_gbs": restore["payload_gbs"], "restore_hbm_frac": restore["hbm_frac"],
            "blocks_per_s": restore["blocks_per_s"],
            "restore": restore, "save": save,
            "build_ms_per_layer": round(build_ms, 4),
            # host side of the submission path: the ring indices and the SGL range of a build
            # are reserved on the CPU (O(1) per call), the rest of the call is kernel launches
            "host_us_per_build_call": round(events["host_s"]["build"] * 1e6 /
                                            max(1, events["host_s"]["n_build"]), 1),
            "host_us_per_issue_call": round(events["host_s"]["issue"] * 1e6 /
                                            max(1, events["host_s"]["n_issue"]), 1),
            "host_calls_per_step": (events["host_s"]["n_build"] + events["host_s"]["n_issue"]) //
            max(1, args.steps),
            "gpu_launches": int(k1 - k0),
            "spot_check": bool(verified),
            "clocks": clocks,
            "roofline": {"bound": "hbm", "kernel": "copy kernel, restore direction",
                         "achieved": round(achieved, 1), "peak": peak, "unit": "GB/s",
                         "frac": round(achieved / peak, 4), "peak_source": f"of {peak_kind}",
                         "peak_note": "the measured peak is another copy's achieved rate "
                                      "(torch copy_), not a ceiling: a fraction just above 1 is "
                                      "expected of a good copy",
                         "nominal_gbs": NOMINAL_HBM_GBS,
                         "frac_of_nominal": round(achieved / NOMINAL_HBM_GBS, 4),
                         "traffic": None if traffic is None else
                         round(traffic * rep.payload_per_layer)},
        }
    rep.close()
    del rep
    torch.cuda.empty_cache()
    # end-to-end leg: object store in pinned host memory, read zero-copy by the kernels
    if not args.no_e2e:
        e2e = run_e2e(args, local_rank, world)
        if rank == 0:
            out["e2e"] = e2e
        phase("e2e leg done")
    # the other configurations, the scheduler demo and the CPU oracle: one GPU, rank 0 only
    if rank == 0 and world == 1:
        if not args.no_configs:
            out["configs"] = {
                "cfg1": run_leg(leg_config1, args, local_rank),
                "cfg3": run_leg(leg_config3, args, local_rank),
                "cfg4": run_leg(leg_config4, args, local_rank),
                "cfg5": run_leg(leg_config5, args, local_rank),
                "shared_prefix": run_leg(leg_shared_prefix, args, local_rank),
                "prefix_sweep": run_leg(leg_prefix_sweep, args, local_rank),
            }
        if not args.no_sched:
            out["sched"] = {"hbm": run_leg(leg_sched_demo, args, local_rank, False),
                            "pinned_host": run_leg(leg_sched_demo, args, local_rank, True)}
        phase("config and scheduler legs done")
        if not args.no_cpu_baseline:
            a2 = argparse.Namespace(**vars(args))
            a2.resident_layers = 1
            rep = Replica(a2, local_rank, n_layers=min(4, w.n_layers))
            out["cpu_baseline"] = cpu_baseline(rep)
            rep.close()
            phase("cpu baseline done")
    if rank == 0:
        print(json.dumps(out), flush=True)
    barrier(world)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def run_leg(fn, args, local_rank, *extra):
    """One auxiliary leg with its own clock samples; a leg that fails is reported, loudly, in
    its own object instead of taking the whole line down."""
    import torch
    sampler = ClockSampler(local_rank)
    sampler.start()
    t0 = time.perf_counter()
    try:
        res = fn(args, local_rank, *extra)
    except Exception as e:                       # noqa: BLE001 - reported in the line
        import traceback
        traceback.print_exc(file=sys.stderr)
        res = {"error": f"{type(e).__name__}: {e}"[:400]}
    torch.cuda.synchronize()
    torch.cuda.empty_cache()
    res["clocks"] = sampler.stop()
    res["leg_seconds"] = round(time.perf_counter() - t0, 1)
    phase(f"{fn.__name__} done")
    return res


def timed_passes(rep, dirs, passes, sm_count=0):
    """ms per layer of `passes` passes in the given directions (after one untimed pass)."""
    import torch
    rep.step(directions=dirs, sm_count=sm_count)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(rep.stream)
    for _ in range(passes):
        rep.step(directions=dirs, sm_count=sm_count)
    e1.record(rep.stream)
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / (passes * rep.w.n_layers)


def leg_config1(args, local_rank):
    """Config 1: one layer, 8 MiB of KV (L2-resident): a latency, not a bandwidth."""
    from paper_2605_03375_b200 import tutti as T
    a2 = argparse.Namespace(**vars(args))
    a2.config, a2.scale, a2.layers, a2.resident_layers, a2.set = 1, 1.0, 0, 0, None
    a2.ioctx_per_iocb = 2048
    rep = Replica(a2, local_rank)
    out = {"config": workload_name(rep.w), "payload_mib": round(rep.payload_per_layer / (1 << 20), 1)}
    import torch
    s = rep.stream
    for name, op in (("restore", T.OP_READ), ("save", T.OP_WRITE)):
        issue = rep.ring.tutti_kv_restore_layer if op == T.OP_READ else rep.ring.tutti_kv_save_layer

        def one():
            # the three calls a user makes for one layer, nothing else around them
            rep.epoch += 1
            rep.batch.plan_epoch = rep.epoch
            rc, first, n = rep.ring.tutti_build_sqes(rep.batch, 0, op, stream=s)
            issue(first, n, 0, stream=s)
            rc, nbytes, err, done = rep.ring.tutti_ring_poll_range(first, n, 5_000_000_000)
            assert (rc, err, nbytes) == (T.OK, 0, rep.payload_per_layer)
        for _ in range(20):
            one()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(300):
            one()
        out[f"build_plus_{name}_us"] = round((time.perf_counter() - t0) / 300 * 1e6, 2)
    out["note"] = ("latency of one layer on the host clock: build call (plan + emit launches), copy "
                   "launch, completion poll; 16 MiB of traffic stays in L2, so no HBM fraction is quoted")
    out["spot_check"] = bool(rep.spot_check(64))
    rep.close()
    return out


def leg_shared_prefix(args, local_rank):
    """Requests of one batch with a common prefix (Section 3.1: a stored chunk is shared by every
    request with that prefix): the config-2 batch with the first 75 % of every request's objects
    being the same stored objects.  The descriptors name each shared object once; the copy
    kernels load it once per stage and store it to every request's blocks.  Restore only (a
    save of several requests into one object is the caller's race)."""
    import torch
    from paper_2605_03375_b200 import tutti as T
    peak, _ = measured_peak()
    out = {"batch": "config-2 shape, 8 requests x 32768 tokens, first 75 % of the objects shared"}
    for store, host, layers in (("hbm", False, 8), ("pinned_host", True, 4)):
        res = {}
        for frac in (0.75, 0.0):
            a2 = argparse.Namespace(**vars(args))
            a2.config, a2.scale, a2.set, a2.layers = 2, 1.0, None, 0
            a2.ioctx_per_iocb = 2048
            a2.layers_per_launch = 0
            a2.resident_layers = layers
            rep = Replica(a2, local_rank, host_store=host, n_layers=layers, shared_prefix_frac=frac)
            if host:
                rep.ctx.tutti_set_option(T.OPT_COPY_ENGINE, T.ENGINE_BULK)
            sm = 16 if host else 0
            ms = timed_passes(rep, (T.OP_READ,), 2 if host else 4, sm_count=sm)
            gbs = rep.payload_per_layer / (ms * 1e-3) / 1e9
            key = "shared" if frac else "private"
            res[key] = {"landed_gbs": round(gbs, 1), "ms_per_layer": round(ms, 4)}
            if frac:
                # bytes the descriptors name in the store, from the library's own contexts
                rep.epoch += 1
                rep.batch.plan_epoch = rep.epoch
                rc, first, n = rep.ring.tutti_build_sqes(rep.batch, 0, T.OP_READ, stream=rep.stream)
                named = 0
                for i in range(first, first + n):
                    info, sq = rep.ring.tutti_ring_read_iocb(i)
                    named += int(sq["len"].sum())
                rep.ring.tutti_kv_restore_layer(first, n, 0, stream=rep.stream)
                rep.poll_list([(first, n)])
                res["store_bytes_named_per_landed_byte"] = round(named / rep.payload_per_layer, 4)
                res["spot_check"] = bool(rep.spot_check(64))
            rep.close()
            del rep
            torch.cuda.empty_cache()
        res["speedup_from_sharing"] = round(res["shared"]["landed_gbs"] / res["private"]["landed_gbs"], 3)
        if not host:
            res["shared"]["pool_write_hbm_frac"] = round(res["shared"]["landed_gbs"] / peak, 4)
        res["sm_count"] = 16 if host else 0
        out[store] = res
    return out


def leg_config4(args, local_rank):
    """Config 4: 1-token pages (2 KiB fragments), 64 requests with partial hits, with 2048 and
    with 64 contexts per IOCB (the latter on a ring of 128 IOCBs that wraps every layer)."""
    from paper_2605_03375_b200 import tutti as T
    peak, _ = measured_peak()
    out = {}
    for cap, depth in ((2048, None), (64, 128)):
        a2 = argparse.Namespace(**vars(args))
        a2.config, a2.scale, a2.set = 4, 1.0, None
        a2.ioctx_per_iocb = cap
        a2.resident_layers = 2
        a2.layers_per_launch = 0
        rep = Replica(a2, local_rank, n_layers=args.cfg4_layers, ring_depth=depth)
        if "config" not in out:
            out["config"] = workload_name(rep.w).replace(f"{args.cfg4_layers} layers", "32 layers")
            out["layers_timed"] = args.cfg4_layers
            out["payload_gib_per_layer"] = round(rep.payload_per_layer / GIB, 3)
        res = {"ring_depth": rep.ring_depth, "iocbs_per_layer": rep.n_iocb_layer,
               "layers_per_launch": rep.layers_per_launch}
        for name, dirs in (("restore", (T.OP_READ,)), ("save", (T.OP_WRITE,))):
            ms = timed_passes(rep, dirs, 3)
            gbs = rep.payload_per_layer / (ms * 1e-3) / 1e9
            res[name] = {"payload_gbs": round(gbs, 1), "ms_per_layer": round(ms, 4),
                         "hbm_frac": round(2 * gbs / peak, 4),
                         "blocks_per_s": round(rep.blocks_per_layer / (ms * 1e-3))}
        res["spot_check"] = bool(rep.spot_check(64))
        out[f"ioctx_per_iocb_{cap}"] = res
        rep.close()
        del rep
        import torch
        torch.cuda.empty_cache()
    return out


def run_e2e(args, local_rank, world):
    """Same metric through the public call with the objects in HOST memory: every step
    uploads the batch tables from pinned host memory, restores every layer from the pinned
    host object store (the kernels read it zero-copy over the host link), saves every layer
    back to it, and reads the completions on the host."""
    import torch
    a2 = argparse.Namespace(**vars(args))
    L_host = min(args.e2e_host_layers, 32)
    a2.resident_layers = L_host
    a2.layers_per_launch = 4
    rep = Replica(a2, local_rank, host_store=True, n_layers=L_host)
    passes = max(1, 32 // L_host) if args.config in (2, 5) else 1
    steps = max(1, min(args.steps, 3))
    layers = L_host * passes
    payload = 2 * layers * rep.payload_per_layer
    T = rep.T

    def measure(mode):
        """ms per step of one mode: 'zero_copy' (the kernels read and write the store over the
        link), 'staged' (copy engines on the link, kernels on HBM) or 'serial'."""
        times = {}
        if mode == "zero_copy":
            rep.ctx.tutti_set_option(T.OPT_COPY_ENGINE, T.ENGINE_BULK)
            one_pass = lambda: rep.step_duplex(upload_tables=True, group=args.e2e_group, times=times)
            finish = rep.finish_duplex
        elif mode == "staged":
            rep.ctx.tutti_set_option(T.OPT_COPY_ENGINE, args.engine or T.ENGINE_AUTO)
            one_pass = lambda: rep.step_staged(upload_tables=True)
            finish = rep.finish_staged
        else:
            one_pass = lambda: rep.step(upload_tables=True)
            finish = lambda: 0
        one_pass()
        finish()
        torch.cuda.synchronize()
        times.clear()
        barrier(world)
        t0 = time.perf_counter()
        e0 = torch.cuda.Event(enable_timing=True)
        e1 = torch.cuda.Event(enable_timing=True)
        e0.record(rep.stream)
        moved = 0
        for _ in range(steps * passes):
            moved += one_pass()
        moved += finish()
        e1.record(rep.stream)
        torch.cuda.synchronize()
        wall_ms = (time.perf_counter() - t0) * 1e3
        ms = max_over_ranks(max(e0.elapsed_time(e1), wall_ms), world, rep.dev) / steps
        assert moved == payload * steps, (mode, moved, payload * steps)
        if not rep.spot_check(64, original=True):
            raise RuntimeError(f"e2e {mode}: spot check failed")
        res = {"gbs": round(sum_over_ranks(float(payload), world, rep.dev) / (ms * 1e-3) / 1e9, 2),
               "ms_per_step": round(ms, 2)}
        if mode == "staged":
            # the copy engines' rate depends on the size of a contiguous copy (here, a context)
            res["mean_copy_mib"] = round(rep.stage_ctx_mib, 2)
            res["staged_frac"] = round(rep.stage_frac, 4)
            res["stage_min_mib"] = args.stage_min_mib
        if mode == "zero_copy" and times:
            # each direction's own rate: its bytes over the time its stream was busy with them
            for key, a, b in (("restore_gbs", "r0", "r1"), ("save_gbs", "w0", "w1")):
                busy = times[a][0].elapsed_time(times[b][-1])
                res[key] = round(steps * layers * rep.payload_per_layer / (busy * 1e-3) / 1e9, 2)
        return res

    modes = {"serial": ["serial"], "zero_copy": ["zero_copy"], "staged": ["staged"],
             "both": ["zero_copy", "staged"]}["serial" if args.e2e_serial else args.e2e_mode]
    res = {m: measure(m) for m in modes}
    best = max(res, key=lambda m: res[m]["gbs"])
    link = host_link_gbs(rep.dev) if world == 1 else None
    link_duplex = host_link_duplex_gbs(rep.dev) if world == 1 else None
    h2d = layers * rep.payload_per_layer + passes * rep.table_bytes
    d2h = layers * rep.payload_per_layer + 2 * layers * 32
    if best == "staged":
        d2h += passes * 24 * len(rep.w.obj_slot)       # the batch's contexts, fetched once per pass
    describe = {
        "zero_copy": f"zero-copy duplex: the kernels read and write the pinned-host store over "
                     f"the link; groups of {args.e2e_group} layers saved while the next group is "
                     f"restored; restore on {rep.duplex_sms} SMs, save on {rep.duplex_save_sms} SMs",
        "staged": "staged duplex: copy engines move each layer's contexts between the pinned-host "
                  "store and staging buffers in HBM (one copy per context), the kernels scatter "
                  "and gather between staging and pool on all SMs; copy-in of the next layer and "
                  "copy-out of the previous one run beside them",
        "serial": "serial: all restores, then all saves"}
    out = {"value": res[best]["gbs"], "unit": "GB/s", "h2d_bytes_per_step": int(h2d),
           "d2h_bytes_per_step": int(d2h), "ms_per_step": res[best]["ms_per_step"],
           "spot_check": True,
           "host_link_duplex_gbs": None if link_duplex is None else round(link_duplex, 1),
           "link_frac": None if link_duplex is None else round(res[best]["gbs"] / link_duplex, 4),
           "mode": describe[best],
           "modes": {m: dict(r, what=describe[m]) for m, r in res.items()},
           "store": f"pinned host memory; {L_host} layers resident, "
                    f"{passes} passes per step = {layers} layer transfers each way"}
    rep.close()
    if link is not None:
        out["host_link_h2d_gbs"], out["host_link_d2h_gbs"] = round(link[0], 2), round(link[1], 2)
    return out


def host_link_gbs(dev, nbytes=1 << 30, reps=10):
    """Pinned host -> HBM copy bandwidth on this machine (cudaMemcpyAsync, best of `reps`)."""
    import torch
    src = torch.empty(nbytes, dtype=torch.uint8, pin_memory=True)
    dst = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    best = 0.0
    for _ in range(reps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        dst.copy_(src, non_blocking=True)
        b.record()
        torch.cuda.synchronize()
        best = max(best, nbytes / (a.elapsed_time(b) * 1e-3) / 1e9)
    h2d = best
    best = 0.0
    for _ in range(reps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        src.copy_(dst, non_blocking=True)
        b.record()
        torch.cuda.synchronize()
        best = max(best, nbytes / (a.elapsed_time(b) * 1e-3) / 1e9)
    return h2d, best


def host_link_duplex_gbs(dev, nbytes=1 << 30, reps=5):
    """Both directions of the host link at once with the copy engines (two streams): the sum
    of pinned->HBM and HBM->pinned bytes over the time both took."""
    import torch
    a_h = torch.empty(nbytes, dtype=torch.uint8, pin_memory=True)
    b_h = torch.empty(nbytes, dtype=torch.uint8, pin_memory=True)
    a_d = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    b_d = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    s1, s2 = torch.cuda.Stream(dev), torch.cuda.Stream(dev)
    best = 0.0
    for _ in range(reps):
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        with torch.cuda.stream(s1):
            a_d.copy_(a_h, non_blocking=True)
        with torch.cuda.stream(s2):
            b_h.copy_(b_d, non_blocking=True)
        torch.cuda.synchronize()
        best = max(best, 2 * nbytes / (time.perf_counter() - t0) / 1e9)
    return best


def leg_config3(args, local_rank):
    """Config 3: Llama-3-70B-shaped KV restored per layer from the pinned-host object store,
    zero-copy.  80 layer transfers per step over a window of resident host layers."""
    import torch
    from paper_2605_03375_b200 import tutti as T
    a2 = argparse.Namespace(**vars(args))
    a2.config, a2.scale, a2.set, a2.layers = 3, 1.0, None, 0
    a2.ioctx_per_iocb = 2048
    a2.layers_per_launch = 4
    a2.resident_layers = 2
    L_host = args.e2e_host_layers
    rep = Replica(a2, local_rank, host_store=True, n_layers=L_host)
    peak, peak_kind = measured_peak()
    h2d, d2h = host_link_gbs(rep.dev)
    passes = max(1, 80 // L_host)
    out = {"config": workload_name(rep.w).replace(f"{L_host} layers", "80 layers"),
           "host_layers_resident": L_host, "host_link_h2d_gbs": round(h2d, 2),
           "host_link_d2h_gbs": round(d2h, 2)}
    for name, dirs in (("restore", (T.OP_READ,)), ("save", (T.OP_WRITE,))):
        for eng in (1, 2):
            rep.ctx.tutti_set_option(T.OPT_COPY_ENGINE, eng)
            rep.step(directions=dirs)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(rep.stream)
            for _ in range(passes):
                rep.step(directions=dirs)
            e1.record(rep.stream)
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / (passes * L_host)
            gbs = rep.payload_per_layer / (ms * 1e-3) / 1e9
            link = h2d if name == "restore" else d2h
            out[f"{name}_engine{eng}"] = {
                "payload_gbs": round(gbs, 2), "ms_per_layer": round(ms, 3),
                "link_frac": round(gbs / link, 4), "hbm_frac": round(gbs / peak, 5),
                "blocks_per_s": round(rep.blocks_per_layer / (ms * 1e-3))}
    # the same transfers staged: copy engines on the link, kernels between staging and pool
    rep.ctx.tutti_set_option(T.OPT_COPY_ENGINE, T.ENGINE_AUTO)
    for name, dirs in (("restore", (T.OP_READ,)), ("save", (T.OP_WRITE,))):
        rep.step_staged(directions=dirs)
        rep.finish_staged()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(rep.stream)
        for _ in range(passes):
            rep.step_staged(directions=dirs)
        rep.finish_staged()
        e1.record(rep.stream)
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / (passes * L_host)
        gbs = rep.payload_per_layer / (ms * 1e-3) / 1e9
        link = h2d if name == "restore" else d2h
        out[f"{name}_staged"] = {"payload_gbs": round(gbs, 2), "ms_per_layer": round(ms, 3),
                                 "link_frac": round(gbs / link, 4),
                                 "mean_copy_mib": round(rep.stage_ctx_mib, 2)}
    out["spot_check"] = bool(rep.spot_check())
    rep.close()
    return out


def leg_config5(args, local_rank):
    """Config 5: config 2's restore as persistent CTAs capped at 8/16/32 SMs while a bf16
    8192^3 GEMM runs on the remaining SMs (green-context partition when the driver allows)."""
    import torch
    from paper_2605_03375_b200 import tutti as T
    a2 = argparse.Namespace(**vars(args))
    a2.config, a2.scale, a2.set, a2.layers = 2, 1.0, None, 0
    a2.ioctx_per_iocb = 2048
    a2.layers_per_launch = 4
    a2.resident_layers = 8
    rep = Replica(a2, local_rank, n_layers=args.cfg5_layers)
    dev = rep.dev
    peak, _ = measured_peak()
    n = 8192
    A = torch.randn(n, n, device=dev, dtype=torch.bfloat16)
    B = torch.randn(n, n, device=dev, dtype=torch.bfloat16)
    Cm = torch.empty(n, n, device=dev, dtype=torch.bfloat16)
    gemm_iters = args.gemm_iters

    def time_gemm(stream, iters):
        with torch.cuda.stream(stream):
            for _ in range(3):
                torch.matmul(A, B, out=Cm)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for _ in range(iters):
                torch.matmul(A, B, out=Cm)
            b.record(stream)
        return a, b

    def restore_pass(stream, sm_count, events):
        rep.stream = stream
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        rep.step(sm_count=sm_count, directions=(T.OP_READ,))
        b.record(stream)
        events.append((a, b))

    main = torch.cuda.Stream(dev)
    a, b = time_gemm(main, gemm_iters)
    torch.cuda.synchronize()
    gemm_alone_ms = a.elapsed_time(b) / gemm_iters
    ev = []
    restore_pass(main, 0, ev)
    restore_pass(main, 0, ev)
    torch.cuda.synchronize()
    full_ms = ev[-1][0].elapsed_time(ev[-1][1]) / rep.w.n_layers
    out = {"config": "cfg5: " + workload_name(rep.w) + "; bf16 GEMM 8192^3 beside it",
           "gemm_alone_ms": round(gemm_alone_ms, 4),
           "gemm_alone_tflops": round(2 * n ** 3 / (gemm_alone_ms * 1e-3) / 1e12, 1),
           "restore_all_sms": {"ms_per_layer": round(full_ms, 4),
                               "payload_gbs": round(rep.payload_per_layer / (full_ms * 1e-3) / 1e9, 1)},
           "capped": []}
    for io_sms in (8, 16, 32):
        entry = {"sm_count": io_sms}
        try:
            io_s, comp_s, got_io, got_comp = rep.ctx.tutti_sm_partition_create(io_sms)
            io_stream = torch.cuda.ExternalStream(io_s, device=dev)
            comp_stream = torch.cuda.ExternalStream(comp_s, device=dev)
            entry["partition"] = {"kind": "green contexts", "io_sms": got_io, "compute_sms": got_comp}
            partition = True
        except T.TuttiError as e:
            io_stream, comp_stream = torch.cuda.Stream(dev), torch.cuda.Stream(dev)
            got_io = io_sms
            entry["partition"] = {"kind": "plain streams (no isolation)", "why": str(e)[:200]}
            partition = False
        # each alone inside its partition
        a, b = time_gemm(comp_stream, gemm_iters)
        torch.cuda.synchronize()
        entry["gemm_alone_in_partition_ms"] = round(a.elapsed_time(b) / gemm_iters, 4)
        ev = []
        restore_pass(io_stream, got_io, ev)
        restore_pass(io_stream, got_io, ev)
        torch.cuda.synchronize()
        alone_ms = ev[-1][0].elapsed_time(ev[-1][1]) / rep.w.n_layers
        entry["restore_alone_capped"] = {
            "ms_per_layer": round(alone_ms, 4),
            "payload_gbs": round(rep.payload_per_layer / (alone_ms * 1e-3) / 1e9, 1)}
        # together: GEMMs keep running for the whole restore pass
        n_gemm = max(8, int(1.5 * alone_ms * rep.w.n_layers / entry["gemm_alone_in_partition_ms"]))
        torch.cuda.synchronize()
        ga, gb = time_gemm(comp_stream, n_gemm)
        ev = []
        restore_pass(io_stream, got_io, ev)
        torch.cuda.synchronize()
        both_ms = ev[-1][0].elapsed_time(ev[-1][1]) / rep.w.n_layers
        gemm_ms = ga.elapsed_time(gb) / n_gemm
        gbs = rep.payload_per_layer / (both_ms * 1e-3) / 1e9
        entry["concurrent"] = {
            "restore_ms_per_layer": round(both_ms, 4), "restore_payload_gbs": round(gbs, 1),
            "restore_hbm_frac": round(2 * gbs / peak, 4),
            "gemm_ms": round(gemm_ms, 4), "gemms_overlapped": n_gemm,
            "gemm_slowdown_vs_all_sms": round(gemm_ms / gemm_alone_ms, 3),
            "gemm_slowdown_vs_partition": round(gemm_ms / entry["gemm_alone_in_partition_ms"], 3),
            "restore_slowdown_vs_capped_alone": round(both_ms / alone_ms, 3)}
        entry["spot_check"] = bool(rep.spot_check(64))
        if partition:
            rep.ctx.tutti_sm_partition_destroy()
        out["capped"].append(entry)
    rep.stream = main
    rep.close()
    return out


def leg_sched_demo(args, local_rank, sched_host):
    """Layer-wise pipelining under the slack-aware scheduler (Section 3.3), with GEMMs standing
    in for a layer's compute: restores of the next layers are sized from the profiled tables
    and issued on the I/O partition while the current layer computes on the other SMs.
    IOCBs are cut by bytes (equal work), the I/O table is filled by the library's own
    profiling pass, and the table's estimate is checked against launches it did not time."""
    import torch
    from paper_2605_03375_b200 import tutti as T
    a2 = argparse.Namespace(**vars(args))
    a2.config, a2.scale, a2.set = 2, 1.0, None
    a2.ioctx_per_iocb = 2048
    a2.one_stream = True
    a2.layers_per_launch = 1
    a2.resident_layers = 8
    n_layers = (args.layers or 6) if sched_host else (args.layers or 32)
    rep = Replica(a2, local_rank, host_store=sched_host, n_layers=n_layers, ring_depth=2048)
    if sched_host:
        # objects in pinned host memory: the restore is bound by the host link, so a few
        # SMs carry it while the rest of the GPU computes
        rep.ctx.tutti_set_option(T.OPT_COPY_ENGINE, T.ENGINE_BULK)
    iocb_bytes = args.sched_iocb_mib << 20
    rep.ring.tutti_ring_set_iocb_bytes(iocb_bytes)
    w, dev = rep.w, rep.dev
    io_sms = 8 if sched_host else args.sched_sms
    io_s, comp_s, got_io, got_comp = rep.ctx.tutti_sm_partition_create(io_sms)
    io_stream = torch.cuda.ExternalStream(io_s, device=dev)
    comp_stream = torch.cuda.ExternalStream(comp_s, device=dev)
    n = 8192
    A = torch.randn(n, n, device=dev, dtype=torch.bfloat16)
    B = torch.randn(n, n, device=dev, dtype=torch.bfloat16)
    Cm = torch.empty(n, n, device=dev, dtype=torch.bfloat16)

    def timed(fn, stream):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record(stream)
        fn()
        b.record(stream)
        torch.cuda.synchronize()
        return a.elapsed_time(b)

    def build_all(stream):
        rep.epoch += 1
        rep.batch.plan_epoch = rep.epoch
        rc, first, per = rep.ring.tutti_build_sqes_layers(rep.batch, 0, w.n_layers, T.OP_READ,
                                                          stream=stream)
        return [(first + l * per, per) for l in range(w.n_layers)]

    def poll(built):
        rep.poll_list(built)

    # warm-up profiling inside the library: restore time against the IOCB count on the I/O
    # partition (1, 2, 4, ... and all IOCBs of a layer)
    sched = T.Scheduler(w.n_layers, 32, 65536, 65536)
    rep.epoch += 1
    rep.batch.plan_epoch = rep.epoch
    n_points = sched.tutti_sched_profile(rep.ring, rep.batch, 0, T.OP_READ, [got_io], reps=2,
                                         stream=io_stream)
    built = build_all(io_stream)
    torch.cuda.synchronize()
    used = sum(1 for i in range(built[0][0], built[0][0] + built[0][1])
               if rep.ring.tutti_ring_read_iocb(i)[0].num_ioctx > 0)
    for first, cnt in built:
        rep.ring.tutti_kv_restore_layer(first, cnt, got_io, stream=io_stream)
    poll(built)
    profile = {k: round(sched.tutti_sched_io_time(T.OP_READ, got_io, k), 1)
               for k in sorted({1, 2, 4, 8, used})}
    # the write kernel is profiled the same way (Section 3.3 profiles both)
    n_points += sched.tutti_sched_profile(rep.ring, rep.batch, 0, T.OP_WRITE, [got_io], reps=1,
                                          stream=io_stream)
    profile_w = {k: round(sched.tutti_sched_io_time(T.OP_WRITE, got_io, k), 1)
                 for k in sorted({1, used})}
    # the table against launches it has not seen: IOCB counts between the profiled points
    est_err = {}
    for k in sorted({3, 5, max(1, used - 3)}):
        if k >= used:
            continue
        built = build_all(io_stream)
        first = built[0][0]
        ms = timed(lambda: rep.ring.tutti_kv_restore_layer(first, k, got_io, stream=io_stream),
                   io_stream)
        rep.ring.tutti_kv_restore_layer(first + k, built[0][1] - k, got_io, stream=io_stream)
        for f, c in built[1:]:
            rep.ring.tutti_kv_restore_layer(f, c, got_io, stream=io_stream)
        poll(built)
        est = sched.tutti_sched_io_time(T.OP_READ, got_io, k)
        est_err[k] = {"measured_us": round(ms * 1e3, 1), "estimated_us": round(est, 1),
                      "error": round(abs(est - ms * 1e3) / (ms * 1e3), 4)}
    layer_restore_ms = profile[used] / 1e3
    # the layer's window: its compute time on the compute partition.  From HBM a layer's KV
    # arrives in a fraction of a 3-GEMM layer; from pinned host memory the link needs ~20 ms
    # per GiB layer, so the stand-in layer is made that long (a long prefill chunk)
    with torch.cuda.stream(comp_stream):
        torch.matmul(A, B, out=Cm)
        gemm_ms = timed(lambda: [torch.matmul(A, B, out=Cm) for _ in range(4)], comp_stream) / 4
    gemms_per_layer = args.sched_gemms
    if sched_host:
        gemms_per_layer = max(gemms_per_layer, int(1.15 * layer_restore_ms / gemm_ms) + 1)

    def layer_compute():
        for _ in range(gemms_per_layer):
            torch.matmul(A, B, out=Cm)
    with torch.cuda.stream(comp_stream):
        layer_ms = timed(layer_compute, comp_stream)
    l_in, l_pre = 8192, 32768
    sched.tutti_sched_set_slack(l_in, l_pre, layer_ms * 1e3, got_io)

    def run(mode):
        built = build_all(io_stream)
        torch.cuda.synchronize()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record(comp_stream)
        if mode == "compute_only":
            with torch.cuda.stream(comp_stream):
                for l in range(w.n_layers):
                    layer_compute()
        elif mode == "serial":
            # restore a layer on all SMs, then compute it: nothing overlaps
            with torch.cuda.stream(comp_stream):
                for l in range(w.n_layers):
                    rep.ring.tutti_kv_restore_layer(built[l][0], built[l][1], 0, stream=comp_stream)
                    layer_compute()
        else:
            for l, (first, cnt) in enumerate(built):
                sched.tutti_sched_enqueue(T.OP_READ, l, first, used)
            for l in range(w.n_layers):
                # before layer l begins: launch what the window holds (at least layer l's reads)
                for (op, first, cnt, sms, lay, est) in sched.tutti_sched_next(
                        T.PHASE_PREFILL, l, l_in, l_pre):
                    rep.ring.tutti_kv_restore_layer(first, cnt, sms, stream=io_stream)
                # layer l may start once its own IOCBs are done (they were launched now or
                # earlier); reads launched ahead for later layers do not hold it back
                for i in range(built[l][0], built[l][0] + used):
                    rep.ring.tutti_stream_wait_iocb(i, comp_stream)
                with torch.cuda.stream(comp_stream):
                    layer_compute()
            assert sched.tutti_sched_pending() == (0, 0)
            # the empty tail of every layer's reservation completes too
            for first, cnt in built:
                if cnt > used:
                    rep.ring.tutti_kv_restore_layer(first + used, cnt - used, got_io, stream=io_stream)
        t1.record(comp_stream)
        torch.cuda.synchronize()
        if mode == "compute_only":
            for f, c in built:
                rep.ring.tutti_kv_restore_layer(f, c, 0, stream=io_stream)
        poll(built)
        return t0.elapsed_time(t1)

    res = {m: round(min(run(m) for _ in range(3)), 3) for m in ("compute_only", "serial", "scheduled")}
    ok = rep.spot_check(64)
    out = {"demo": "slack-aware layer-wise pipelining, config-2 batch, GEMMs as layer compute",
           "store": "pinned host, zero-copy" if sched_host else "hbm", "layers": w.n_layers,
           "io_partition_sms": got_io, "compute_partition_sms": got_comp,
           "iocb_mib": args.sched_iocb_mib, "iocbs_per_layer_used": used,
           "profile": "tutti_sched_profile (library), %d table entries" % n_points,
           "io_profile_us_by_iocbs": profile, "io_profile_write_us_by_iocbs": profile_w,
           "estimate_vs_measured": est_err,
           "gemms_per_layer": gemms_per_layer, "layer_compute_ms": round(layer_ms, 3),
           "restore_ms_per_layer_on_partition": round(layer_restore_ms, 3),
           "total_ms": res,
           "bubble_ms_scheduled": round(res["scheduled"] - res["compute_only"], 3),
           "bubble_ms_serial": round(res["serial"] - res["compute_only"], 3),
           "spot_check": bool(ok)}
    sched.close()
    rep.ctx.tutti_sm_partition_destroy()
    rep.close()
    return out


def sweep_rows(args, local_rank, token_list, host_store=False, n_layers=32):
    """Restore / save of one request's prefix, all layers, for every prefix length asked for."""
    import torch
    from paper_2605_03375_b200 import tutti as T
    peak, _ = measured_peak()
    rows = []
    for tokens in token_list:
        a2 = argparse.Namespace(**vars(args))
        a2.config, a2.scale, a2.layers = 2, 1.0, 0
        # every layer has a pool buffer of its own: one launch moves all layers, its agents work
        # on several layers at once, and layers that shared a buffer would meet in L2
        a2.resident_layers = n_layers
        a2.ioctx_per_iocb = 2048
        a2.layers_per_launch = 0
        a2.iocb_mib = 0
        rep = Replica(a2, local_rank, host_store=host_store, n_layers=n_layers, hit_tokens=[tokens])
        assert rep.R == n_layers
        res = {"prefix_tokens": tokens,
               "payload_mib_per_layer": round(rep.payload_per_layer / (1 << 20), 1)}
        L, st = rep.w.n_layers, rep.stream
        for name, op in (("restore", T.OP_READ), ("save", T.OP_WRITE)):
            issue = rep.ring.tutti_kv_restore_layer if op == T.OP_READ else rep.ring.tutti_kv_save_layer

            def one_pass():
                # a pass as a user issues it: one build call and one copy launch for all layers,
                # then the completions of every layer
                rep.epoch += 1
                rep.batch.plan_epoch = rep.epoch
                rc, first, per = rep.ring.tutti_build_sqes_layers(rep.batch, 0, L, op, stream=st)
                issue(first, L * per, 0, stream=st)
                rc, nbytes, err, done = rep.ring.tutti_ring_poll_range(first, L * per, 20_000_000_000)
                assert (rc, err, nbytes) == (T.OK, 0, L * rep.payload_per_layer)
            for _ in range(2):
                one_pass()
            torch.cuda.synchronize()
            reps = 10 if tokens <= 16384 else 3
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            t0 = time.perf_counter()
            e0.record(st)
            for _ in range(reps):
                one_pass()
            e1.record(st)
            torch.cuda.synchronize()
            ms = max(e0.elapsed_time(e1), (time.perf_counter() - t0) * 1e3) / reps
            gbs = rep.w.n_layers * rep.payload_per_layer / (ms * 1e-3) / 1e9
            res[name + "_gbs"] = round(gbs, 1)
            res[name + "_us_per_layer"] = round(ms * 1e3 / rep.w.n_layers, 1)
            if not host_store:
                res[name + "_hbm_frac"] = round(2 * gbs / peak, 3)
        res["spot_check"] = bool(rep.spot_check(32))
        rows.append(res)
        rep.close()
        del rep
        torch.cuda.empty_cache()
    return rows


def leg_prefix_sweep(args, local_rank):
    """Raw restore / save bandwidth against prefix length, model bypassed (the measurement of the
    paper's Section 4.2.1, here against the HBM object store): one request, Llama-3-8B-shaped
    KV, 32 layers, descriptor build and host polls included; every pass is one build launch and
    one copy launch."""
    return {"sweep": "1 request, 8 KV heads x 128 x bf16, block 16, 32 layers, hbm store; whole "
                     "pass = 1 plan + 1 emit + 1 copy launch and one range poll",
            "rows": sweep_rows(args, local_rank, (1024, 2048, 4096, 16384, 131072))}


def run_length_sweep(args):
    """The same sweep on its own, all eight lengths, against the HBM or the pinned-host store."""
    rank, local_rank, world = init_dist("nccl")
    lengths = (1024, 2048, 4096, 8192, 16384, 32768, 65536, 131072)
    if args.sweep_tokens:
        lengths = tuple(int(t) for t in args.sweep_tokens.split(","))
    rows = sweep_rows(args, local_rank, lengths, host_store=args.sweep_host,
                      n_layers=args.layers or 32)
    if rank == 0:
        print(json.dumps({"sweep": "raw restore/save bandwidth vs prefix length, 1 request, "
                          "8 KV heads x 128 x bf16, block 16, 32 layers",
                          "store": "pinned host, zero-copy" if args.sweep_host else "hbm",
                          "rows": rows}), flush=True)


def run_reference(args):
    """The reference arm of this tier is the oracle on the host cores: each step is a
    bounded sample of the same workload (restore + save of one layer of the batch)."""
    rank, _, world = rank_env()
    if rank != 0:
        return
    import torch
    import oracle
    from paper_2605_03375_b200 import workload as wl
    w = wl.config(args.config, args.scale)
    og = oracle.geom(1, w.n_kv_heads, w.head_dim, w.elem_bytes, w.block_tokens, w.obj_tokens,
                     w.n_devices, w.layout, w.n_slots)
    lo = oracle.obj_layout(og)
    ob = (w.hit_tokens, w.obj_start, w.obj_slot, w.blk_start, w.block_ids)
    bb = int(lo.block_bytes)
    store = [wl.fill_u16_torch(w.seed, STREAM_STORE + d, 0, int(lo.dev_bytes) // 2, "cpu")
             .numpy().view(np.uint8) for d in range(w.n_devices)]
    pool = wl.fill_u16_torch(w.seed, STREAM_POOL, 0, w.n_pool_blocks * bb, "cpu").numpy().view(np.uint8)
    payload = w.total_tokens * 2 * int(lo.token_bytes)

    def step():
        assert oracle.restore_layer(og, 0, ob, store, pool, 0, w.n_pool_blocks * bb, bb,
                                    w.n_pool_blocks) == 0
        assert oracle.save_layer(og, 0, ob, store, pool, 0, w.n_pool_blocks * bb, bb,
                                 w.n_pool_blocks) == 0
    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = time.perf_counter() - t0
    value = 2 * payload * args.steps / dt / 1e9
    sample = "each step = restore+save of 1 layer of the batch (oracle, single thread)"
    # the block-granular form on every host core, beside it (a few steps)
    cores = os.cpu_count() or 1
    v_off = w.n_pool_blocks * bb
    n_mt = max(3, min(args.steps, 10))
    t1 = time.perf_counter()
    for _ in range(n_mt):
        for to_pool in (True, False):
            assert oracle.move_layer_blocks_mt(og, 0, ob, store, pool, 0, v_off, bb,
                                               w.n_pool_blocks, to_pool, cores) == 0
    all_cores = 2 * payload * n_mt / (time.perf_counter() - t1) / 1e9
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": round(value, 3), "unit": "GB/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": round(dt / args.steps * 1e3, 2), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "u8", "data": "synthetic",
        "config": {"workload": workload_name(w), "sample": sample},
        "cpu_baseline": {"value": round(value, 3), "unit": "GB/s", "cores": 1,
                         "host_cores": os.cpu_count(), "kind": "oracle", "sample": sample,
                         "all_cores": {"value": round(all_cores, 3), "unit": "GB/s", "cores": cores,
                                       "sample": f"{n_mt} such steps, one memcpy per block and K/V "
                                                 f"half, blocks dealt out over {cores} threads"}},
        "e2e": {"value": round(value, 3), "unit": "GB/s", "h2d_bytes_per_step": 0,
                "d2h_bytes_per_step": 0},
        "gpu_launches": 0}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=2, choices=[1, 2, 3, 4, 5])
    ap.add_argument("--scale", type=float, default=1.0)
    ap.add_argument("--layers", type=int, default=0,
                    help="override the layer count (small captures under a profiler)")
    ap.add_argument("--engine", type=int, default=0, help="0 auto, 1 ld/st, 2 bulk-async")
    ap.add_argument("--resident-layers", type=int, default=0)
    ap.add_argument("--sm-count", type=int, default=0,
                    help="run the copies as a capped launch of this many persistent CTAs")
    ap.add_argument("--ioctx-per-iocb", type=int, default=2048)
    ap.add_argument("--iocb-mib", type=int, default=0,
                    help="cut IOCBs by bytes (MiB per IOCB) instead of by context count")
    ap.add_argument("--ctas-per-sm", type=int, default=0)
    ap.add_argument("--bulk-warps", type=int, default=0)
    ap.add_argument("--bulk-stages", type=int, default=0)
    ap.add_argument("--claim", type=int, default=0)
    ap.add_argument("--bulk-chunk", type=int, default=0)
    ap.add_argument("--e2e-host-layers", type=int, default=8)
    ap.add_argument("--e2e-sms", type=int, default=12,
                    help="e2e leg, duplex mode: SMs of the restore direction")
    ap.add_argument("--e2e-save-sms", type=int, default=8,
                    help="e2e leg, duplex mode: SMs of the save direction")
    ap.add_argument("--e2e-group", type=int, default=2,
                    help="e2e leg, duplex mode: layers per copy launch")
    ap.add_argument("--e2e-mode", choices=["both", "zero_copy", "staged"], default="both",
                    help="e2e leg: kernels on the link (zero_copy), copy engines on the link (staged)")
    ap.add_argument("--stage-min-mib", type=float, default=2.0,
                    help="staged transfers: contexts smaller than this stay on the zero-copy path")
    ap.add_argument("--e2e-serial", action="store_true",
                    help="e2e leg: restore pass then save pass instead of overlapping them")
    ap.add_argument("--gemm-iters", type=int, default=20)
    ap.add_argument("--sweep-length", action="store_true",
                    help="raw restore/save bandwidth against prefix length (1K..128K tokens)")
    ap.add_argument("--sweep-tokens", default="", help="comma-separated prefix lengths for --sweep-length")
    ap.add_argument("--sweep-host", action="store_true", help="sweep against the pinned-host store")
    ap.add_argument("--sched-demo", action="store_true",
                    help="layer-wise pipelining under the slack-aware scheduler")
    ap.add_argument("--sched-host", action="store_true")
    ap.add_argument("--sched-sms", type=int, default=16)
    ap.add_argument("--sched-iocb-mib", type=int, default=64,
                    help="scheduler legs: bytes per IOCB (IOCBs cut by bytes)")
    ap.add_argument("--sched-gemms", type=int, default=3)
    ap.add_argument("--layers-per-launch", type=int, default=0,
                    help="consecutive layers whose IOCBs one copy launch executes "
                         "(0: chosen from the payload per layer)")
    ap.add_argument("--one-stream", action="store_true",
                    help="build and copy on one stream (default: descriptors on their own stream)")
    ap.add_argument("--pool-hnd", action="store_true",
                    help="head-major pool blocks [head][token][dim] (transposing copy)")
    ap.add_argument("--set", action="append", metavar="KEY=INT",
                    help="override a workload field, e.g. layout=0 n_devices=2 elem_bytes=1")
    ap.add_argument("--cfg4-layers", type=int, default=8,
                    help="config-4 leg: layers resident and timed (the figures are per layer)")
    ap.add_argument("--cfg5-layers", type=int, default=8)
    ap.add_argument("--no-configs", action="store_true",
                    help="skip the config 1/3/4/5 legs of the default line")
    ap.add_argument("--no-sched", action="store_true", help="skip the scheduler legs")
    ap.add_argument("--shared-prefix", action="store_true",
                    help="run the shared-prefix leg on its own")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--e2e-only", action="store_true", help="run the end-to-end leg on its own")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif (args.sched_demo or args.sweep_length or args.e2e_only or args.shared_prefix or
          args.config != 2):
        # a single leg on its own (one GPU)
        rank, local_rank, world = init_dist("nccl")
        if args.sweep_length:
            run_length_sweep(args)
            return
        if args.e2e_only:
            res = run_e2e(args, local_rank, world)
            if rank == 0:
                print(json.dumps(res), flush=True)
            return
        leg = (leg_sched_demo if args.sched_demo else leg_shared_prefix if args.shared_prefix else
               {1: leg_config1, 3: leg_config3, 4: leg_config4, 5: leg_config5}[args.config])
        extra = (args.sched_host,) if args.sched_demo else ()
        res = run_leg(leg, args, local_rank, *extra)
        if rank == 0:
            print(json.dumps(res), flush=True)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
