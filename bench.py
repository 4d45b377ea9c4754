#!/usr/bin/env python
"""Benchmark of the FlashLoop loop-r prefill hot path on B200.

One "step" = one pass of the whole hot path over one synthetic prompt: for every sparse loop
r = 2..R, one token selection, then for every layer: gather of the active hidden rows (input of
the projections, which are scaffolding outside the library), column selection (loop 2 only, from
the dense source loop's statistics), K/V residual quantization (which also leaves the active
rows' reconstructed K/V as bf16 rows in a transient workspace), and the loop attention on the
position-indexed stores (it reads the carried rows and writes the new O / Q rows itself: no
gathers or scatters around it); and one hidden-state scatter per loop.  Loop 2 recomputes the old
term of the replacement equation and leaves each row's background and mass; loops 3.. reuse them
(constant column budget) and compute the new term only.  A second timed variant runs the same
step without the materialized rows: every residual-carrying column is dequantized and added
inside the attention kernel (reported under "variants").
The dense source loop (loop 1) and the Q/K/V/O projections are outside the timed region; their
times are printed separately ("setup_ms", "scaffold_ms").

Metric: prompt tokens per second of the loop-r prefill, L / (time of one step).
Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle instead.
"""
from __future__ import annotations

import argparse
import ctypes as C
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)
from paper_2609_29812_b200 import replicas  # noqa: E402  (plain Python: importable without CUDA)

METRIC = "loop_r_prefill_tokens_per_s"
UNIT = "tokens/s"


# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) one attention launch moves, from ncu captures of exactly
# these launch shapes (one layer: every layer launches the same grid); the live timing of this file cannot measure
# it, so the bench line says "not measured in this run".  Keyed by (workload, L, layers-independent) and loop kind;
# a shape that is not listed reports null.
NCU_ATTN_TRAFFIC_BYTES = {
    ("c3:L=32768", "recompute"): 170.9e6,   # loop 2: loop_attn_tc_kernel<4,1,0> (144.0 MB read + 26.8 MB written)
    ("c3:L=32768", "economy"): 132.6e6,     # loops 3, 4: loop_attn_stream_kernel<4,1> (mean of 134.0 and 131.2 MB)
}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--loops", type=int, default=0, help="sched: number of loops R (default 8)")
    ap.add_argument("--workload", default="c3", choices=["c2", "c3", "c4", "c5", "sched", "decode", "proj"],
                    help="c3: the 48-layer stack at 32K (default, the metric's configuration); c2: one layer at 8K; "
                         "c5: the 128K memory configuration (prefill part; 24 layers resident unless --layers); "
                         "c4: the sparsity / depth sweep (one layer at 8K, a table of points); "
                         "decode: config 5's second phase, 32 single-token queries over the 4-loop store (sparse decode "
                         "attention, loops 2-4; a separate metric); "
                         "proj: the projections of the active rows as one gathered / scattering tensor-core GEMM "
                         "(fl_project_rows) beside row copies + library GEMMs (a separate line, not the metric); "
                         "sched: budgets that decay from loop to loop with real column pruning (Table 6's deep "
                         "schedule: tokens 90% -> 20%, columns pruned inside the previous set every loop)")
    ap.add_argument("--sweep", default="subset", choices=["subset", "full"], help="c4: which points to run")
    ap.add_argument("--int4-base", action="store_true",
                    help="keep every layer's loop-1 K/V packed (Appendix E: int4, keys per channel, values per token, "
                         "groups of 64, last 64 positions unquantized) and rebuild one layer's rows into a transient "
                         "buffer before each layer's work in each loop (fl_dequant_kv_base, inside the timed step)")
    ap.add_argument("--no-overlap", action="store_true",
                    help="issue the column selections in the main stream's order instead of on a second stream")
    ap.add_argument("--no-economy", action="store_true", help="recompute the old term in every loop")
    ap.add_argument("--no-variants", action="store_true", help="skip the in-kernel dequantization variant")
    ap.add_argument("--layers", type=int, default=0, help="override the number of layers (development)")
    ap.add_argument("--L", type=int, default=0, help="override the context length (development / profiling)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="launch call by call instead of replaying a CUDA graph")
    return ap.parse_args()


def get_workload(args):
    from paper_2609_29812_b200 import workloads
    if args.workload == "c2":
        w = workloads.config2()
        w = workloads.replace(w, rmsnorm=False)
    elif args.workload == "c5":
        w = workloads.config5(n_layers=args.layers or 24)
    else:
        w = workloads.config3()
    if args.L:
        w = workloads.replace(w, L=args.L)
    if args.layers:
        w = workloads.replace(w, n_layers=args.layers)
    return w


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p.get("bf16_tflops_sustained", p["bf16_tflops"]),
                "source": "measured (MEASURED_PEAKS.json; bf16 sustained)"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1400.0, "source": "fallback (6.65 TB/s, 1.4 PFLOP/s sustained)"}


# ------------------------------------------------------------------------------------------------
# clocks sampler
# ------------------------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc = index, None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for nm, val in zip(names, parts[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ------------------------------------------------------------------------------------------------
# the CUDA arm
# ------------------------------------------------------------------------------------------------
class Bench:
    def __init__(self, args, w, device, economy=True):
        import torch
        from paper_2609_29812_b200 import binding as B, pipeline as P, workloads
        self.torch, self.B, self.P, self.w, self.dev = torch, B, P, w, device
        self.ctx = B.Context(torch.device(device).index or 0)
        self.shape = P.shape_of(w)
        self.R, self.NL, self.H, self.dh, self.L, self.d = w.n_loops, w.n_layers, w.n_heads, w.head_dim, w.L, w.d
        self.nb = (w.L + w.q_block - 1) // w.q_block
        self.c = w.col_budget
        self.economy = economy
        self.int4_base = bool(getattr(args, "int4_base", False))
        self.base_group, self.base_tail = 64, 64
        self.stream = torch.cuda.Stream(device=device)
        self.sp = int(self.stream.cuda_stream)
        self.side = torch.cuda.Stream(device=device)      # column selections of the step (see run_step)
        self.sp2 = int(self.side.cuda_stream)
        self.overlap_select = not bool(getattr(args, "no_overlap", False))
        self.keep = []           # keeps tensors and host structs alive
        self.attn_flops_min, self.attn_flops_exec, self.attn_bytes = {}, {}, {}   # per loop r: lists over layers
        self.setup_ms = {}
        self._setup(workloads)

    # -- set-up: dense source loop per layer, token sets, buffers ------------------------------------
    def _setup(self, workloads):
        torch, B, P, w = self.torch, self.B, self.P, self.w
        dev, ctx, sh = self.dev, self.ctx, self.shape
        stack = workloads.DeviceStack(w, seed=0, device=dev)
        self.G = stack.stack_hidden()
        k_tok = w.k_tokens
        dense_ms = []
        with torch.cuda.stream(self.stream):
            self.sels, cand = [], None
            for r in range(2, self.R + 1):
                sel = P.select_tokens(ctx, sh, r, self.G[r - 2], self.G[r - 1], cand, k_tok)
                self.sels.append(sel)
                cand = sel.active_idx
            self.stream.synchronize()
            self.g_work = self.G[0].clone()
            n_max = self.sels[0].n
            # compact buffers shared by all layers (a real engine reuses them the same way)
            mkrows = lambda: torch.empty(n_max, self.H, self.dh, dtype=torch.bfloat16, device=dev)
            self.xbuf = torch.empty(n_max, self.d, dtype=torch.bfloat16, device=dev)
            self.o_out_buf = mkrows()      # end-to-end arm: the last layer's new O rows, gathered for the read-back
            self.layers = []
            if self.int4_base:
                # one transient copy of a layer's rebuilt base for the whole stack; the packed form is what stays
                self.k_transient = torch.empty(self.L, self.H, self.dh, dtype=torch.bfloat16, device=dev)
                self.v_transient = torch.empty_like(self.k_transient)
            for l in range(self.NL):
                gen = stack.layer(l)
                q1, k1, v1 = gen.qkv1()
                st = P.LayerState(ctx, w, dev)
                if self.int4_base:
                    g_, t_ = self.base_group, self.base_tail
                    Lq = max(0, self.L - t_)
                    n_tg = (Lq + g_ - 1) // g_
                    u8 = lambda *s_: torch.empty(s_, dtype=torch.uint8, device=dev)
                    f16 = lambda *s_: torch.empty(s_, dtype=torch.float16, device=dev)
                    st.base_tensors = [u8(Lq, self.d * w.bits // 8), f16(n_tg, self.d), f16(n_tg, self.d),
                                       u8(Lq, self.d * w.bits // 8), f16(Lq, self.d // g_), f16(Lq, self.d // g_),
                                       torch.empty(self.L - Lq, self.d, dtype=torch.bfloat16, device=dev),
                                       torch.empty(self.L - Lq, self.d, dtype=torch.bfloat16, device=dev)]
                    st.base_q = B.make_base_q(*st.base_tensors, g_, t_)
                    st.row_mask = torch.zeros(self.H, (self.L + 31) // 32, dtype=torch.int32, device=dev)
                    B.fl_quant_kv_base(ctx, sh, k1, v1, st.base_q)
                    B.fl_dequant_kv_base(ctx, sh, st.base_q, self.k_transient, self.v_transient)
                    # every loop of the layer, the dense one included, reads the base as it is stored
                    k1, v1 = self.k_transient, self.v_transient
                e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
                e0.record(self.stream)
                st.dense_loop(q1, k1, v1)
                e1.record(self.stream)
                st.select_columns_dense()
                st.hidden = gen.hidden(self.R)
                st.lse1 = st.lse
                st.lse_work = st.lse.clone()
                st.q_work, st.o_work = st.q_store.clone(), st.o_store.clone()
                st.carry_buffers()
                st.rows = {}
                for r in range(2, self.R + 1):
                    sel = self.sels[r - 2]
                    st.rows[r] = gen.rows(r, sel.active_idx)
                    # loops that reuse the carried old term read only the rows after the loop's residual
                    st.alloc_stream(sel, rows="cur" if (self.economy and r > 2) else True)
                # the same store without the transient rows: the attention kernel then rebuilds every
                # residual-carrying column itself (dequantize-and-add inside the kernel)
                strip = lambda streams: [{k: v for k, v in s_.items() if not k.startswith("rows_")} for s_ in streams]
                st.store_plain = B.make_store(st.k_base, st.v_base, strip(st.k_streams), strip(st.v_streams))
                gen.release()
                self.stream.synchronize()
                dense_ms.append(e0.elapsed_time(e1))
                if l == 0 or w.name.startswith("c4"):
                    self._account(st)
                self.layers.append(st)
        torch.cuda.synchronize()
        self.setup_ms["dense_source_loop_per_layer"] = statistics.median(dense_ms)
        self.setup_ms["dense_source_loop_all_layers"] = sum(dense_ms)
        self._scaffold()
        self.plans = {}

    def _scaffold(self):
        """Times the projections around the hot path (cuBLAS through torch; scaffolding, not part of the metric):
        [n, d] x [d, 3d] for Q/K/V and [n, d] x [d, d] for the output projection, per layer and loop."""
        torch = self.torch
        n = self.sels[0].n
        x = torch.randn(n, self.d, device=self.dev, dtype=torch.bfloat16)
        wqkv = torch.randn(self.d, 3 * self.d, device=self.dev, dtype=torch.bfloat16)
        wo = torch.randn(self.d, self.d, device=self.dev, dtype=torch.bfloat16)
        out = {}
        for name, wt in (("qkv_projection", wqkv), ("o_projection", wo)):
            for _ in range(3):
                x @ wt
            e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(10):
                x @ wt
            e1.record(); torch.cuda.synchronize()
            out[name + "_per_layer_loop"] = e0.elapsed_time(e1) / 10
        out["per_step"] = (out["qkv_projection_per_layer_loop"] + out["o_projection_per_layer_loop"]) * self.NL * (self.R - 1)
        self.scaffold_ms = out

    def _account(self, st):
        """Algorithmic FLOPs and bytes of each loop's attention launch for one layer, from the index sets (every
        layer of the stack has the same token sets; its column sets differ but not their sizes)."""
        torch, w = self.torch, self.w
        e, H, dh, d, c, L = 2, self.H, self.dh, self.d, self.c, self.L
        col = st.col_idx.long()                                 # [H, nb, c], -1 padded
        pay_col_head = 2 * (dh * w.bits // 8 + 4 * (dh // w.group)) if w.bits != 16 else 2 * dh * e
        uniq = []
        for h in range(H):
            u = torch.unique(col[h]); uniq.append(u[u >= 0])
        for r in range(2, self.R + 1):
            sel = self.sels[r - 2]
            act = sel.active_idx.long()
            blk = act // w.q_block
            pairs = 0
            for h in range(H):
                rows_cols = col[h][blk]                         # [n, c]
                pairs += int(((rows_cols >= 0) & (rows_cols <= act[:, None])).sum().item())
            one_term = 4.0 * dh * pairs                         # QK^T and PV of one term over the kept (row, column) pairs
            # minimum the method needs: the old term is recomputed only after a dense source loop (loop 2) or a
            # pruned set; otherwise it is the previous loop's new term
            need_old = r == 2
            self.attn_flops_min.setdefault(r, []).append(one_term * (2.0 if need_old else 1.0))
            self.attn_flops_exec.setdefault(r, []).append(one_term * (2.0 if (need_old or not self.economy) else 1.0))
            byt = 0.0
            for h in range(H):
                byt += float(len(uniq[h])) * 2 * dh * e         # K and V base rows of the selected columns
                for rr in range(2, r + 1):                      # residual payloads those columns carry
                    slot = self.sels[rr - 2].slot_of_pos.long()
                    byt += float((slot[uniq[h]] >= 0).sum().item()) * pay_col_head
            byt += 4.0 * sel.n * d * e + 8.0 * H * sel.n + 4.0 * H * self.nb * (c + 1) + 4.0 * L * (r - 1)
            self.attn_bytes.setdefault(r, []).append(byt)

    # -- the step as a flat list of C-ABI calls ---------------------------------------------------------
    def plan(self, rows=True):
        """The step as a list of (tag, function, arguments, loop).  rows: the attention gathers the loop's active
        columns from the rows the quantization kernel materialized (True) or rebuilds them itself (False)."""
        key = bool(rows)
        if key in self.plans:
            return self.plans[key]
        B, lib, w = self.B, self.B.lib, self.w
        ctx, shp, sp = self.ctx.handle, C.byref(self.shape), self.sp
        p = lambda t: C.c_void_p(int(t.data_ptr())) if t is not None else None
        e = 2
        row_bytes = self.d * e
        calls, launches = [], 0
        # per-step algorithmic bytes of the memory-bound stages (for the whole-step roofline)
        stage_bytes = {"select_tokens": 0.0, "gather_scatter": 0.0, "quant": 0.0, "select_columns": 0.0}
        if self.int4_base:
            stage_bytes["dequant_base"] = 0.0
            base_q_bytes = B.fl_kv_base_q_bytes(self.shape, self.base_group, self.base_tail)
            if not hasattr(self, "base_share"):
                # share of a layer's (head, position) pairs its sparse loops read, measured on layer 0
                st0, sel0 = self.layers[0], self.sels[0]
                B.fl_mark_base_rows(self.ctx, self.shape, st0.col_idx, st0.col_cnt, self.c, sel0.active_idx, sel0.n,
                                    st0.row_mask, stream=self.stream)
                self.stream.synchronize()
                m = st0.row_mask.view(self.torch.uint8)
                lut = self.torch.tensor([bin(i).count("1") for i in range(256)], device=m.device)
                self.base_share = float(lut[m.long()].sum().item()) / (self.H * self.L)
        pay_row = 2 * (self.d * w.bits // 8 + 4 * (self.d // w.group)) if w.bits != 16 else 2 * self.d * e
        for r in range(2, self.R + 1):
            sel = self.sels[r - 2]
            prev = self.sels[r - 3] if r > 2 else None
            n_cand = prev.n if prev is not None else self.L
            cand = prev.active_idx if prev is not None else None
            calls.append(("select_tokens", lib.fl_select_tokens,
                          (ctx, shp, r, p(self.G[r - 2]), p(self.G[r - 1]), p(cand), n_cand, w.k_tokens,
                           p(sel.scores), p(sel.active_idx), p(sel.slot_of_pos), None, sp), r))
            launches += 2
            stage_bytes["select_tokens"] += 2.0 * n_cand * self.d * e + 8.0 * n_cand + 4.0 * sel.n + 4.0 * self.L
            n = sel.n
            for st in self.layers:
                store = st.store if rows else st.store_plain
                self.keep.append(store)
                calls.append(("gather", lib.fl_gather_rows, (ctx, p(st.hidden), p(sel.active_idx), n, row_bytes,
                                                             p(self.xbuf), sp), r))
                if r == 2:
                    calls.append(("select_columns", lib.fl_select_columns,
                                  (ctx, shp, p(st.col_scores), None, None, self.L, self.c, p(st.col_idx),
                                   p(st.col_cnt), None, sp), r))
                    launches += 1
                    tri = sum(min(self.L, (b + 1) * w.q_block) for b in range(self.nb))
                    stage_bytes["select_columns"] += 4.0 * self.H * (tri + self.nb * (self.c + 1))
                if self.int4_base:
                    # the rows this layer's sparse loops read (selected columns per head, active positions) are marked
                    # once, in loop 2 (later active sets are nested in loop 2's, the column lists stay), and only they
                    # are rebuilt into the transient buffer before the layer's work in every loop
                    if r == 2:
                        calls.append(("dequant_base", lib.fl_mark_base_rows,
                                      (ctx, shp, p(st.col_idx), p(st.col_cnt), self.c, p(sel.active_idx), n,
                                       p(st.row_mask), None, sp), r))
                        launches += 1
                        stage_bytes["dequant_base"] += 4.0 * self.H * self.nb * (self.c + 1) + 4.0 * n
                    calls.append(("dequant_base", lib.fl_dequant_kv_base,
                                  (ctx, shp, C.byref(st.base_q), p(st.row_mask), p(self.k_transient),
                                   p(self.v_transient), None, sp), r))
                    launches += 1
                    # algorithmic bytes: packed codes + metadata in, rows out, for the marked share of the rows
                    stage_bytes["dequant_base"] += self.base_share * (base_q_bytes + 2.0 * self.L * self.d * e)
                q_new, k_new, v_new = st.rows[r]
                calls.append(("quant", lib.fl_quant_kv_residual,
                              (ctx, shp, r, p(k_new), p(v_new), p(sel.active_idx), n, C.byref(store), None, sp), r))
                # Q^(r-1), O^(r-1) are read from and O^(r), Q^(r) written to position-indexed stores by the attention
                # call itself; loop 2 reads the pristine loop-1 stores and writes the work stores, so that every
                # step starts from the same state
                q_src = st.q_store if r == 2 else st.q_work
                o_src = st.o_store if r == 2 else st.o_work
                lse_prev = st.lse1 if r == 2 else st.lse_work
                if self.economy:
                    carry = B.make_carry(st.bg_store, st.mass, r > 2)
                    self.keep.append(carry)
                    calls.append(("attention", lib.fl_loop_attention_indexed_carry,
                                  (ctx, shp, r, p(q_new), p(q_src), p(st.q_work), p(sel.active_idx), n,
                                   C.byref(store), p(st.col_idx), p(st.col_cnt), self.c, p(lse_prev), p(st.lse_work),
                                   p(o_src), p(st.o_work), C.byref(carry), None, None, sp), r))
                else:
                    calls.append(("attention", lib.fl_loop_attention_indexed,
                                  (ctx, shp, r, p(q_new), p(q_src), p(st.q_work), p(sel.active_idx), n,
                                   C.byref(store), p(st.col_idx), p(st.col_cnt), self.c, p(lse_prev), p(st.lse_work),
                                   p(o_src), p(st.o_work), None, None, sp), r))
                # gather, quantization, attention; with the carried old term and the materialized rows the recomputing
                # call of loop 2 is two launches (old-term pass, new-term pass)
                launches += 3 + (1 if (self.economy and rows and r == 2) else 0)
                stage_bytes["gather_scatter"] += 2.0 * n * row_bytes
                stage_bytes["quant"] += 4.0 * n * self.d * e + n * pay_row * (r - 1)
            calls.append(("scatter", lib.fl_scatter_update, (ctx, p(self.xbuf), p(sel.active_idx), n, row_bytes,
                                                             p(self.g_work), sp), r))
            launches += 1
            stage_bytes["gather_scatter"] += 2.0 * n * row_bytes
        self.plans[key] = (calls, launches, stage_bytes)
        return self.plans[key]

    def run_step(self, rows=True, attn_events=None):
        """Issue one step on self.stream.  attn_events: list to which (loop, start, end) events are appended.
        Column selection depends on nothing inside the step (its scores come from the source loop), so unless
        --no-overlap is given every layer's selection is issued on a second stream when the step starts and the
        layer's first consumer (the attention call of loop 2, or the row marking of the packed base) waits for it:
        the selections then run in the SM slots the attention launches leave idle."""
        torch = self.torch
        calls = self.plan(rows)[0]
        bad = 0
        overlap = self.overlap_select and attn_events is None
        sel_events = {}
        if overlap:
            start = torch.cuda.Event()
            start.record(self.stream)
            self.side.wait_event(start)          # the previous step's readers of the column lists are done
            for i, (tag, fn, a, r) in enumerate(calls):
                if tag == "select_columns":
                    bad |= fn(*(a[:-1] + (self.sp2,)))
                    ev = torch.cuda.Event()
                    ev.record(self.side)
                    sel_events[i] = ev
        pending = None
        for i, (tag, fn, a, r) in enumerate(calls):
            if overlap and tag == "select_columns":
                pending = sel_events[i]
                continue
            if pending is not None and tag in ("attention", "dequant_base"):
                self.stream.wait_event(pending)
                pending = None
            if attn_events is not None and tag == "attention":
                e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
                e0.record(self.stream)
                bad |= fn(*a)
                e1.record(self.stream)
                attn_events.append((r, e0, e1))
            else:
                bad |= fn(*a)
        if bad:
            raise RuntimeError("a C-ABI call failed inside the step")

    def breakdown(self, rows=True):
        """One untimed-for-the-metric pass with events around every call: per-stage GPU time (ms), per stage and
        loop, and the time of each loop r (select_tokens of loop r up to the call before loop r + 1)."""
        torch = self.torch
        evs = []
        with torch.cuda.stream(self.stream):
            for tag, fn, a, r in self.plan(rows)[0]:
                e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
                e0.record(self.stream); rc = fn(*a); e1.record(self.stream)
                assert rc == 0
                evs.append((tag, e0, e1, r))
        self.stream.synchronize()
        out, by_loop = {}, {}
        for tag, e0, e1, r in evs:
            ms = e0.elapsed_time(e1)
            out[tag] = out.get(tag, 0.0) + ms
            d = by_loop.setdefault(f"loop_{r}", {})
            d[tag] = d.get(tag, 0.0) + ms
        starts = [i for i, (tag, _, _, _) in enumerate(evs) if tag == "select_tokens"] + [len(evs)]
        per_loop = {}
        for li in range(len(starts) - 1):
            ms = evs[starts[li]][1].elapsed_time(evs[starts[li + 1] - 1][2])
            per_loop[f"loop_{li + 2}"] = {"ms": round(ms, 4), "tokens_per_s": round(self.L / (ms * 1e-3), 1),
                                          "stages_ms": {k: round(v, 4) for k, v in by_loop[f"loop_{li + 2}"].items()}}
        self.per_loop = per_loop
        return {k: round(v, 4) for k, v in out.items()}

    def time_graph(self, rows, steps, barrier):
        """Captures one step into a CUDA graph and times `steps` replays with CUDA events on the stream."""
        torch = self.torch
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=self.stream):
            self.run_step(rows)
        with torch.cuda.stream(self.stream):
            for _ in range(2):
                graph.replay()
        barrier()
        t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
        host_t0 = time.perf_counter()
        with torch.cuda.stream(self.stream):
            t0.record(self.stream)
            for _ in range(steps):
                graph.replay()
            t1.record(self.stream)
        host_issue_ms = (time.perf_counter() - host_t0) * 1e3 / steps
        barrier()
        return t0.elapsed_time(t1) / steps, host_issue_ms


def kv_bytes_per_token(bench):
    B, w = bench.B, bench.w
    fl, dense = B.fl_kv_store_bytes(bench.shape, bench.layers[0].store, w.n_loops, w.n_layers)
    if bench.int4_base:   # the packed base replaces the bf16 rows; the transient copy of one layer is shared by the stack
        fl += B.fl_kv_base_q_bytes(bench.shape, bench.base_group, bench.base_tail) - 2 * w.L * w.d * 2
        fl += 2 * w.L * w.d * 2 / w.n_layers
    return fl / w.L, dense / w.L


def attention_roofline(bench, attn_events, steps, peaks, workload_key):
    """Roofline of the attention launches (the dominant kernel) from the live event timings: the whole set and per
    loop.  FLOPs are the minimum the method needs (old term counted only where it must be recomputed: loop 2); the
    count the kernel executes is printed beside it."""
    P_tc, BW = peaks["bf16_tflops"] * 1e12, peaks["hbm_gbs"] * 1e9
    per_loop, tot_ms, tot_fmin, tot_fexec, tot_b, tot_roof = {}, 0.0, 0.0, 0.0, 0.0, 0.0
    n_launch = 0
    for r in sorted(bench.attn_flops_min):
        ms = [a.elapsed_time(b) for rr, a, b in attn_events if rr == r]
        if not ms:
            continue
        avg = sum(ms) / len(ms)
        fmin = sum(bench.attn_flops_min[r]) / len(bench.attn_flops_min[r])
        fexec = sum(bench.attn_flops_exec[r]) / len(bench.attn_flops_exec[r])
        byt = sum(bench.attn_bytes[r]) / len(bench.attn_bytes[r])
        t_roof = max(fmin / P_tc, byt / BW)
        traffic = NCU_ATTN_TRAFFIC_BYTES.get((workload_key, "recompute" if fexec > 1.5 * fmin or r == 2 else "economy"))
        per_loop[f"loop_{r}"] = {"avg_launch_ms": avg, "launches_per_step": len(ms) // steps, "flops_min": fmin,
                                 "flops_executed": fexec, "bytes": byt, "t_roof_us": t_roof * 1e6,
                                 "bound": "tensor" if fmin / P_tc >= byt / BW else "hbm",
                                 "frac": t_roof / (avg * 1e-3), "tflops_min": fmin / (avg * 1e-3) / 1e12,
                                 "traffic": traffic}
        k = len(ms)
        tot_ms += sum(ms); tot_fmin += fmin * k; tot_fexec += fexec * k; tot_b += byt * k; tot_roof += t_roof * k
        n_launch += k
    avg_ms = tot_ms / n_launch
    flops, byt = tot_fmin / n_launch, tot_b / n_launch
    if tot_fmin / P_tc >= tot_b / BW:
        roof = {"bound": "tensor", "achieved": flops / (avg_ms * 1e-3) / 1e12, "peak": peaks["bf16_tflops"],
                "unit": "TFLOP/s"}
    else:
        roof = {"bound": "hbm", "achieved": byt / (avg_ms * 1e-3) / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s"}
    roof["frac"] = roof["achieved"] / roof["peak"]
    traffics = [v["traffic"] for v in per_loop.values()]
    roof.update({"kernel": "fl_loop_attention_indexed_carry", "kernel_name": "loop_attn_tc_kernel",
                 "avg_launch_ms": avg_ms, "launches": n_launch // steps,
                 "flops_per_launch": flops, "flops_executed_per_launch": tot_fexec / n_launch,
                 "bytes_per_launch": byt,
                 "flop_count": "minimum the method needs: both terms in loop 2 (dense source), the new term only in "
                               "later loops over unchanged column sets; flops_executed is what the kernel ran",
                 "frac_per_launch_roofs": tot_roof / (tot_ms * 1e-3),
                 "traffic": (sum(t * v["launches_per_step"] for t, v in zip(traffics, per_loop.values())) /
                             sum(v["launches_per_step"] for v in per_loop.values())) if all(t is not None for t in traffics) else None,
                 "traffic_source": "ncu dram__bytes_read.sum + dram__bytes_write.sum per launch of this shape, from the "
                                   "captures summarised under profiles/; not measured in this run",
                 "peak_source": peaks["source"],
                 "avg_launch_ms_source": "CUDA events around every attention launch of K steps issued call by call on "
                                         "the timed stream, right after the timed graph replays",
                 "per_loop": per_loop})
    return roof


def step_roofline(bench, stage_bytes, peaks, ms):
    """The benchmark spec's definition for the whole step: the slower of (all kept FLOPs at the tensor peak) and (all
    algorithmic bytes at the HBM bandwidth); the sum of per-stage maxima is printed beside it for diagnosis."""
    P_tc, BW = peaks["bf16_tflops"] * 1e12, peaks["hbm_gbs"] * 1e9
    NL = bench.NL
    F = sum(sum(v) / len(v) * NL for v in bench.attn_flops_min.values())
    Bt = sum(sum(v) / len(v) * NL for v in bench.attn_bytes.values()) + sum(stage_bytes.values())
    t_roof = max(F / P_tc, Bt / BW)
    t_sum = sum(max(sum(bench.attn_flops_min[r]) / len(bench.attn_flops_min[r]) / P_tc,
                    sum(bench.attn_bytes[r]) / len(bench.attn_bytes[r]) / BW) * NL for r in bench.attn_flops_min)
    t_sum += sum(stage_bytes.values()) / BW
    return {"t_roof_ms": t_roof * 1e3, "frac": t_roof * 1e3 / ms, "flops": F, "bytes": Bt,
            "t_flops_ms": F / P_tc * 1e3, "t_bytes_ms": Bt / BW * 1e3,
            "definition": "max(sum of kept FLOPs / bf16 peak, sum of algorithmic bytes / HBM copy bandwidth) over the step",
            "sum_of_stage_maxima_ms": t_sum * 1e3, "frac_sum_of_stage_maxima": t_sum * 1e3 / ms,
            # the same definition against the nominal figures (7.7 TB/s HBM3e, 2250 TFLOP/s dense bf16), for context
            "frac_of_nominal": max(F / 2250e12, Bt / 7.7e12) * 1e3 / ms}


def run_ours(args):
    import torch
    import torch.distributed as dist
    rank = int(os.environ.get("RANK", 0)); world = int(os.environ.get("WORLD_SIZE", 1))
    local = int(os.environ.get("LOCAL_RANK", 0))
    torch.cuda.set_device(local)
    device = f"cuda:{local}"
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(device))
    if args.workload in ("c4", "sched", "decode", "proj"):
        {"c4": run_sweep, "sched": run_schedule, "decode": run_decode, "proj": run_projection}[args.workload](
            args, device, rank)
        if world > 1:
            dist.destroy_process_group()
        return
    w = get_workload(args)
    peaks = load_peaks()
    bench = Bench(args, w, device, economy=not args.no_economy)
    stream = bench.stream

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    calls, launches_per_step, stage_bytes = bench.plan(True)
    with torch.cuda.stream(stream):
        for _ in range(max(args.warmup, 3)):
            bench.run_step()
    barrier()
    sampler = ClockSampler(local)
    sampler.start()
    # The step (a few hundred dependent launches) is captured once into a CUDA graph; the timed region replays it K
    # times. Events cannot sit between the kernels of a replay, so the attention launches are timed in a second pass
    # of K steps issued call by call on the same stream, whose step time is reported next to the graph's.
    host_issue_ms = None
    ms_graph = None
    if not args.no_graph:
        ms_graph, host_issue_ms = bench.time_graph(True, args.steps, barrier)
    attn_events = []
    e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(stream):
        e0.record(stream)
        for _ in range(args.steps):
            bench.run_step(True, attn_events)
        e1.record(stream)
    barrier()
    clocks = sampler.stop()
    ms_evented = e0.elapsed_time(e1) / args.steps
    ms = ms_graph if ms_graph is not None else ms_evented
    ms = replicas.max_over_ranks(ms, world, device)
    value = replicas.job_throughput(w.L, world, ms)

    wl_key = f"{args.workload}:L={w.L}"
    roof = attention_roofline(bench, attn_events, args.steps, peaks, wl_key)
    roof["share_of_step"] = sum(a.elapsed_time(b) for _, a, b in attn_events) / args.steps / ms_evented
    step_roof = step_roofline(bench, stage_bytes, peaks, ms)

    out = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
           "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
           "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
           "config": {"workload": f"{w.name}: L={w.L}, {w.n_layers} layers, d={w.d}, {w.n_heads}x{w.head_dim} MHA, "
                                  f"R={w.n_loops}, token budget {w.k_tokens} rows, column budget {w.col_budget}, "
                                  f"q_block {w.q_block}, int{w.bits} g{w.group} residuals",
                      "base": ("int4 per-channel K / per-token V, groups of 64, last 64 positions bf16; one layer's rows "
                               "rebuilt into a transient buffer per layer and loop inside the step"
                               if bench.int4_base else "bf16 rows resident"),
                      "column_selection": ("every layer's selection issued on a second stream at the start of the step, "
                                           "joined before its first consumer" if bench.overlap_select
                                           else "in the main stream's order"),
                      "old_term": ("recomputed in loop 2, carried (background rows + mass) in later loops"
                                   if bench.economy else "recomputed in every loop"),
                      "parallelism": "replicas only" if world > 1 else "single GPU",
                      "l2": "inputs exceed L2 (each step streams the per-layer stores, far above 126 MB)"},
           "gpu_launches": launches_per_step * args.steps, "host_issue_ms_per_step": host_issue_ms,
           "launch_mode": ("CUDA graph of one step, replayed" if ms_graph is not None else "call by call"),
           "ms_per_step_call_by_call_with_events": ms_evented,
           "clocks": clocks, "roofline": roof,
           "step_roofline": step_roof,
           "setup_ms": {k: round(v, 3) for k, v in bench.setup_ms.items()},
           "scaffold_ms": {k: round(v, 4) for k, v in bench.scaffold_ms.items()}}
    fl_b, dense_b = kv_bytes_per_token(bench)
    out["kv_bytes_per_token"] = {"flashloop": fl_b * w.n_layers, "dense_looped": dense_b * w.n_layers,
                                 "ratio": dense_b / fl_b, "per": "token, all layers"}
    if rank == 0:
        out["breakdown_ms"] = bench.breakdown()
        out["per_loop"] = bench.per_loop
        # the memory-bound stages: algorithmic bytes per step, time of the evented pass, achieved bandwidth
        bd = out["breakdown_ms"]
        stage_ms = {"select_tokens": bd.get("select_tokens", 0.0), "quant": bd.get("quant", 0.0),
                    "select_columns": bd.get("select_columns", 0.0),
                    "gather_scatter": bd.get("gather", 0.0) + bd.get("scatter", 0.0),
                    "dequant_base": bd.get("dequant_base", 0.0)}
        out["memory_bound_stages"] = {
            k: {"bytes_per_step": v, "ms_per_step": stage_ms[k], "achieved_gbs": v / (stage_ms[k] * 1e-3) / 1e9,
                "frac_of_hbm_peak": v / (stage_ms[k] * 1e-3) / 1e9 / peaks["hbm_gbs"]}
            for k, v in stage_bytes.items() if stage_ms.get(k, 0.0) > 0.0}
    if not args.no_variants and not args.no_graph:
        # stage (4) as the paper words it: the packed residual streams are read, dequantized and added inside the
        # attention kernel (no materialized rows); same step otherwise
        with torch.cuda.stream(stream):
            for _ in range(3):
                bench.run_step(False)
        barrier()
        ms_b, _ = bench.time_graph(False, args.steps, barrier)
        ev_b = []
        with torch.cuda.stream(stream):
            bench.run_step(False, ev_b)
        barrier()
        ms_b = replicas.max_over_ranks(ms_b, world, device)
        out["variants"] = {"in_kernel_dequantize_and_add": {
            "ms_per_step": ms_b, "value": replicas.job_throughput(w.L, world, ms_b), "unit": UNIT,
            "attention_avg_launch_ms": {f"loop_{r}": (lambda v: sum(v) / len(v))([a.elapsed_time(b) for rr, a, b in ev_b if rr == r])
                                        for r in sorted(set(rr for rr, _, _ in ev_b))},
            "note": "fl_quant_kv_residual writes no rows; the attention kernel rebuilds every selected column that is "
                    "active in the loop from base + residual streams (Eq. 8) on its way into shared memory"}}
        if rank == 0:
            out["variants"]["in_kernel_dequantize_and_add"]["breakdown_ms"] = bench.breakdown(False)
    if not args.no_e2e:
        out["e2e"] = run_e2e(bench, args, world, barrier)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline(bench)
    if rank == 0:
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def run_decode(args, device, rank):
    """Config 5's decode phase on the hot path's side of it: a batch of 32 single-token queries runs loops 2..4 of the
    sparse decode attention over the store the prefill left (bf16 base + int4 residual streams), column budget 2048
    per (query, head), every layer.  Column subsets are random ascending subsets of the prompt (what they are does not
    change the traffic); K/V of the selected columns are rebuilt in registers.  HBM-bound: the roofline is the bytes
    of the selected base rows and payloads.  Prints one JSON line (a metric of its own, not the prefill metric)."""
    import torch
    from paper_2609_29812_b200 import binding as B, pipeline as P, workloads
    L, NL, Bq = args.L or 131072, args.layers or 8, 32
    w = workloads.config5(L=L, n_layers=NL)
    c = w.col_budget
    peaks = load_peaks()
    ctx = B.Context(torch.device(device).index or 0)
    sh = P.shape_of(w)
    stack = workloads.DeviceStack(w, seed=0, device=device)
    G = stack.stack_hidden()
    H, dh, R = w.n_heads, w.head_dim, w.n_loops
    sels, cand = [], None
    for r in range(2, R + 1):
        sel = P.select_tokens(ctx, sh, r, G[r - 2], G[r - 1], cand, w.k_tokens)
        sels.append(sel); cand = sel.active_idx
    layers = []
    for l in range(NL):
        gen = stack.layer(l)
        st = P.LayerState(ctx, w, device)
        _, k1, v1 = gen.qkv1()
        st.k_base, st.v_base = k1, v1
        for r in range(2, R + 1):
            sel = sels[r - 2]
            st.alloc_stream(sel, rows=False)
            _, kr, vr = gen.rows(r, sel.active_idx)
            st.quantize(r, kr, vr, sel)
        gen.release()
        layers.append(st)
    g = torch.Generator(device=device); g.manual_seed(7)
    col_idx = torch.stack([torch.sort(torch.randperm(L, device=device, generator=g)[:c])[0]
                           for _ in range(Bq * H)]).to(torch.int32).view(Bq, H, c).contiguous()
    col_cnt = torch.full((Bq, H), c, dtype=torch.int32, device=device)
    mk = lambda: (torch.randn(Bq, H, dh, device=device, generator=g) * 0.5).to(torch.bfloat16)
    q = [mk() for _ in range(R)]
    o = mk(); lse = torch.full((Bq, H), 12.0, dtype=torch.float32, device=device)
    stream = torch.cuda.Stream(device=device)
    def step():
        for st in layers:
            for r in range(2, R + 1):
                B.fl_decode_attention(ctx, sh, r, q[r - 1], q[r - 2], Bq, st.store, col_idx, col_cnt, c, lse, lse, o, o,
                                      None, stream=stream)
    with torch.cuda.stream(stream):
        for _ in range(3):
            step()
    torch.cuda.synchronize()
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(stream):
        t0.record(stream)
        for _ in range(args.steps):
            step()
        t1.record(stream)
    torch.cuda.synchronize()
    ms = t0.elapsed_time(t1) / args.steps
    n_calls = NL * (R - 1)
    # bytes per call: base K and V rows of every selected column, plus the payloads those columns carry
    pay = 2 * (dh * w.bits // 8 + 4 * (dh // w.group))
    byt = 0.0
    flat = col_idx.long().view(-1)
    for r in range(2, R + 1):
        b_r = float(flat.numel()) * 2 * dh * 2
        for rr in range(2, r + 1):
            b_r += float((sels[rr - 2].slot_of_pos.long()[flat] >= 0).sum().item()) * pay
        byt += b_r
    byt *= NL
    if rank == 0:
        print(json.dumps({"metric": "sparse_decode_attention_ms_per_step", "value": ms, "unit": "ms", "n_gpus": 1,
                          "steps": args.steps, "warmup": 3, "higher_is_better": False, "dtype": "f32",
                          "data": "synthetic",
                          "config": {"workload": f"decode over the 4-loop store: L={L}, {NL} layers, batch {Bq} single-token "
                                                 f"queries, {H}x{dh} heads, column budget {c}, loops 2..{R}, int4 g128"},
                          "gpu_launches": n_calls * args.steps, "ms_per_layer_loop": ms / n_calls,
                          "roofline": {"bound": "hbm", "achieved": byt / (ms * 1e-3) / 1e9, "peak": peaks["hbm_gbs"],
                                       "unit": "GB/s", "frac": byt / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                       "bytes_per_step": byt, "traffic": None, "peak_source": peaks["source"]},
                          "scaled_to_48_layers_ms": ms * 48 / NL}))


def run_projection(args, device, rank):
    """The projections around the hot path at the benchmark shape (3277 active rows of 32768, d = 2048), per layer and
    loop: Q/K/V ([n, d] x [d, 3d]) from rows gathered out of the hidden store, and the output projection ([n, d] x
    [d, d]) added into the rows of the hidden store.  Two arms on the same buffers: fl_project_rows (one kernel each:
    the gather is the GEMM's A-operand load, the scatter-add its epilogue) and row copies + library GEMMs
    (fl_gather_rows + cuBLAS through torch; cuBLAS + torch's index_add_).  Eight layers' stores and weights are used in
    turn (1.3 GB: each call finds its inputs in HBM, not in L2).  Prints one JSON line, a metric of its own."""
    import torch
    from paper_2609_29812_b200 import binding as B
    L, d, NL = args.L or 32768, 2048, args.layers or 8
    n = max(1, L // 10)
    peaks = load_peaks()
    ctx = B.Context(torch.device(device).index or 0)
    g = torch.Generator(device=device); g.manual_seed(3)
    bf = torch.bfloat16
    hid = [(torch.randn(L, d, device=device, generator=g)).to(bf) for _ in range(NL)]
    wqkv = [(torch.randn(3 * d, d, device=device, generator=g) / d ** 0.5).to(bf) for _ in range(NL)]
    wo = [(torch.randn(d, d, device=device, generator=g) / d ** 0.5).to(bf) for _ in range(NL)]
    idx = torch.sort(torch.randperm(L, device=device, generator=g)[:n])[0].to(torch.int32)
    idx64 = idx.long()
    qkv = torch.empty(n, 3 * d, device=device, dtype=bf)
    rows = torch.empty(n, d, device=device, dtype=bf)
    attn_out = (torch.randn(n, d, device=device, generator=g)).to(bf)
    status = torch.zeros(1, dtype=torch.int32, device=device)
    stream = torch.cuda.Stream(device=device)

    def timed(fn, reps):
        with torch.cuda.stream(stream):
            for l in range(3):
                fn(l % NL)
        torch.cuda.synchronize()
        t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(stream):
            t0.record(stream)
            for it in range(reps):
                fn(it % NL)
            t1.record(stream)
        torch.cuda.synchronize()
        return t0.elapsed_time(t1) / reps

    reps = max(8, args.steps * NL)
    fused_qkv = lambda l: B.fl_project_rows(ctx, hid[l], L, idx, n, d, wqkv[l], 3 * d, qkv, n, None, 0, status, stream=stream)
    fused_o = lambda l: B.fl_project_rows(ctx, attn_out, n, None, n, d, wo[l], d, hid[l], L, idx, 1, status, stream=stream)
    fused_qkv_compact = lambda l: B.fl_project_rows(ctx, rows, n, None, n, d, wqkv[l], 3 * d, qkv, n, None, 0, status, stream=stream)
    lib_gather = lambda l: B.fl_gather_rows(ctx, hid[l], idx, n, d * 2, rows, stream=stream)
    lib_qkv = lambda l: torch.matmul(rows, wqkv[l].t(), out=qkv)
    o_tmp = torch.empty(n, d, device=device, dtype=bf)
    lib_o = lambda l: torch.matmul(attn_out, wo[l].t(), out=o_tmp)
    lib_add = lambda l: hid[l].index_add_(0, idx64, o_tmp)
    def lib_qkv_both(l):
        lib_gather(l); lib_qkv(l)
    def lib_o_both(l):
        lib_o(l); lib_add(l)
    # the same with the residual codec (Eq. 8) as the epilogue of the K and V columns, against row copy + library GEMM
    # + fl_quant_kv_residual: loop 2 of a config-3 layer (random base rows, one residual stream, materialized rows)
    from paper_2609_29812_b200 import pipeline as P, workloads
    wl = workloads.replace(workloads.config3(L=L, n_layers=1))
    slot = torch.full((L,), -1, dtype=torch.int32, device=device)
    slot[idx64] = torch.arange(n, dtype=torch.int32, device=device)
    sel = P.TokenSelection(idx, slot, None, n)
    states = []
    for l in range(NL):
        st = P.LayerState(ctx, wl, device)
        st.k_base = torch.randn(L, wl.n_heads, wl.head_dim, device=device, generator=g).to(bf)
        st.v_base = torch.randn(L, wl.n_heads, wl.head_dim, device=device, generator=g).to(bf)
        st.alloc_stream(sel)
        states.append(st)
    sh = states[0].shape
    q_out = torch.empty(n, d, device=device, dtype=bf)
    qkv3 = torch.empty(3, n, d, device=device, dtype=bf)
    w3 = [w_.view(3, d, d).transpose(1, 2) for w_ in wqkv]
    fused_qkv_quant = lambda l: B.fl_project_qkv_quant(ctx, sh, 2, hid[l], L, idx, n, wqkv[l], q_out, None,
                                                       states[l].store, status, stream=stream)
    lib_qkv3 = lambda l: torch.matmul(rows.unsqueeze(0), w3[l], out=qkv3)
    lib_quant = lambda l: B.fl_quant_kv_residual(ctx, sh, 2, qkv3[1], qkv3[2], idx, n, states[l].store, stream=stream)
    def lib_qkv_quant(l):
        lib_gather(l); lib_qkv3(l); lib_quant(l)
    sampler = ClockSampler(torch.device(device).index or 0)
    sampler.start()
    res = {"fused_qkv": timed(fused_qkv, reps), "fused_o": timed(fused_o, reps),
           "fused_qkv_with_codec_epilogue": timed(fused_qkv_quant, reps),
           "library_qkv_then_quant": timed(lib_qkv_quant, reps),
           "library_batched_qkv_gemm_alone": timed(lib_qkv3, reps), "quant_alone": timed(lib_quant, reps),
           "same_kernel_qkv_on_compact_rows": timed(fused_qkv_compact, reps),
           "library_qkv": timed(lib_qkv_both, reps), "library_o": timed(lib_o_both, reps),
           "library_gather_alone": timed(lib_gather, reps), "library_qkv_gemm_alone": timed(lib_qkv, reps),
           "library_o_gemm_alone": timed(lib_o, reps), "library_index_add_alone": timed(lib_add, reps)}
    clocks = sampler.stop()
    assert int(status.item()) == 0, "a bounded wait ran out inside fl_project_rows"
    fl_qkv, fl_o = 2.0 * n * d * 3 * d, 2.0 * n * d * d
    ms = res["fused_qkv"] + res["fused_o"]
    if rank == 0:
        print(json.dumps({"metric": "active_row_projection_ms_per_layer_loop", "value": ms, "unit": "ms", "n_gpus": 1,
                          "steps": reps, "warmup": 3, "higher_is_better": False, "dtype": "bf16", "data": "synthetic",
                          "config": {"workload": f"projections of the active rows: L={L}, n={n}, d={d}, Q/K/V + output "
                                                 f"projection with scattered residual add; {NL} layers' stores and "
                                                 "weights in turn (inputs exceed L2)"},
                          "gpu_launches": 2 * reps, "ms": {k: round(v, 5) for k, v in res.items()},
                          "library_ms_per_layer_loop": res["library_qkv"] + res["library_o"],
                          "roofline": {"bound": "tensor", "achieved": (fl_qkv + fl_o) / (ms * 1e-3) / 1e12,
                                       "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                                       "frac": (fl_qkv + fl_o) / (ms * 1e-3) / 1e12 / peaks["bf16_tflops"],
                                       "qkv_tflops": fl_qkv / (res["fused_qkv"] * 1e-3) / 1e12,
                                       "o_tflops": fl_o / (res["fused_o"] * 1e-3) / 1e12,
                                       "library_qkv_gemm_tflops": fl_qkv / (res["library_qkv_gemm_alone"] * 1e-3) / 1e12,
                                       "traffic": None, "peak_source": peaks["source"]},
                          "clocks": clocks}))


def run_schedule(args, device, rank):
    """Decaying schedule (Appendix E, Table 6, the deep model's row): the token budget falls linearly from 90% to 20%
    of the prompt over loops 2..R and every loop prunes the column sets inside the previous ones (Appendix D.2, a
    sparse source loop), from 2048 down to 256 columns per block.  The old term is recomputed in every loop (the
    sets change), next-loop column scores are emitted by the attention call and fl_select_columns runs on candidate
    lists.  Prints one JSON line: step time, tokens/s and the per-stage breakdown."""
    import torch
    from paper_2609_29812_b200 import binding as B, pipeline as P, workloads
    L, R, NL = args.L or 8192, args.loops or 8, args.layers or 4
    lin = lambda a, b: [a + (b - a) * i / max(R - 2, 1) for i in range(R - 1)]
    tok_frac = lin(0.90, 0.20)
    c_cols = [max(64, int(round(x / 64.0)) * 64) for x in lin(2048, 256)]
    w = workloads.replace(workloads.sweep_point(R, tok_frac[0], c_cols[0], 4, L=L), name=f"sched_R{R}", rmsnorm=False,
                          n_layers=NL, changed_fracs=tuple(tok_frac))
    k_tok = [int(f * L + 0.5) for f in tok_frac]
    ctx = B.Context(torch.device(device).index or 0)
    sh = P.shape_of(w)
    stream = torch.cuda.Stream(device=device)
    sp = int(stream.cuda_stream)
    stack = workloads.DeviceStack(w, seed=0, device=device)
    G = stack.stack_hidden()
    H, dh, d = w.n_heads, w.head_dim, w.d
    nb = (L + w.q_block - 1) // w.q_block
    lib = B.lib
    p = lambda t: C.c_void_p(int(t.data_ptr())) if t is not None else None
    calls, keep = [], []
    with torch.cuda.stream(stream):
        sels, cand = [], None
        for r in range(2, R + 1):
            sel = P.select_tokens(ctx, sh, r, G[r - 2], G[r - 1], cand, k_tok[r - 2])
            sels.append(sel); cand = sel.active_idx
        stream.synchronize()
        xbuf = torch.empty(sels[0].n, d, dtype=torch.bfloat16, device=device)
        g_work = G[0].clone()
        layers = []
        for l in range(NL):
            gen = stack.layer(l)
            st = P.LayerState(ctx, w, device)
            st.dense_loop(*gen.qkv1())
            st.hidden = gen.hidden(R)
            st.lse1, st.lse_work = st.lse, st.lse.clone()
            st.q_work, st.o_work = st.q_store.clone(), st.o_store.clone()
            st.rows = {r: gen.rows(r, sels[r - 2].active_idx) for r in range(2, R + 1)}
            for r in range(2, R + 1):
                st.alloc_stream(sels[r - 2])
            st.cols = {r: (torch.empty(H, nb, c_cols[r - 2], dtype=torch.int32, device=device),
                           torch.empty(H, nb, dtype=torch.int32, device=device),
                           torch.zeros(H, nb, c_cols[r - 2], dtype=torch.float32, device=device)) for r in range(2, R + 1)}
            gen.release()
            layers.append(st)
        stream.synchronize()
    launches = 0
    for r in range(2, R + 1):
        sel, prev = sels[r - 2], (sels[r - 3] if r > 2 else None)
        n_cand = prev.n if prev is not None else L
        calls.append(("select_tokens", lib.fl_select_tokens,
                      (ctx.handle, C.byref(sh), r, p(G[r - 2]), p(G[r - 1]), p(prev.active_idx) if prev else None, n_cand,
                       k_tok[r - 2], p(sel.scores), p(sel.active_idx), p(sel.slot_of_pos), None, sp)))
        launches += 2
        for st in layers:
            ci, cc, cs = st.cols[r]
            calls.append(("gather", lib.fl_gather_rows, (ctx.handle, p(st.hidden), p(sel.active_idx), sel.n, d * 2, p(xbuf), sp)))
            if r == 2:
                calls.append(("select_columns", lib.fl_select_columns,
                              (ctx.handle, C.byref(sh), p(st.col_scores), None, None, L, c_cols[0], p(ci), p(cc), None, sp)))
                launches += 1
            q_new, k_new, v_new = st.rows[r]
            keep.append(st.store)
            calls.append(("quant", lib.fl_quant_kv_residual,
                          (ctx.handle, C.byref(sh), r, p(k_new), p(v_new), p(sel.active_idx), sel.n, C.byref(st.store), None, sp)))
            q_src, o_src, lse_prev = (st.q_store, st.o_store, st.lse1) if r == 2 else (st.q_work, st.o_work, st.lse_work)
            last = r == R
            calls.append(("attention", lib.fl_loop_attention_indexed,
                          (ctx.handle, C.byref(sh), r, p(q_new), p(q_src), p(st.q_work), p(sel.active_idx), sel.n,
                           C.byref(st.store), p(ci), p(cc), c_cols[r - 2], p(lse_prev), p(st.lse_work), p(o_src),
                           p(st.o_work), None if last else p(cs), None, sp)))
            launches += 3 + (0 if last else 1)
            if not last:
                ni, nc, _ = st.cols[r + 1]
                calls.append(("prune_columns", lib.fl_select_columns,
                              (ctx.handle, C.byref(sh), p(cs), p(ci), p(cc), c_cols[r - 2], c_cols[r - 1], p(ni), p(nc), None, sp)))
                launches += 1
        calls.append(("scatter", lib.fl_scatter_update, (ctx.handle, p(xbuf), p(sel.active_idx), sel.n, d * 2, p(g_work), sp)))
        launches += 1

    def step():
        for tag, fn, a in calls:
            assert fn(*a) == 0
    with torch.cuda.stream(stream):
        for _ in range(3):
            step()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=stream):
        step()
    with torch.cuda.stream(stream):
        graph.replay()
    torch.cuda.synchronize()
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(stream):
        t0.record(stream)
        for _ in range(args.steps):
            graph.replay()
        t1.record(stream)
    torch.cuda.synchronize()
    ms = t0.elapsed_time(t1) / args.steps
    evs = []
    with torch.cuda.stream(stream):
        for tag, fn, a in calls:
            e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
            e0.record(stream); assert fn(*a) == 0; e1.record(stream)
            evs.append((tag, e0, e1))
    torch.cuda.synchronize()
    brk = {}
    for tag, e0, e1 in evs:
        brk[tag] = brk.get(tag, 0.0) + e0.elapsed_time(e1)
    fl_b, dense_b = B.fl_kv_store_bytes(sh, layers[0].store, R, NL)
    if rank == 0:
        print(json.dumps({"metric": METRIC, "value": L / (ms * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": args.steps,
                          "warmup": 3, "ms_per_step": ms, "higher_is_better": True, "dtype": "bf16", "data": "synthetic",
                          "config": {"workload": f"decaying schedule: L={L}, {NL} layers, R={R}, token budgets {k_tok}, "
                                                 f"column budgets {c_cols} (pruned inside the previous set), int4 g128"},
                          "gpu_launches": launches * args.steps, "launch_mode": "CUDA graph of one step, replayed",
                          "breakdown_ms": {k: round(v, 4) for k, v in brk.items()},
                          "kv_bytes_per_token": {"flashloop": fl_b / L * NL, "dense_looped": dense_b / L * NL,
                                                 "ratio": dense_b / fl_b}}))


SWEEP_SUBSET = [(R, t, c, b) for R in (2, 4, 8, 16) for t in (0.10,) for c in (512,) for b in (4,)] + \
               [(4, t, 512, 4) for t in (0.05, 0.25, 0.50)] + [(4, 0.10, c, 4) for c in (128, 2048)] + \
               [(4, 0.10, 512, b) for b in (2, 8)]


def run_sweep(args, device, rank):
    """Config 4: one layer at L = 8192; R x token budget x column budget x bit width.  Each point: the step as a
    CUDA graph, K replays timed with CUDA events.  Prints one JSON line holding the table."""
    import torch
    from paper_2609_29812_b200 import workloads
    pts = SWEEP_SUBSET if args.sweep == "subset" else \
        [(R, t, c, b) for R in (2, 4, 8, 16) for t in (0.05, 0.10, 0.25, 0.50) for c in (128, 512, 2048) for b in (2, 4, 8)]
    peaks = load_peaks()
    rows = []
    barrier = torch.cuda.synchronize
    for (R, t, c, b) in pts:
        w = workloads.replace(workloads.sweep_point(R, t, c, b, L=args.L or 8192), rmsnorm=False)
        bench = Bench(args, w, device, economy=not args.no_economy)
        calls, launches, stage_bytes = bench.plan(True)
        with torch.cuda.stream(bench.stream):
            for _ in range(3):
                bench.run_step()
        barrier()
        ms, _ = bench.time_graph(True, args.steps, barrier)
        sr = step_roofline(bench, stage_bytes, peaks, ms)
        fl_b, dense_b = kv_bytes_per_token(bench)
        rows.append({"R": R, "token_frac": t, "c": c, "bits": b, "ms_per_step": round(ms, 4),
                     "tokens_per_s": round(w.L / (ms * 1e-3), 1), "step_roofline_frac": round(sr["frac"], 4),
                     "kv_ratio": round(dense_b / fl_b, 3), "launches": launches})
        del bench
        torch.cuda.empty_cache()
    if rank == 0:
        print(json.dumps({"metric": METRIC, "unit": UNIT, "n_gpus": 1, "steps": args.steps, "warmup": 3,
                          "higher_is_better": True, "dtype": "bf16", "data": "synthetic",
                          "config": {"workload": f"c4 sweep ({args.sweep}): one layer, L={args.L or 8192}, "
                                                 "d=2048, 16x128 MHA, g128 residuals"},
                          "value": statistics.median([r_["tokens_per_s"] for r_ in rows]),
                          "sweep": rows}))


def run_e2e(bench, args, world, barrier):
    """Same step, but every step's inputs (hidden state of each loop; Q/K/V rows of every layer and loop)
    come from pinned host memory and the last layer's new attention rows go back to the host."""
    import torch
    import torch.distributed as dist
    w = bench.w
    copy_stream = torch.cuda.Stream(device=bench.dev)
    host = {}
    h2d = 0
    for r in range(2, bench.R + 1):
        g = bench.G[r - 1]
        host[("G", r)] = g.cpu().pin_memory(); h2d += g.numel() * g.element_size()
        for li, st in enumerate(bench.layers):
            for j, t in enumerate(st.rows[r]):
                host[(li, r, j)] = t.cpu().pin_memory(); h2d += t.numel() * t.element_size()
    out_host = torch.empty_like(bench.o_out_buf, device="cpu").pin_memory()
    d2h = out_host.numel() * out_host.element_size() * (bench.R - 1)
    # which call index starts each (loop) and each (layer, loop)
    calls = bench.plan(True)[0]
    marks = {}
    li = -1
    for i, (tag, fn, a, r) in enumerate(calls):
        if tag == "select_tokens":
            li = -1; marks[i] = ("G", r)
        elif tag == "quant":
            li += 1; marks[i] = (li, r)

    def one_step():
        events = {}
        copy_stream.wait_stream(bench.stream)          # the previous step has consumed its inputs
        with torch.cuda.stream(copy_stream):
            for i in sorted(marks):
                key = marks[i]
                if key[0] == "G":
                    bench.G[key[1] - 1].copy_(host[key], non_blocking=True)
                else:
                    for j, t in enumerate(bench.layers[key[0]].rows[key[1]]):
                        t.copy_(host[(key[0], key[1], j)], non_blocking=True)
                ev = torch.cuda.Event(); ev.record(copy_stream); events[i] = ev
        n_calls = len(calls)
        with torch.cuda.stream(bench.stream):
            for i, (tag, fn, a, r) in enumerate(calls):
                if i in events:
                    bench.stream.wait_event(events[i])
                rc = fn(*a)
                assert rc == 0
                end_of_loop = i == n_calls - 1 or calls[i + 1][0] == "select_tokens"
                if end_of_loop:                        # result of the loop: the last layer's new attention rows
                    sel = bench.sels[r - 2]
                    rc = bench.B.fl_gather_rows(bench.ctx, bench.layers[-1].o_work, sel.active_idx, sel.n,
                                                bench.d * 2, bench.o_out_buf, stream=bench.sp)
                    out_host.copy_(bench.o_out_buf, non_blocking=True)

    copy_stream.wait_stream(bench.stream)
    for _ in range(2):
        one_step()
    barrier()
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    t0.record(bench.stream)
    steps = max(2, min(args.steps, 5))
    for _ in range(steps):
        one_step()
    bench.stream.wait_stream(copy_stream)
    t1.record(bench.stream)
    barrier()
    ms = t0.elapsed_time(t1) / steps
    ms = replicas.max_over_ranks(ms, world, bench.dev)
    return {"value": replicas.job_throughput(w.L, world, ms), "unit": UNIT, "ms_per_step": ms, "h2d_bytes_per_step": h2d,
            "d2h_bytes_per_step": d2h,
            "note": "pinned host inputs copied on a side stream ahead of the compute stream; last layer's new O rows read back per loop"}


# ------------------------------------------------------------------------------------------------
# CPU oracle arm (reported baseline; `--impl reference`)
# ------------------------------------------------------------------------------------------------
def oracle_sample(w, n_heads_sample=16, n_blocks_sample=0, seed=0):
    """Times the oracle, as it stands, on a bounded sample of the workload: token selection of every loop
    in full (stack hidden state), and for `n_heads_sample` heads of ONE layer the residual codec on all
    active rows and the sparse attention of `n_blocks_sample` query blocks (0 = all); scaled to all heads,
    blocks and layers."""
    import torch
    from oracle import flashloop_oracle as fo
    from paper_2609_29812_b200 import workloads
    t_setup = time.time()
    stack = workloads.DeviceStack(w, seed=seed, device="cpu")
    R, L, dh = w.n_loops, w.L, w.head_dim
    nb = (L + w.q_block - 1) // w.q_block
    G = [g.float().numpy() for g in stack.stack_hidden()]
    f = lambda t: t.float().numpy()
    # token selection: full
    t0 = time.time()
    cand = np.arange(L); act_sets = []
    for r in range(2, R + 1):
        _, cand = fo.select_tokens(G[r - 2], G[r - 1], cand, w.k_tokens, w.eps)
        act_sets.append(cand)
    t_tok = time.time() - t0
    gen = stack.layer(0)
    n_heads_sample = max(1, min(n_heads_sample, w.n_heads))
    if n_blocks_sample <= 0 or n_blocks_sample >= nb:
        blocks = list(range(nb))
    else:
        blocks = sorted(set(int(b) for b in np.linspace(nb // 3, nb - 1, n_blocks_sample)))
    qkv1 = [f(t) for t in gen.qkv1()]
    rows_r = {r: [f(t) for t in gen.rows(r, torch.from_numpy(act_sets[r - 2].astype(np.int32)))]
              for r in range(2, R + 1)}
    t_quant = t_attn = 0.0
    for h in range(n_heads_sample):
        q1, k1, v1 = [t[:, h:h + 1, :].copy() for t in qkv1]
        d1 = fo.dense_loop_attention(q1, k1, v1, w.sm_scale, w.q_block, rows_to_cache=act_sets[0], head_list=[0],
                                     block_list=blocks)                   # set-up (dense source), not timed
        sets, cache = {}, {}
        for b in range(nb):
            sets[(0, b)] = np.zeros(0, dtype=np.int64)
            cache[(0, b)] = (np.zeros(0, dtype=np.int64), np.zeros((0, 0)))
        for b in blocks:
            end = min(L, (b + 1) * w.q_block)
            S = fo.select_columns(d1["col_scores"][0, b, :end], np.arange(end), w.col_budget)
            rows, P = d1["probs"][(0, b)]
            sets[(0, b)] = S; cache[(0, b)] = (rows, P[:, S])
        khat, vhat = k1.astype(np.float32), v1.astype(np.float32)
        o_full = d1["O"]
        for r in range(2, R + 1):
            act = act_sets[r - 2]
            qr, kr, vr = [t[:, h:h + 1, :].copy() for t in rows_r[r]]
            t0 = time.time()
            khat_new, _ = fo.residual_update(kr, khat, act, w.bits, w.group)
            vhat_new, _ = fo.residual_update(vr, vhat, act, w.bits, w.group)
            t_quant += time.time() - t0
            t0 = time.time()
            res = fo.sparse_loop_attention(qr, khat_new, vhat_new, vhat, o_full[act], act, sets, cache, w.sm_scale,
                                           w.q_block, head_list=[0], block_list=blocks, kv_round=fo.round_bf16)
            t_attn += time.time() - t0
            o_full = o_full.copy(); o_full[act] = res["O"]
            cache = {key: (res["probs"][key] if key[1] in blocks else cache[key]) for key in cache}
            khat, vhat = khat_new, vhat_new
    per_head = (t_quant + t_attn * nb / len(blocks)) / n_heads_sample
    total = t_tok + w.n_layers * w.n_heads * per_head
    cores = os.cpu_count() or 1
    try:
        cores = len(os.sched_getaffinity(0))
    except Exception:
        pass
    return {"value": L / total, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"token selection of loops 2..{R} in full ({t_tok:.2f} s); {n_heads_sample} of {w.n_heads} heads of one "
                      f"of {w.n_layers} layers: residual codec on all active rows ({t_quant:.2f} s) and sparse attention of "
                      f"{len(blocks)} of {nb} query blocks ({t_attn:.2f} s); scaled by heads x blocks x layers = "
                      f"{total:.1f} s per prompt",
            "measured_s": t_tok + t_quant + t_attn, "setup_s": time.time() - t_setup - (t_tok + t_quant + t_attn)}


def cpu_baseline(bench):
    return oracle_sample(bench.w)


def run_reference(args):
    rank = int(os.environ.get("RANK", 0))
    if rank != 0:
        return
    w = get_workload(args)
    for _ in range(min(args.warmup, 1)):
        oracle_sample(w, n_heads_sample=1, n_blocks_sample=1)
    vals = []
    steps = max(1, args.steps)
    t_all = time.time()
    for _ in range(steps):
        s = oracle_sample(w)
        vals.append(s)
        if time.time() - t_all > 150:
            break
    v = statistics.median([s["value"] for s in vals])
    out = {"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": len(vals),
           "warmup": min(args.warmup, 1), "ms_per_step": 1e3 * w.L / v, "higher_is_better": True, "scaling": "weak",
           "vs_baseline": None, "dtype": "f64", "data": "synthetic",
           "config": {"workload": f"{w.name}: L={w.L}, {w.n_layers} layers (oracle timed on a bounded sample and scaled)"},
           "cpu_baseline": {"value": v, "unit": UNIT, "kind": "oracle", "cores": vals[0]["cores"],
                            "sample": vals[0]["sample"]},
           "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
           "gpu_launches": 0}
    print(json.dumps(out))


if __name__ == "__main__":
    a = parse_args()
    if a.impl == "reference":
        run_reference(a)
    else:
        run_ours(a)
