"""In-kernel timeline of one CTA (debugging aid; not used by the library's normal operation).

Builds a second copy of the library with -DATTN_JVP_TRACE=2 (clock64 stamps at the hand-over points of the
roles of one CTA, see attn_jvp_kernel.cuh), runs one shape through it and prints, per 64-key tile, when the MMA
warp issued the score and value MMAs and when the softmax warps saw the scores, agreed on the reference max,
stored P~ and handed the tile back -- plus the mean tile period:

    python -m paper_2510_08431_b200.trace --B 1 --H 8 --Lq 18944 --Lk 4096 --D 128 [--mode jvp|kv_free|fwd] [--groups 1|2] [--pair 1|2]

With --totals the build is -DATTN_JVP_TRACE=1 instead: no per-tile stamps (they cost the MMA warp 10-20 % of a
tile), only the cycles each role of the traced CTA spent in blocking waits, summed in a register and written once
at the end -- who waits for whom, at the shipped build's speed.
"""
from __future__ import annotations

import argparse
import ctypes
import os
import subprocess

import numpy as np
import torch

from . import attn_jvp as binding
from . import build as lib_build
from . import synth

TRACE_LIB = os.path.join(lib_build.PKG, "libattn_jvp_trace.so")
TOTALS_LIB = os.path.join(lib_build.PKG, "libattn_jvp_trace_totals.so")
EVENTS, STEPS = 32, 96


def build_trace_library(level: int = 2) -> str:
    path = TRACE_LIB if level == 2 else TOTALS_LIB
    stale = (not os.path.exists(path)) or any(os.path.getmtime(d) > os.path.getmtime(path) for d in lib_build.DEPS)
    if stale:
        cmd = [lib_build._nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
               f"-DATTN_JVP_TRACE={level}", "-shared", "-Xcompiler", "-fPIC", "-I", os.path.join(lib_build.ROOT, "include"),
               "-o", path, lib_build.SRC, "-lcudart"]
        subprocess.run(cmd, check=True, capture_output=True)
    return path


def run(B, H, Lq, Lk, D, mode="jvp", groups=0, first=20, count=6, seed=4, pair=0, level=2):
    """Runs the shape three times through the trace build and returns the [EVENTS][STEPS] stamp array."""
    lib = ctypes.CDLL(build_trace_library(level))
    x = synth.make_inputs(B, H, Lq, Lk, D, 1.0, 0.5, seed, kv_tangent_free=(mode != "jvp"))
    g = {k: (None if t is None else t.cuda()) for k, t in x.items()}
    flags = {"jvp": 0, "kv_free": binding.KV_TANGENT_FREE, "fwd": binding.FWD_ONLY}[mode]
    lib.attn_jvp_set_tuning(binding.TUNE_SOFTMAX_GROUPS, int(groups))
    lib.attn_jvp_set_tuning(binding.TUNE_CTA_PAIR, int(pair))
    o = torch.empty_like(g["q"]); to = torch.empty_like(g["q"])
    lse = torch.empty((B, H, Lq), dtype=torch.float32, device="cuda")
    vp = ctypes.c_void_p
    lib.attn_jvp_fwd_stream.argtypes = [vp] * 9 + [ctypes.c_int] * 5 + [ctypes.c_float, ctypes.c_uint, vp]
    p = lambda t: None if t is None else t.data_ptr()
    for _ in range(3):
        rc = lib.attn_jvp_fwd_stream(p(g["q"]), p(g["k"]), p(g["v"]), p(g["tq"]), p(g["tk"]), p(g["tv"]), p(o), p(to),
                                     p(lse), B, H, Lq, Lk, D, D ** -0.5, flags, torch.cuda.current_stream().cuda_stream)
        assert rc == 0, rc
    torch.cuda.synchronize()
    assert lib.attn_jvp_device_status() == 0
    buf = (ctypes.c_longlong * (EVENTS * STEPS))()
    lib.attn_jvp_debug_read_trace.argtypes = [vp, ctypes.c_int]
    assert lib.attn_jvp_debug_read_trace(buf, EVENTS * STEPS) == EVENTS * STEPS
    return np.array(buf, dtype=np.int64).reshape(EVENTS, STEPS)


NAMES = {21: "MMA   score MMAs: issue begins", 2: "MMA   score MMAs issued", 3: "MMA   value MMAs: issue begins",
         4: "MMA   value MMAs issued", 29: "MMA   burst begins (loop top)", 30: "MMA   after tensor-core fence",
         23: "MMA   burst issued, warp reconverged", 19: "MMA   (blocked) V and K slots seen full", 22: "MMA   blocks for the tile's barriers", 24: "  softmax pass over the columns begins", 25: "  softmax pass over the columns ends",
         5: "  softmax scores seen (s_full)", 26: "  softmax scores in registers", 27: "  softmax reference max agreed",
         28: "  softmax P~, H~ stores issued", 13: "  softmax tile handed back"}


ITEM_NAMES = {1: "producer: Q, tQ may be replaced (q_free seen)", 10: "MMA   Q, tQ of the item seen", 11: "MMA   K(0) of the item seen",
              12: "  softmax epilogue begins", 20: "  softmax epilogue ends", 9: "producer: staging slots handed over",
              17: "producer: staged tiles complete, stores issued", 18: "producer: staging slots back in the ring"}


def report_items(t, first_item=3, count=2, tiles_per_item=8):
    """Timeline around the hand-over between work items of a persistent CTA (item-indexed events plus the tile
    events of the items' first and last tiles)."""
    ev = [(t[e][i], nm + f" (item {i})", i) for e, nm in ITEM_NAMES.items() for i in range(first_item, first_item + count) if t[e][i] > 0]
    for i in range(first_item, first_item + count):
        for g in (i * tiles_per_item - 1, i * tiles_per_item, i * tiles_per_item + 1):
            if 0 <= g < STEPS:
                ev += [(t[e][g], nm + f" (tile {g})", g) for e, nm in NAMES.items() if t[e][g] > 0]
    ev.sort()
    base = ev[0][0] if ev else 0
    for tm, nm, _ in ev:
        print(f"{tm - base:8d}  {nm}")


def report(t, first=20, count=6):
    ev = [(t[e][g], nm, g) for e, nm in NAMES.items() for g in range(first, first + count) if t[e][g] > 0]
    ev.sort()
    base = ev[0][0] if ev else 0
    for tm, nm, g in ev:
        print(f"{tm - base:8d}  {nm} (tile {g})")
    pv = t[3][10:60]
    pv = pv[pv > 0]
    if len(pv) > 1:
        print(f"mean tile period (value-MMA issue, tiles 10..{9 + len(pv)}): {(pv[-1] - pv[0]) / (len(pv) - 1):.0f} cycles")
    sm = (t[13][10:60] - t[5][10:60])[(t[13][10:60] > 0) & (t[5][10:60] > 0)]
    if len(sm):
        print(f"softmax warp, scores seen -> tile handed back: mean {sm.mean():.0f} cycles")
    print("MMA warp had to block for a tile:", int((t[22][10:60] > 0).sum()), "of 50 tiles; CTA lifetime",
          int(t[EVENTS - 1][1] - t[EVENTS - 1][0]), "cycles")


TOTALS = ["MMA warp blocked for a tile's P~ / operands", "MMA warp blocked at an item's start",
          "softmax warp blocked for the next scores", "epilogue: blocked for the item's last value MMAs",
          "epilogue: its own run"]


def report_totals(t, Lk):
    """Blocked-cycle totals of the traced CTA's roles (level-1 build): row EVENTS - 2 holds (cycles, count) pairs."""
    life = int(t[EVENTS - 1][1] - t[EVENTS - 1][0])
    tiles = int(t[EVENTS - 2][5])          # the softmax warp waits once per key tile
    n_kv = (Lk + 63) // 64
    print(f"CTA lifetime {life} cycles, {tiles} key tiles, {tiles / n_kv:.1f} work items: "
          f"{life / max(tiles, 1):.0f} cycles per tile, {life * n_kv / max(tiles, 1):.0f} per item")
    for k, name in enumerate(TOTALS):
        tot, n = int(t[EVENTS - 2][2 * k]), int(t[EVENTS - 2][2 * k + 1])
        print(f"  {name:50s} {tot:9d} cycles = {100.0 * tot / life:5.1f} % of the lifetime, {n} times, mean {tot / max(n, 1):.0f}")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--B", type=int, default=1); ap.add_argument("--H", type=int, default=8)
    ap.add_argument("--Lq", type=int, default=128 * 148); ap.add_argument("--Lk", type=int, default=4096)
    ap.add_argument("--D", type=int, default=128)
    ap.add_argument("--mode", default="jvp", choices=["jvp", "kv_free", "fwd"])
    ap.add_argument("--groups", type=int, default=0)
    ap.add_argument("--pair", type=int, default=0, help="CTA-pair kernel: 0 library's choice, 1 off, 2 on")
    ap.add_argument("--first", type=int, default=20); ap.add_argument("--count", type=int, default=4)
    ap.add_argument("--items", action="store_true", help="print the hand-over between work items instead of the tiles")
    ap.add_argument("--totals", action="store_true", help="blocked-cycle totals per role (no per-tile stamps)")
    a = ap.parse_args()
    if a.totals:
        report_totals(run(a.B, a.H, a.Lq, a.Lk, a.D, a.mode, a.groups, pair=a.pair, level=1), a.Lk)
        return
    t = run(a.B, a.H, a.Lq, a.Lk, a.D, a.mode, a.groups, pair=a.pair)
    if a.items:
        report_items(t, tiles_per_item=(a.Lk + 63) // 64)
    report(t, a.first, 0 if a.items else a.count)


if __name__ == "__main__":
    main()
