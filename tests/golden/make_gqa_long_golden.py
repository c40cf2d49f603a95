"""Writes tests/golden/gqa_long_group<g>.npz: the fp64 oracle's results for ONE WHOLE KV GROUP of the
long-context GQA configuration (B = 1, Hq = 32, Hkv = 8, S = 16384, D = 128, causal), computed on the CPU.

Calls only ``oracle/`` and the seeded input generator; never the CUDA library.  The group's backward is one
oracle task (a KV group owns its dK / dV), about six minutes on one core.  The whole group is computed; to keep
the stored file small only whole 128-row tiles are kept, as float32:

  * O, LSE, dQ of all four query heads of the group at query tiles QUERY_TILES,
  * dK, dV of the group's KV head at key tiles KEY_TILES (key tile 0 sums over all 4 x 16384 query rows,
    i.e. the longest accumulation the backward has), plus
  * max|dQ|, max|dK|, max|dV| over the whole group (the denominators of the gradient tolerance) and
    per-column sums of dK, dV over all keys (a whole-group check at any size).

Usage:  python tests/golden/make_gqa_long_golden.py [--group 5]
"""
import argparse
import os
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import attn_oracle as orc                                   # noqa: E402
from paper_2601_16238_b200.inputs import CONFIGS, make_inputs          # noqa: E402

QUERY_TILES = (0, 64, 127)
KEY_TILES = (0, 63, 127)
TILE = 128


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--group", type=int, default=5)
    args = ap.parse_args()
    cfg = CONFIGS["gqa_long"]
    G = cfg.Hq // cfg.Hkv
    g = args.group
    q, k, v, d_o = make_inputs(cfg)
    hs = slice(g * G, (g + 1) * G)
    qg, kg, vg, dog = q[:, hs], k[:, g:g + 1], v[:, g:g + 1], d_o[:, hs]
    t0 = time.time()
    o, lse = orc.attn_fwd(qg, kg, vg, True, cfg.scale)
    t1 = time.time()
    dq, dk, dv = orc.attn_bwd(qg, kg, vg, dog, True, cfg.scale)
    t2 = time.time()
    rows_q = np.concatenate([np.arange(t * TILE, (t + 1) * TILE) for t in QUERY_TILES])
    rows_k = np.concatenate([np.arange(t * TILE, (t + 1) * TILE) for t in KEY_TILES])
    out = os.path.join(os.path.dirname(os.path.abspath(__file__)), f"gqa_long_group{g}.npz")
    np.savez(out,
             group=np.int32(g), query_tiles=np.array(QUERY_TILES, np.int32), key_tiles=np.array(KEY_TILES, np.int32),
             o=o[0][:, rows_q].astype(np.float32), lse=lse[0][:, rows_q].astype(np.float32),
             dq=dq[0][:, rows_q].astype(np.float32),
             dk=dk[0, 0][rows_k].astype(np.float32), dv=dv[0, 0][rows_k].astype(np.float32),
             max_abs=np.array([np.abs(o).max(), np.abs(dq).max(), np.abs(dk).max(), np.abs(dv).max()]),
             dk_colsum=dk[0, 0].sum(axis=0), dv_colsum=dv[0, 0].sum(axis=0),
             dk_abs_colsum=np.abs(dk[0, 0]).sum(axis=0), dv_abs_colsum=np.abs(dv[0, 0]).sum(axis=0),
             oracle_seconds=np.array([t1 - t0, t2 - t1]), oracle_threads=np.int32(orc.num_threads()))
    print(f"wrote {out}: forward {t1 - t0:.1f} s, backward {t2 - t1:.1f} s, {orc.num_threads()} thread(s) available")


if __name__ == "__main__":
    main()
