"""Row activity of the gate masks at tensor-tile granularity (oracle only, no GPU).

TEST INFRASTRUCTURE / ANALYSIS: runs the CPU oracle on the synthetic workloads and prints, as a
markdown table, how much of the conditional path (Eq. 1, second case) a kernel that works on
blocks of pixel rows x output channels can skip.  For column blocks of N output channels:

  row activity   fraction of (pixel row, column block) pairs with at least one open gate: the
                 rows a row-compacting kernel must still compute;
  idle blocks    fraction of (128-pixel tile, column block) pairs with no open gate at all: the
                 MMAs a tile-skipping kernel drops.

With independent decisions of density tau a row of N gates is active with probability
1 - (1 - tau)^N; the table shows how far the spatially smooth inputs and a static reordering of
the output channels (most active channels first) move the masks away from that.

    python -m oracle.row_activity [--images 8] [--layers c64@56,c128@28]
"""
from __future__ import annotations

import argparse

import numpy as np

from oracle import oracle as O
from paper_1805_12549_b200 import synth

BLOCKS = (8, 16, 32, 64, 128)
TILE_ROWS = 128


def masks_for(shape, images, density, rho):
    """Gate decisions [pixels, c_out] of one layer: statistics from the partial sums of the first
    four images, one scalar Delta at the quantile that gives `density`."""
    key = ("row_activity", shape.name)
    s = O.Shape(images, shape.hw, shape.hw, shape.c_in, shape.c_out, 3, 3, shape.stride, 1, shape.groups)
    x = synth.bf16_round(synth.smoothed_noise((key, "x"), images, shape.hw, shape.hw, shape.c_in, rho=rho))
    wb, wc = synth.kaiming_weights(key, shape.c_out, 3, 3, shape.c_in, shape.groups)
    wb, wc = synth.bf16_round(wb), synth.bf16_round(wc)
    bn = synth.bn_params(key, shape.c_out)
    shut = np.full(shape.c_out, np.inf, np.float32)
    p = O.gated_conv(s, x, wb, wc, bn, shut).p.reshape(-1, shape.c_out).astype(np.float64)
    cal = p[: 4 * s.ho * s.wo]
    mean, var = cal.mean(0), np.maximum(cal.var(0), 1e-6)
    p_hat = (p - mean) / np.sqrt(var + s.bn_eps)
    delta = np.quantile(p_hat[: 4 * s.ho * s.wo], 1.0 - density)
    return p_hat >= delta


def activity(d, n_block):
    """(row activity, idle 128-row blocks) of decisions d [pixels, channels] for column blocks of
    n_block channels."""
    m, c = d.shape
    blocks = d[:, : c - c % n_block].reshape(m, -1, n_block).any(2)          # [pixels, column blocks]
    rows = blocks.mean()
    t = m - m % TILE_ROWS
    idle = 1.0 - blocks[:t].reshape(-1, TILE_ROWS, blocks.shape[1]).any(1).mean()
    return rows, idle


def by_firing_rate(d_cal):
    """Static order of the output channels: most active first (from calibration decisions)."""
    return np.argsort(-d_cal.mean(0), kind="stable")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--images", type=int, default=8)
    ap.add_argument("--layers", default="c64@56,c128@28,c256@14,c512@7")
    args = ap.parse_args()
    keep = set(args.layers.split(","))
    shapes = [s for s in synth.imagenet_resnet18_layers(args.images, 4, transitions=False) if s.name in keep]
    print("| layer | rho | density | order | " + " | ".join(f"rows N={n}" for n in BLOCKS) + " | " +
          " | ".join(f"idle N={n}" for n in BLOCKS) + " |")
    print("|---|---|---|---|" + "---|" * (2 * len(BLOCKS)))
    for sh in shapes:
        for rho in (0.0, 0.5):
            for density in (0.1, 0.3):
                d = masks_for(sh, args.images, density, rho)
                hw = d.shape[0] // args.images
                perm = by_firing_rate(d[: 4 * hw])
                for label, dd in (("as generated", d), ("by firing rate", d[:, perm])):
                    cells = [activity(dd, n) for n in BLOCKS if n <= sh.c_out]
                    pad = [""] * (len(BLOCKS) - len(cells))
                    print(f"| {sh.name} | {rho} | {d.mean():.3f} | {label} | " +
                          " | ".join([f"{r:.3f}" for r, _ in cells] + pad) + " | " +
                          " | ".join([f"{i:.3f}" for _, i in cells] + pad) + " |")
                iid = [1.0 - (1.0 - d.mean()) ** n for n in BLOCKS]
                print(f"| {sh.name} | - | {d.mean():.3f} | independent gates | " +
                      " | ".join(f"{v:.3f}" for v in iid) + " | " + " | ".join(["0.000"] * len(BLOCKS)) + " |")


if __name__ == "__main__":
    main()
