"""Static reordering of a gated layer's output channels (model preparation, host side).

A kernel that works on blocks of output channels can skip a block only when no gate in it fires
(Eq. 1, second case).  Which channel sits in which block is free: relabelling the output
channels of a layer, and the input channels of the layer that consumes them, leaves the network
unchanged.  Putting the channels whose gates fire most often next to each other concentrates the
open gates in few column blocks.

The order is fixed before inference (from the gate decisions of calibration images); nothing
here runs per batch.  All arrays are numpy, channel-last.
"""
from __future__ import annotations

import numpy as np


def unpack_mask(mask_words: np.ndarray, c_out: int) -> np.ndarray:
    """mask_out words [pixels, ceil(c_out/32)] -> decisions [pixels, c_out] (bit c%32 of word c/32)."""
    w = np.ascontiguousarray(mask_words).view(np.uint32)
    bits = (w[:, :, None] >> np.arange(32, dtype=np.uint32)) & np.uint32(1)
    return bits.reshape(w.shape[0], -1)[:, :c_out].astype(bool)


def order_by_firing_rate(decisions: np.ndarray) -> np.ndarray:
    """perm such that new channel j is old channel perm[j]; most active channels first (stable)."""
    return np.argsort(-np.asarray(decisions, np.float64).mean(0), kind="stable")


def permute_output_channels(w_base, w_cond, per_channel: dict, perm):
    """The producing layer with its output channels reordered: filter rows and every per-channel
    vector (gamma, beta, statistics, Delta, ...) are gathered by perm."""
    perm = np.asarray(perm)
    return (np.ascontiguousarray(w_base[perm]), np.ascontiguousarray(w_cond[perm]),
            {k: (None if v is None else np.ascontiguousarray(np.asarray(v)[perm])) for k, v in per_channel.items()})


def permute_input_channels(w_full, perm, groups):
    """The consuming layer reading the reordered tensor: its filter [c_out,kh,kw,c_in] over ALL
    input channels is gathered by perm, then split again into base (first c_in/G channels of the
    new order, Section 3.1) and conditional part.  The split moves with the order: the base path of
    the consumer reads whichever channels now come first."""
    w = np.ascontiguousarray(np.asarray(w_full)[..., np.asarray(perm)])
    cp = w.shape[-1] // groups
    return np.ascontiguousarray(w[..., :cp]), np.ascontiguousarray(w[..., cp:])
