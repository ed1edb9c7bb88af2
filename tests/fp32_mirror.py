"""fp32 mirror of the aggregator's arithmetic, for the tests only.

The aggregator (Sec. 3.3) is p <- sum_i p_i 1[p in W_i] / sum_i 1[p in W_i].  The oracle evaluates it in float64; the
CUDA path evaluates it in float32 with a fixed order: running sum over the covering subnets in ascending subnet
index, then one IEEE division by the count.  This module writes that float32 evaluation out with numpy scalars'
IEEE arithmetic, so that a GPU result can be required to match it bit for bit.  tests/test_oracle_math.py ties
the mirror to the float64 oracle (within the rounding of count float32 operations); it shares no code with
either side.
"""
import numpy as np


def aggregate_f32(W_full, subs, blueprints, block_rows, live_mask=None, row_offset=0):
    """W_full [rows, d]; subs[s] [n_sub * block_rows, d]; blueprints[s] kept block ids (ascending).
    Returns the float32 result; rows held by no live subnet keep W_full's value."""
    out = np.array(W_full, dtype=np.float32, copy=True)
    acc = np.zeros_like(out)
    cnt = np.zeros(out.shape[0], dtype=np.int64)
    for s, (sub, blocks) in enumerate(zip(subs, blueprints)):           # ascending s
        if live_mask is not None and not (live_mask >> s) & 1:
            continue
        blocks = np.asarray(blocks, dtype=np.int64)
        rows = (row_offset + blocks[:, None] * block_rows + np.arange(block_rows)[None, :]).reshape(-1)
        acc[rows] = acc[rows] + np.asarray(sub, dtype=np.float32)[: len(rows)]      # float32 addition
        cnt[rows] += 1
    held = cnt > 0
    out[held] = acc[held] / cnt[held].astype(np.float32)[:, None]                  # float32 division
    return out
