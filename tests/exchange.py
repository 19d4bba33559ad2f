"""Test helper: what the network would do between pack and unpack, in numpy.

Every source rank's staged buffer holds, for each step k, the rows it sends in that step at send_off[k][i];
the destination of that chunk is lane_dst[k][i] and it lands at recv_off[k][dst] of the destination's
receive buffer (Section 5: one contiguous transfer per peer and step).  Returns the receive buffer of
``rank`` and the same movement applied to any per-row metadata.
"""
import numpy as np


def deliver(plan: dict, rank: int, staged_by_src, row_bytes: int, meta_by_src=None):
    K = int(plan["n_steps"])
    R = int(plan["recv_off"][K][rank]) // row_bytes
    width = next(iter(staged_by_src.values())).shape[1] if staged_by_src else 0
    recv = np.zeros((R, width), np.uint8)
    meta = np.full(R, -1, np.int32)
    for k in range(K):
        for i, staged in staged_by_src.items():
            if plan["lane_dst"][k][i] != rank:
                continue
            n = int(plan["lane_bytes"][k][i]) // row_bytes
            s0 = int(plan["send_off"][k][i]) // row_bytes
            r0 = int(plan["recv_off"][k][rank]) // row_bytes
            recv[r0:r0 + n] = staged[s0:s0 + n]
            if meta_by_src is not None:
                meta[r0:r0 + n] = meta_by_src[i][s0:s0 + n]
    return recv, meta
