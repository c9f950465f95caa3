"""Per-warp timeline of the default split-KV kernel on the 64K-context workload (a diagnostic, not part of the path).

    python -m paper_2602_11937_b200.timeline            (from the repository root, on a B200)

Builds the library a second time with -DPUZZLE_TIMELINE (lib/libpuzzle_attn_timeline.so: every warp of the FP8
kernel stamps %globaltimer at kernel entry, when its first tile has landed and when it leaves its tile loop, and
notes its SM), runs a few launches on different seeded caches and prints where the launch time goes: the set-up
before the first tile, the spread of the finishing times, how much of it belongs to the SM (systematic) and how
much to the worker's place in the schedule.
"""
from __future__ import annotations

import ctypes
import os
import sys


def main() -> None:
    from . import build
    from . import binding as B
    assert B._lib is None, "the library is already loaded"
    B._LIB_PATH = build.build_timeline()        # this process uses the instrumented build
    import numpy as np
    import torch

    import synth
    from synth.device import fill_layer

    dev = "cuda:0"
    w = synth.workload(3)                       # batch 16, context 65536, paged random table
    seq = torch.full((w.batch,), w.context, dtype=torch.int32, device=dev)
    desc = B.layer_desc()
    q, sinks = synth.draw_q(w, 0, dev), synth.draw_sinks(w, 0, dev)
    out = torch.empty(w.batch, w.hq, w.head_dim, dtype=torch.bfloat16, device=dev)
    ws = torch.zeros(B.puzzle_decode_attn_workspace_bytes(desc, w.batch, 0), dtype=torch.uint8, device=dev)
    B.puzzle_decode_attn_workspace_init(desc, w.batch, ws)
    lib = B._load()
    n_warps = torch.cuda.get_device_properties(0).multi_processor_count * 12

    def launch(view):
        B.puzzle_decode_attn(desc, view, q, sinks, out, None, workspace=ws)
        torch.cuda.synchronize()
        buf = np.zeros(4096 * 4, dtype=np.uint64)
        assert lib.puzzle_debug_timeline(buf.ctypes.data_as(ctypes.c_void_p)) == 0
        t = buf.reshape(4096, 4)[:n_warps].astype(np.int64)
        t0 = t[:, 0].min()
        return (t[:, 0] - t0) / 1e3, (t[:, 1] - t0) / 1e3, (t[:, 2] - t0) / 1e3, t[:, 3]

    per_sm, dev_in_cta = [], []
    for layer in range(3):
        L = fill_layer(w, layer, dev)
        view = B.kv_view(L["k_cache"], L["v_cache"], seq, block_table=L["table"], max_blocks_per_seq=w.blocks_per_seq,
                         k_scale=L["k_scale"], v_scale=L["v_scale"])
        for _ in range(2):
            launch(view)
        for rep in range(2):
            start, first, end, smid = launch(view)
            cta = end.reshape(-1, 12)[:-1]                     # the last CTA has a shorter share
            sm = np.zeros(int(smid.max()) + 1)
            sm[smid.reshape(-1, 12)[:-1, 0]] = cta.mean(axis=1)
            per_sm.append(sm)
            dev_in_cta.append((cta - cta.mean(axis=1, keepdims=True)).reshape(-1))
            if rep == 0:
                print("cache %d: CTAs start within %.1f us; first tile landed: median %.1f, latest %.1f us; tile loop left: "
                      "median %.1f, latest %.1f us; per-SM mean %.1f .. %.1f (sigma %.1f); range inside an SM (median) %.1f us"
                      % (layer, start.max(), np.median(first), first.max(), np.median(end), end.max(),
                         sm[sm > 0].min(), sm.max(), sm[sm > 0].std(), np.median(cta.max(axis=1) - cta.min(axis=1))))
        del L, view
    c = lambda a, b: float(np.corrcoef(a, b)[0, 1])
    print("per-SM means, correlation between launches on different caches: %.2f %.2f" % (c(per_sm[0], per_sm[2]), c(per_sm[2], per_sm[4])))
    print("a warp's finish relative to its CTA's mean (sigma %.1f us): correlation between two launches on the same cache "
          "%.2f %.2f, on different caches %.2f %.2f" % (dev_in_cta[0].std(), c(dev_in_cta[0], dev_in_cta[1]), c(dev_in_cta[2], dev_in_cta[3]),
                                                       c(dev_in_cta[0], dev_in_cta[2]), c(dev_in_cta[1], dev_in_cta[4])))
    mean_dev = sum(dev_in_cta) / len(dev_in_cta)
    wid = np.arange(mean_dev.size)
    T = w.batch * w.hkv * (w.context // 64)
    qrun = (T + n_warps - 1) // n_warps
    per_pair = w.context // 64
    cross = (wid * qrun) // per_pair != ((wid + 1) * qrun - 1) // per_pair
    print("workers whose run crosses a (sequence, KV head) boundary: %d, %.1f us later than their CTA's mean on average "
          "(the others %.1f us)" % (int(cross.sum()), mean_dev[cross].mean(), mean_dev[~cross].mean()))


if __name__ == "__main__":
    sys.exit(main())
