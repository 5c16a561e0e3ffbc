"""Writes tests/golden/oracle_small.json from the CPU oracle alone.

The paper prints no worked numeric example (no scale, code, MSE, SQNR or list for any tensor), so
there is no published value to store.  This fixture instead freezes the ORACLE's results on three
tiny deterministic tensors, so that an accidental change of the oracle's arithmetic shows up as a
diff of a committed text file, and so that the CUDA path can be checked against stored values as
well as against a live oracle run.  Inputs come from integer arithmetic only (a 32-bit LCG), never
from a library random generator, so every platform regenerates the same bytes.

    python tests/golden/make_golden.py        # rewrites the fixture
"""
import json
import os
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))
import oracle  # noqa: E402


def lcg_floats(n, seed, scale):
    """n floats in [-scale, scale): 32-bit LCG (a = 1664525, c = 1013904223), top 24 bits."""
    out = np.empty(n, np.float32)
    s = seed & 0xFFFFFFFF
    for i in range(n):
        s = (1664525 * s + 1013904223) & 0xFFFFFFFF
        out[i] = np.float32(((s >> 8) - (1 << 23)) / float(1 << 23) * scale)
    return out


def cases():
    w = lcg_floats(6 * 50, 1, 0.25).reshape(6, 50)
    w *= np.float32([1, 2, 0.5, 4, 1, 0.25])[:, None]            # per-channel spread
    x = np.maximum(lcg_floats(3000, 2, 3.0), 0)                   # post-ReLU activation
    y = (x + lcg_floats(3000, 3, 0.02)).astype(np.float32)
    g = lcg_floats(2 * 3 * 200, 4, 1.5)                           # [2][3][200], signed
    return [
        dict(name="weights_per_channel_sym", x=w.reshape(-1), y=None, outer=1, channels=6, inner=50,
             per_channel=True, asym_u8=False, percentile=None),
        dict(name="relu_act_pair_percentile", x=x, y=y, outer=1, channels=1, inner=3000,
             per_channel=False, asym_u8=True, percentile=0.99),
        dict(name="signed_act_per_channel_asym", x=g, y=None, outer=2, channels=3, inner=200,
             per_channel=True, asym_u8=True, percentile=None),
        dict(name="signed_act_per_channel_own_percentile", x=g * np.float32([1, 8, 0.125]).repeat(200)[None, :].repeat(2, 0).reshape(-1),
             y=None, outer=2, channels=3, inner=200, per_channel=True, asym_u8=True, percentile=0.95,
             group_percentile=True),
    ]


def hexf(a):
    return [float(v).hex() for v in np.asarray(a, np.float64).reshape(-1)]


def compute():
    out = {"_about": "values computed by oracle/ (see make_golden.py); the paper prints no worked example",
           "tensors": []}
    for c in cases():
        kw = {k: c[k] for k in ("x", "y", "outer", "channels", "inner", "per_channel", "asym_u8", "percentile")}
        r = oracle.sweep_tensor(want_codes=True, group_percentile=c.get("group_percentile", False), **kw)
        mode = oracle.PAIR_SELF if c["y"] is None else oracle.PAIR_REQUANT
        cos = oracle.cosine(c["x"], c["y"], c["outer"], c["channels"], c["inner"], c["per_channel"],
                            c["asym_u8"], mode, r.step, r.inv, r.offset)
        out["tensors"].append(dict(
            name=c["name"], gmin=hexf(r.gmin), gmax=hexf(r.gmax), step=hexf(r.step), inv=hexf(r.inv),
            offset=hexf(r.offset), clip=float(r.clip).hex(),
            hist_nonzero=[] if r.hist is None else [[int(i), int(v)] for i, v in enumerate(r.hist) if v],
            codes_head=[int(v) for v in r.codes[:40]], codes_sum=int(r.codes.astype(np.int64).sum()),
            sse=float(r.sse).hex(), sig=float(r.sig).hex(), mse=float(r.mse).hex(),
            sqnr_db=float(r.sqnr_db).hex(), cosine=float(cos).hex(),
            group_clip=hexf(r.gclip),
            group_hist_nonzero=[] if r.ghist is None else
            [[int(g), int(i), int(v)] for g in range(r.ghist.shape[0]) for i, v in enumerate(r.ghist[g]) if v]))
    sw = [41.5, 38.25, 39.0, 33.75, 40.5, 36.0, 37.5]
    sa = [30.0, 29.5, 31.25, 27.0, 28.5, 30.75, 26.0]
    mw = [1e-6, 2e-6, 1e-6, 9e-6, 1e-6, 1e-6, 2e-6]
    ma = [1e-3, 1e-3, 2e-3, 4e-2, 1e-3, 1e-3, 1e-3]
    macs = [118013952, 115605504, 115605504, 57802752, 115605504, 25690112, 512000]
    o, k, nk = oracle.rank_layers(sw, mw, sa, ma, macs=macs, select_mode=1, rate_permyriad=6000)
    fo, fk, fnk = oracle.rank_layers_fused(sw, mw, sa, ma, [0, 0, 0xFFFFFFFF, 1, 1, 0xFFFFFFFF, 0xFFFFFFFF],
                                           macs=macs, select_mode=1, rate_permyriad=6000)
    out["rank"] = dict(sqnr_w=sw, sqnr_a=sa, mse_w=mw, mse_a=ma, macs=macs, rate_permyriad=6000,
                       fuse_group=[0, 0, 0xFFFFFFFF, 1, 1, 0xFFFFFFFF, 0xFFFFFFFF],
                       order=o.tolist(), keep=k.tolist(), n_keep=nk,
                       fused_order=fo.tolist(), fused_keep=fk.tolist(), fused_n_keep=fnk)
    return out


if __name__ == "__main__":
    with open(os.path.join(HERE, "oracle_small.json"), "w") as f:
        json.dump(compute(), f, separators=(",", ":"))
        f.write("\n")
    print("wrote oracle_small.json")
