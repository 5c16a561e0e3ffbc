"""Stored expected values (tests/golden/oracle_small.json, written by tests/golden/make_golden.py
from the oracle alone): the oracle must still reproduce them bit for bit, and the CUDA path must
match them -- integers, scales and lists exactly, metrics within the parity tolerances."""
import importlib.util
import json
import os

import numpy as np
import pytest

HERE = os.path.dirname(os.path.abspath(__file__))
GOLD = os.path.join(HERE, "golden", "oracle_small.json")


def _maker():
    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(HERE, "golden", "make_golden.py"))
    m = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(m)
    return m


def test_oracle_reproduces_the_stored_values_exactly():
    stored = json.load(open(GOLD))
    fresh = json.loads(json.dumps(_maker().compute()))
    assert fresh == stored


def test_input_generator_of_the_fixture_is_plain_integer_arithmetic():
    v = _maker().lcg_floats(3, 1, 1.0)
    s = 1
    exp = []
    for _ in range(3):
        s = (1664525 * s + 1013904223) & 0xFFFFFFFF
        exp.append(np.float32(((s >> 8) - (1 << 23)) / float(1 << 23)))
    assert v.tolist() == exp


@pytest.mark.gpu
def test_cuda_path_matches_the_stored_values():
    import torch
    import paper_2501_07161_b200 as q
    stored = json.load(open(GOLD))
    mk = _maker()
    fx = lambda lst: np.array([float.fromhex(h) for h in lst], np.float64)
    ctx = q.Context(0)
    try:
        for c, ref in zip(mk.cases(), stored["tensors"]):
            x = torch.from_numpy(c["x"]).cuda()
            y = None if c["y"] is None else torch.from_numpy(c["y"]).cuda()
            pct = c["percentile"]
            d = q.make_desc(x, y, c["outer"], c["channels"], c["inner"],
                            q.PER_CHANNEL if c["per_channel"] else q.PER_TENSOR,
                            q.ASYM_U8 if c["asym_u8"] else q.SYM_I8,
                            (q.PERCENTILE_GROUP if c.get("group_percentile") else q.PERCENTILE)
                            if pct is not None else q.MINMAX, pct or 0.0, q.STORE_CODES)
            descs = q.desc_array([d])
            cal = ctx.calibrate(descs, want_group=True)
            codes = [torch.zeros(x.numel(), dtype=torch.uint8, device="cuda")]
            met = ctx.quant_metrics(descs, cal.step, cal.inv, cal.offset, codes, want_cosine=True)
            torch.cuda.synchronize()
            for field in ("gmin", "gmax", "step", "inv", "offset"):
                got = getattr(cal, field).cpu().numpy().astype(np.float64)
                assert np.array_equal(got, fx(ref[field])), (c["name"], field)
            assert float(cal.clip[0]) == float.fromhex(ref["clip"])
            hist = cal.hist.cpu().numpy().view(np.uint64)[:2048]
            assert [[int(i), int(v)] for i, v in enumerate(hist) if v] == ref["hist_nonzero"]
            assert np.array_equal(cal.group_clip.cpu().numpy().astype(np.float64), fx(ref["group_clip"])), c["name"]
            if c.get("group_percentile"):
                gh = cal.group_hist.cpu().numpy().view(np.uint64).reshape(-1, 2048)
                got = [[int(g), int(i), int(v)] for g in range(c["channels"]) for i, v in enumerate(gh[g]) if v]
                assert got == ref["group_hist_nonzero"], c["name"]
            cd = codes[0].cpu().numpy()
            cd = cd if c["asym_u8"] else cd.view(np.int8)
            assert cd[:40].tolist() == ref["codes_head"] and int(cd.astype(np.int64).sum()) == ref["codes_sum"]
            mse, sq = float.fromhex(ref["mse"]), float.fromhex(ref["sqnr_db"])
            assert abs(float(met.mse[0]) - mse) <= 1e-5 * mse and abs(float(met.sqnr_db[0]) - sq) <= 1e-3
            assert abs(float(met.cosine[0]) - float.fromhex(ref["cosine"])) <= 1e-7
        r = stored["rank"]
        dv = lambda a, dt: torch.tensor(a, dtype=dt, device="cuda")
        cfg = q.default_rank_cfg(select_mode=q.BY_BOPS_RATE, rate_permyriad=r["rate_permyriad"])
        args = (dv(r["sqnr_w"], torch.float64), dv(r["mse_w"], torch.float64), dv(r["sqnr_a"], torch.float64),
                dv(r["mse_a"], torch.float64), dv(r["macs"], torch.int64), None, cfg)
        o, k, nk = ctx.rank_layers(*args)
        fg = torch.from_numpy(np.array(r["fuse_group"], np.uint32).view(np.int32)).cuda()
        fo, fk, fnk = ctx.rank_layers(*args, fuse_group=fg)
        torch.cuda.synchronize()
        assert o.cpu().numpy().view(np.uint32).tolist() == r["order"] and k.tolist() == r["keep"] and int(nk) == r["n_keep"]
        assert fo.cpu().numpy().view(np.uint32).tolist() == r["fused_order"] and fk.tolist() == r["fused_keep"]
        assert int(fnk) == r["fused_n_keep"]
    finally:
        ctx.close()
