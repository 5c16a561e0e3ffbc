"""GPU parity on model-shaped workloads: every benchmark configuration at a reduced batch (all
layers, compared tensor by tensor with the CPU oracle) and the benchmark's own full-size
configuration in the launch configuration bench.py times (sampled layers computed by the oracle,
plus properties that hold for every tensor)."""
import ctypes as C
import math

import numpy as np
import pytest
import torch

import gen
import oracle
import paper_2501_07161_b200 as q
from parity import MSE_RTOL, SQNR_ATOL_DB, assert_metric_close, bits

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = q.Context(0)
    yield c
    c.close()


def _np(t):
    return t.detach().cpu().numpy()


def oracle_layer_jobs(model, layer_ids=None, act_per_channel=False):
    """Oracle jobs in the library's descriptor order: weights, activations, extra weight scorings."""
    cfg = model.config
    layers = model.layers if layer_ids is None else [model.layers[i] for i in layer_ids]
    pct = cfg.a_percentile if cfg.a_range == "percentile" else None
    jobs = []
    for l in layers:
        jobs.append(dict(x=_np(l.w).reshape(-1), y=None, outer=1, channels=l.w.shape[0], inner=l.w.shape[1],
                         per_channel=cfg.w_granularity[0] == "channel", asym_u8=False))
    for l in layers:
        b, c, hw = l.x.shape
        jobs.append(dict(x=_np(l.x).reshape(-1), y=_np(l.y).reshape(-1), outer=b, channels=c, inner=hw,
                         per_channel=act_per_channel, asym_u8=True, percentile=pct,
                         group_percentile=act_per_channel))
    for g in cfg.w_granularity[1:]:
        for l in layers:
            jobs.append(dict(x=_np(l.w).reshape(-1), y=None, outer=1, channels=l.w.shape[0],
                             inner=l.w.shape[1], per_channel=g == "channel", asym_u8=False))
    return jobs


def py_scores(sw, mw, sa, ma, wg=2.0, ag=1.0, cap=200.0):
    cl = lambda v: max(-cap, min(cap, v))
    n = len(sw)
    sc = [0.0] + [wg * (cl(sw[i]) - cl(sw[i - 1])) + ag * (cl(sa[i]) - cl(sa[i - 1])) for i in range(1, n)]
    mean_w, mean_a = sum(mw) / n, sum(ma) / n
    sev = [max(mw[i] / mean_w if mean_w > 0 else 0.0, ma[i] / mean_a if mean_a > 0 else 0.0) for i in range(n)]
    return sc, sev


def run_sweep(ctx, model, act_granularity="tensor"):
    md = q.model_descs(model, act_granularity=act_granularity)
    cfg = q.default_rank_cfg(select_mode=q.BY_BOPS_RATE, rate_permyriad=md.rate_permyriad)
    sb, t = ctx.alloc_sweep_buffers(md.descs, md.n_layers)
    ctx.sweep_model(md.descs, md.n_layers, md.macs, None, cfg, sb)
    torch.cuda.synchronize()
    return md, t


def compare_tensor(t, idx, g0, ref, name, check_hist):
    ng = ref.step.size
    for field in ("gmin", "gmax", "gabsmax", "step", "inv", "offset"):
        got = t[field][g0:g0 + ng].cpu().numpy()
        assert np.array_equal(bits(got), bits(getattr(ref, field))), f"{name}: {field}"
    assert int(t["nonfinite"][idx]) == 0 == ref.nonfinite
    assert bits(t["clip"][idx:idx + 1].cpu().numpy())[0] == bits([ref.clip])[0], f"{name}: clip"
    h = t["hist"].cpu().numpy().view(np.uint64).reshape(-1, 2048)[idx]
    if check_hist:
        assert np.array_equal(h, ref.hist), f"{name}: hist"
    else:
        assert not h.any()
    assert_metric_close(float(t["mse"][idx]), float(t["sqnr_db"][idx]), ref.mse, ref.sqnr_db, name)


@pytest.mark.parametrize("name,batch", [("resnet18", 3), ("mobilenetv2", 2), ("squeezenet", 1)])
def test_model_sweep_with_per_channel_activations_matches_oracle(ctx, name, batch):
    """The per-channel variant of the activation quantizer over whole models: every channel of every
    layer its own range and, where the configuration clips, its own histogram and clip."""
    model = gen.make_model(name, seed=3, device="cuda", batch=batch)
    md, t = run_sweep(ctx, model, act_granularity="channel")
    refs = oracle.sweep_tensors(oracle_layer_jobs(model, act_per_channel=True), threads=8)
    g0 = 0
    for idx, ref in enumerate(refs):
        compare_tensor(t, idx, g0, ref, f"{name}[{idx}] per-channel activations", check_hist=ref.hist is not None)
        g0 += ref.step.size
    assert g0 == int(q.lib().qv2_group_count(md.descs, md.n_tensors))


@pytest.mark.parametrize("name,batch", [("squeezenet", 1), ("resnet18", 2), ("resnet50", 1),
                                        ("mobilenetv2", 1), ("vgg16", 1)])
def test_model_sweep_matches_oracle(ctx, name, batch):
    model = gen.make_model(name, seed=0, device="cuda", batch=batch)
    md, t = run_sweep(ctx, model)
    refs = oracle.sweep_tensors(oracle_layer_jobs(model), threads=8)
    L = md.n_layers
    g0 = 0
    for idx, ref in enumerate(refs):
        compare_tensor(t, idx, g0, ref, f"{name}[{idx}]", check_hist=ref.hist is not None)
        g0 += ref.step.size
    # ranking: the kernel is a bit-exact function of ITS metrics ...
    mse, sq = t["mse"].cpu().numpy(), t["sqnr_db"].cpu().numpy()
    macs = md.macs.cpu().numpy().astype(np.uint64)
    o_gpu = t["order"].cpu().numpy().view(np.uint32).tolist()
    k_gpu = t["keep_fp32"].cpu().numpy().tolist()
    ro, rk, rn = oracle.rank_layers(sq[:L], mse[:L], sq[L:2 * L], mse[L:2 * L], macs=macs,
                                    select_mode=1, rate_permyriad=md.rate_permyriad)
    assert o_gpu == ro.tolist() and k_gpu == rk.tolist() and int(t["n_keep"][0]) == rn
    assert sorted(o_gpu) == list(range(L))
    # ... and end to end it equals the oracle's list unless two scores (or a severity and the 5x
    # threshold) are closer than the metric tolerance allows to separate
    sw = [r.sqnr_db for r in refs[:L]]; mw = [r.mse for r in refs[:L]]
    sa = [r.sqnr_db for r in refs[L:2 * L]]; ma = [r.mse for r in refs[L:2 * L]]
    eo, ek, en = oracle.rank_layers(sw, mw, sa, ma, macs=macs, select_mode=1,
                                    rate_permyriad=md.rate_permyriad)
    if o_gpu != eo.tolist():
        sc, sev = py_scores(sw, mw, sa, ma)
        band = 6 * SQNR_ATOL_DB
        srt = sorted(sc)
        gap = min(b - a for a, b in zip(srt, srt[1:]))
        margin = min(abs(s - 5.0) for s in sev)
        assert gap < band or margin < 1e-4, f"order differs with score gap {gap} and margin {margin}"
    else:
        assert k_gpu == ek.tolist()


def test_host_buffer_entry_point_matches_device_sweep(ctx):
    model = gen.make_model("squeezenet", seed=3, device="cuda", batch=1)
    md, t = run_sweep(ctx, model)
    host = gen.make_model("squeezenet", seed=3, device="cuda", batch=1)
    for l in host.layers:                                  # same bytes, now in pinned host memory
        l.w, l.x, l.y = (a.cpu().pin_memory() for a in (l.w, l.x, l.y))
    hd = q.model_descs(host, host=True)
    staging = torch.empty(q.binding.staging_bytes(hd.descs, hd.n_layers), dtype=torch.uint8, device="cuda")
    sb, t2 = ctx.alloc_sweep_buffers(hd.descs, hd.n_layers)
    n, L = hd.n_tensors, hd.n_layers
    out = dict(mse=np.zeros(n), sqnr_db=np.zeros(n), nonfinite=np.zeros(n, np.uint64),
               order=np.zeros(L, np.uint32), keep_fp32=np.zeros(L, np.uint8), n_keep=np.zeros(1, np.uint32))
    hr = q.binding.HostResults(**{k: v.ctypes.data for k, v in out.items()})
    cfg = q.default_rank_cfg(select_mode=q.BY_BOPS_RATE, rate_permyriad=hd.rate_permyriad)
    st = ctx.sweep_model_host(hd.descs, L, hd.macs, None, cfg, staging, sb, hr)
    assert st == 0
    assert np.array_equal(out["mse"].view(np.uint64), t["mse"].cpu().numpy().view(np.uint64))
    assert np.array_equal(out["sqnr_db"].view(np.uint64), t["sqnr_db"].cpu().numpy().view(np.uint64))
    assert out["order"].tolist() == t["order"].cpu().numpy().view(np.uint32).tolist()
    assert out["keep_fp32"].tolist() == t["keep_fp32"].cpu().numpy().tolist()
    assert int(out["n_keep"][0]) == int(t["n_keep"][0])
    # a NaN in a host tensor is reported through the status
    host.layers[2].x[0, 0, 0] = float("nan")
    st = ctx.sweep_model_host(hd.descs, L, hd.macs, None, cfg, staging, sb, hr)
    assert st == -5 and out["nonfinite"][L + 2] == 1


def test_full_size_benchmark_workload_sampled_against_oracle(ctx):
    """The benchmark's workload (VGG-16 shapes, batch 64, ~7.5 GB resident) run exactly as bench.py
    runs it; four layers -- among them the largest activation and the largest weight tensor -- are
    copied back and recomputed by the oracle; every tensor is checked through invariants."""
    name = "vgg16"
    free, _ = torch.cuda.mem_get_info()
    if free < 24 * 2 ** 30:
        pytest.skip("needs about 24 GiB of free device memory")
    model = gen.make_model(name, seed=0, device="cuda")
    md, t = run_sweep(ctx, model)
    L = md.n_layers
    sample = [0, 6, 13, 15]
    jobs = oracle_layer_jobs(model, sample)
    refs = oracle.sweep_tensors(jobs, threads=len(jobs))
    group_base = np.concatenate([[0], np.cumsum([l.w.shape[0] for l in model.layers] + [1] * L)])
    for j, li in enumerate(sample):
        compare_tensor(t, li, int(group_base[li]), refs[j], f"{name}.w[{li}]", False)
        compare_tensor(t, L + li, int(group_base[L + li]), refs[len(sample) + j], f"{name}.a[{li}]", True)
    hist = t["hist"].cpu().numpy().view(np.uint64).reshape(-1, 2048)
    mse, sq = t["mse"].cpu().numpy(), t["sqnr_db"].cpu().numpy()
    for i, l in enumerate(model.layers):
        assert int(hist[L + i].sum()) == l.x.numel()            # every element lands in one bin
        assert not hist[i].any()
        assert np.isfinite(sq[i]) and np.isfinite(sq[L + i]) and mse[i] > 0 and mse[L + i] > 0
        assert 20.0 < sq[i] < 60.0                               # 8-bit per-channel weights
        clip = float(t["clip"][L + i]); am = float(t["gabsmax"][int(group_base[L + i])])
        assert 0 < clip <= am
        # identity: SQNR == 10 log10(SIG / (N * MSE))
        n = l.x.numel()
        assert abs(sq[L + i] - 10 * math.log10(float(t["sig"][L + i]) / (n * mse[L + i]))) < 1e-9
    o = t["order"].cpu().numpy().view(np.uint32).tolist()
    assert sorted(o) == list(range(L))
    ro, rk, rn = oracle.rank_layers(sq[:L], mse[:L], sq[L:2 * L], mse[L:2 * L],
                                    macs=md.macs.cpu().numpy().astype(np.uint64), select_mode=1,
                                    rate_permyriad=md.rate_permyriad)
    assert o == ro.tolist() and t["keep_fp32"].cpu().numpy().tolist() == rk.tolist()
    # a second pass over the same inputs gives the same bits
    md2, t2 = run_sweep(ctx, model)
    for k in ("sse", "sig", "mse", "sqnr_db"):
        assert torch.equal(t[k].view(torch.int64), t2[k].view(torch.int64))


def test_sweep_can_be_captured_in_a_cuda_graph_and_replayed():
    """Once the tile table of a descriptor set is resident, a pass enqueues only kernels and
    memsets on the context's stream: it can be captured once and replayed (one launch per pass,
    which matters for small models whose pass is launch-bound)."""
    s = torch.cuda.Stream()
    gctx = q.Context(0, stream=s)
    try:
        model = gen.make_model("squeezenet", seed=5, device="cuda", batch=1)
        md = q.model_descs(model)
        cfg = q.default_rank_cfg(select_mode=q.BY_BOPS_RATE, rate_permyriad=md.rate_permyriad)
        sb, t = gctx.alloc_sweep_buffers(md.descs, md.n_layers)
        torch.cuda.synchronize()
        with torch.cuda.stream(s):
            gctx.sweep_model(md.descs, md.n_layers, md.macs, None, cfg, sb)     # warm-up: builds the plan
        s.synchronize()
        ref = {k: t[k].clone() for k in ("mse", "sqnr_db", "order", "keep_fp32", "n_keep", "step", "hist")}
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            gctx.sweep_model(md.descs, md.n_layers, md.macs, None, cfg, sb)
        for k in ("mse", "sqnr_db", "order", "step", "hist"):
            t[k].zero_()
        g.replay()
        torch.cuda.synchronize()
        for k, v in ref.items():
            assert torch.equal(t[k].view(torch.uint8), v.view(torch.uint8)), k
        # new inputs, same buffers: the replay recomputes everything
        model.layers[3].x.mul_(1.5)
        g.replay()
        torch.cuda.synchronize()
        with torch.cuda.stream(s):
            sb2, t2 = gctx.alloc_sweep_buffers(md.descs, md.n_layers)
            gctx.sweep_model(md.descs, md.n_layers, md.macs, None, cfg, sb2)
        torch.cuda.synchronize()
        assert torch.equal(t["mse"].view(torch.int64), t2["mse"].view(torch.int64))
        assert not torch.equal(t["mse"].view(torch.int64), ref["mse"].view(torch.int64))
    finally:
        gctx.close()


def test_two_contexts_on_two_streams_do_not_interfere():
    """The library keeps no global state besides per-kernel occupancy caches: two contexts, each on
    its own stream, sweeping different models at the same time give the results each gives alone."""
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    c1, c2 = q.Context(0, stream=s1), q.Context(0, stream=s2)
    try:
        m1 = gen.make_model("squeezenet", seed=11, device="cuda", batch=2)
        m2 = gen.make_model("resnet18", seed=12, device="cuda", batch=1)
        torch.cuda.synchronize()
        alone = []
        for c, s, m in ((c1, s1, m1), (c2, s2, m2)):
            with torch.cuda.stream(s):
                md, t = run_sweep(c, m)
            alone.append({k: t[k].clone() for k in ("mse", "sqnr_db", "order", "step", "clip")})
        runs = []
        for _ in range(3):                              # interleave launches of the two streams
            with torch.cuda.stream(s1):
                md1 = q.model_descs(m1); sb1, t1 = c1.alloc_sweep_buffers(md1.descs, md1.n_layers)
            with torch.cuda.stream(s2):
                md2 = q.model_descs(m2); sb2, t2 = c2.alloc_sweep_buffers(md2.descs, md2.n_layers)
            torch.cuda.synchronize()
            cfg1 = q.default_rank_cfg(select_mode=q.BY_BOPS_RATE, rate_permyriad=md1.rate_permyriad)
            cfg2 = q.default_rank_cfg(select_mode=q.BY_BOPS_RATE, rate_permyriad=md2.rate_permyriad)
            c1.sweep_model(md1.descs, md1.n_layers, md1.macs, None, cfg1, sb1)
            c2.sweep_model(md2.descs, md2.n_layers, md2.macs, None, cfg2, sb2)
            c1.sweep_model(md1.descs, md1.n_layers, md1.macs, None, cfg1, sb1)
            c2.sweep_model(md2.descs, md2.n_layers, md2.macs, None, cfg2, sb2)
            torch.cuda.synchronize()
            runs.append((t1, t2))
        for t1, t2 in runs:
            for ref, t in ((alone[0], t1), (alone[1], t2)):
                for k, v in ref.items():
                    assert torch.equal(t[k].view(torch.uint8), v.view(torch.uint8)), k
    finally:
        c1.close(); c2.close()


def test_library_sweep_graph_replays_the_pass():
    """qv2_sweep_graph_create / _launch: same bits as the ordinary call, new inputs picked up in
    place, and the default-stream context is refused."""
    s = torch.cuda.Stream()
    gctx = q.Context(0, stream=s)
    dctx = q.Context(0)                                   # torch's default stream: cannot be captured
    try:
        model = gen.make_model("squeezenet", seed=8, device="cuda", batch=1)
        md = q.model_descs(model)
        cfg = q.default_rank_cfg(select_mode=q.BY_BOPS_RATE, rate_permyriad=md.rate_permyriad)
        torch.cuda.synchronize()
        with torch.cuda.stream(s):
            sb, t = gctx.alloc_sweep_buffers(md.descs, md.n_layers)
            sb_ref, t_ref = gctx.alloc_sweep_buffers(md.descs, md.n_layers)
            m0 = gctx.launches
            gctx.sweep_model(md.descs, md.n_layers, md.macs, None, cfg, sb_ref)
            per_pass = gctx.launches - m0                  # range + fold, metrics + fold, rank: no clearing launch, no histogram pass
            g = gctx.sweep_graph(md.descs, md.n_layers, md.macs, None, cfg, sb)
            n0 = gctx.launches
            for k in ("mse", "sqnr_db", "order", "hist"):
                t[k].zero_()
            g.launch()
            s.synchronize()
            assert gctx.launches - n0 == per_pass == 5
            for k in ("mse", "sqnr_db", "order", "keep_fp32", "n_keep", "step", "hist", "clip"):
                assert torch.equal(t[k].view(torch.uint8), t_ref[k].view(torch.uint8)), k
            model.layers[5].x.mul_(0.5)                   # refill a tensor in place
            g.launch(); g.launch()
            gctx.sweep_model(md.descs, md.n_layers, md.macs, None, cfg, sb_ref)
            s.synchronize()
            assert torch.equal(t["mse"].view(torch.int64), t_ref["mse"].view(torch.int64))
            g.close()
        sb2, _ = dctx.alloc_sweep_buffers(md.descs, md.n_layers)
        if torch.cuda.current_stream().cuda_stream == 0:
            with pytest.raises(q.binding.Qv2Error) as e:
                dctx.sweep_graph(md.descs, md.n_layers, md.macs, None, cfg, sb2)
            assert e.value.status == -8
    finally:
        gctx.close(); dctx.close()
