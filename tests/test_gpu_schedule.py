"""GPU tests of the scheduling side of the library: the L2-chunked schedule against the oracle and
against the phase-major schedule, passes that need no clearing launch and no host synchronisation,
captured passes that pin the context's plan, the literal outlier order of Algorithm 2, and Conv+BN
folding in place."""
import ctypes as C
import math

import numpy as np
import pytest
import torch

import gen
import oracle
import paper_2501_07161_b200 as q
from parity import Spec, bits, check_specs
from test_gpu_models import compare_tensor, oracle_layer_jobs

pytestmark = pytest.mark.gpu

INT_FIELDS = ("gmin", "gmax", "gabsmax", "step", "inv", "offset", "hist", "clip", "nonfinite")


def _sweep(ctx, model):
    md = q.model_descs(model)
    cfg = q.default_rank_cfg(select_mode=q.BY_BOPS_RATE, rate_permyriad=md.rate_permyriad)
    sb, t = ctx.alloc_sweep_buffers(md.descs, md.n_layers)
    for v in t.values():
        v.view(torch.uint8).fill_(0xA5)                  # nothing may depend on what the buffers held
    ctx.sweep_model(md.descs, md.n_layers, md.macs, None, cfg, sb)
    torch.cuda.synchronize()
    return md, t


@pytest.mark.parametrize("fold", [q.FOLD_SEPARATE, q.FOLD_FUSED])
@pytest.mark.parametrize("name,batch,chunk", [("resnet18", 2, 4 << 20), ("mobilenetv2", 1, 2 << 20),
                                              ("squeezenet", 1, 1 << 20), ("vgg16", 1, 8 << 20)])
def test_l2_chunked_schedule_matches_oracle_and_phase_major(name, batch, chunk, fold):
    """The chunked schedule (range -> histogram -> metrics stage by stage) gives the oracle's
    results, the same bits as the phase-major schedule for everything that is integer-decided,
    and sums within the metric tolerance; the ranking is a bit-exact function of its metrics."""
    model = gen.make_model(name, seed=0, device="cuda", batch=batch)
    a, b = q.Context(0), q.Context(0)
    try:
        b.set_schedule(q.SCHEDULE_L2_CHUNKED, chunk)
        b.set_fold_mode(fold)
        md, ta = _sweep(a, model)
        _, tb = _sweep(b, model)
        assert a.stages == 1 and b.stages > 3, (a.stages, b.stages)
        for k in INT_FIELDS:
            assert torch.equal(ta[k].view(torch.uint8), tb[k].view(torch.uint8)), k
        refs = oracle.sweep_tensors(oracle_layer_jobs(model), threads=8)
        g0 = 0
        for idx, ref in enumerate(refs):
            compare_tensor(tb, idx, g0, ref, f"{name}[{idx}] chunked", check_hist=ref.hist is not None)
            g0 += ref.step.size
        L = md.n_layers
        mse, sq = tb["mse"].cpu().numpy(), tb["sqnr_db"].cpu().numpy()
        ro, rk, rn = oracle.rank_layers(sq[:L], mse[:L], sq[L:2 * L], mse[L:2 * L],
                                        macs=md.macs.cpu().numpy().astype(np.uint64), select_mode=1,
                                        rate_permyriad=md.rate_permyriad)
        assert tb["order"].cpu().numpy().view(np.uint32).tolist() == ro.tolist() and int(tb["n_keep"][0]) == rn
        # a second chunked pass over the same buffers: identical bits (accumulators were left clean)
        keep = {k: v.clone() for k, v in tb.items()}
        b.sweep_model(md.descs, L, md.macs, None, q.default_rank_cfg(select_mode=q.BY_BOPS_RATE,
                      rate_permyriad=md.rate_permyriad), q.binding.SweepBuffers(**{k: v.data_ptr() for k, v in tb.items()}))
        torch.cuda.synchronize()
        for k in tb:
            assert torch.equal(tb[k].view(torch.uint8), keep[k].view(torch.uint8)), k
        # the three separate calls follow the same plan (calibrate stage by stage, then metrics)
        cal = b.calibrate(md.descs)
        met = b.quant_metrics(md.descs, cal.step, cal.inv, cal.offset)
        torch.cuda.synchronize()
        assert torch.equal(cal.step.view(torch.int32), tb["step"].view(torch.int32)[: cal.step.numel()])
        assert torch.equal(met.sse.view(torch.int64), tb["sse"].view(torch.int64)[: met.sse.numel()])
    finally:
        a.close(); b.close()


def test_schedule_selection():
    """AUTO takes the schedule that measured faster, which on a B200 is phase-major at every size;
    the chunked schedule is there on request and an unknown value is refused."""
    ctx = q.Context(0)
    try:
        big = gen.make_model("squeezenet", seed=1, device="cuda", batch=1)
        ctx.set_schedule(q.SCHEDULE_AUTO, 1 << 20)
        _sweep(ctx, big)
        assert ctx.stages == 1
        ctx.set_schedule(q.SCHEDULE_L2_CHUNKED, 1 << 20)
        _sweep(ctx, big)
        assert ctx.stages > 1
        ctx.set_schedule(q.SCHEDULE_PHASE_MAJOR)
        _sweep(ctx, big)
        assert ctx.stages == 1
        with pytest.raises(q.binding.Qv2Error):
            ctx.set_schedule(7)
    finally:
        ctx.close()


def test_dependent_launch_and_phase_timing_do_not_change_results():
    """Programmatic dependent launch only changes when a kernel may start, and the phase events only
    add markers: every output of a pass is the same bits with either switched on or off, also when
    the pass is replayed from a graph captured with dependent launch on."""
    model = gen.make_model("resnet18", seed=3, device="cuda", batch=1)
    outs = []
    torch.cuda.synchronize()
    stream = torch.cuda.Stream()             # a captured pass needs a non-default stream; torch's fills run on it too
    for dependent in (True, False):
        ctx = q.Context(0, stream=stream)
        try:
          with torch.cuda.stream(stream):
            ctx.set_dependent_launch(dependent)
            md, t = _sweep(ctx, model)
            outs.append({k: v.clone() for k, v in t.items()})
            if dependent:
                cfg = q.default_rank_cfg(select_mode=q.BY_BOPS_RATE, rate_permyriad=md.rate_permyriad)
                g = ctx.sweep_graph(md.descs, md.n_layers, md.macs, None, cfg,
                                    q.binding.SweepBuffers(**{k: v.data_ptr() for k, v in t.items()}))
                for v in t.values():
                    v.view(torch.uint8).fill_(0x5A)
                g.launch(); g.launch()
                torch.cuda.synchronize()
                for k in t:
                    assert torch.equal(t[k].view(torch.uint8), outs[0][k].view(torch.uint8)), ("graph", k)
                with pytest.raises(q.binding.Qv2Error):
                    ctx.set_dependent_launch(False)          # a live captured pass keeps its edges
                g.close()
            # the phase events: same bits, and two positive durations
            ctx.set_phase_timing(True)
            cal = ctx.calibrate(md.descs)
            r_ms, h_ms = ctx.calibrate_phase_ms()
            assert r_ms > 0.0 and h_ms > 0.0
            assert torch.equal(cal.step.view(torch.int32), t["step"].view(torch.int32)[: cal.step.numel()])
            assert torch.equal(cal.hist.view(torch.int64), t["hist"].view(torch.int64)[: cal.hist.numel()])
            ctx.set_phase_timing(False)
            with pytest.raises(q.binding.Qv2Error):
                ctx.calibrate_phase_ms()
        finally:
            ctx.close()
    for k in outs[0]:
        assert torch.equal(outs[0][k].view(torch.uint8), outs[1][k].view(torch.uint8)), k


def test_chunked_schedule_with_empty_tensors_mixed_modes_and_codes():
    """Stage boundaries fall between tensors of every kind; empty tensors are folded by block 0."""
    g = torch.Generator(); g.manual_seed(3)
    r = lambda n: torch.randn(n, generator=g)
    specs = [Spec(r(40000), 1, 1, 40000, asym=True, percentile=0.999),
             Spec(torch.zeros(0), 1, 1, 0, asym=True, percentile=0.99),
             Spec(r(64 * 700), 1, 64, 700, per_channel=True),
             Spec(torch.zeros(0), 1, 4, 0, per_channel=True),
             Spec(r(3 * 9 * 5000), 3, 9, 5000, per_channel=True, asym=True, y=r(3 * 9 * 5000)),
             Spec(r(100000).abs(), 1, 1, 100000, asym=True, percentile=0.9999, y=r(100000).abs()),
             Spec(r(960 * 9), 1, 960, 9, per_channel=True),
             Spec(r(17), 1, 1, 17, zp=True, asym=True)]
    ctx = q.Context(0)
    try:
        ctx.set_schedule(q.SCHEDULE_L2_CHUNKED, 256 << 10)
        check_specs(ctx, specs)
        assert ctx.stages >= 4
    finally:
        ctx.close()


@pytest.mark.parametrize("fold,per_phase", [(q.FOLD_FUSED, 1), (q.FOLD_SEPARATE, 2), (q.FOLD_AUTO, 2)])
def test_steady_state_passes_never_synchronise_and_need_no_clearing_launch(fold, per_phase):
    """After the first call of a descriptor set nothing synchronises the stream: not a calibrate
    after a code-storing metrics call, not new code buffers.  A percentile pass is range,
    histogram and metrics, each one launch (fused fold) or two (separate fold kernel): there is
    no clearing launch."""
    ctx = q.Context(0)
    try:
        ctx.set_fold_mode(fold)
        g = torch.Generator(device="cuda"); g.manual_seed(0)
        x = torch.randn(70000, generator=g, device="cuda")
        w = torch.randn(32 * 300, generator=g, device="cuda")
        descs = q.desc_array([q.make_desc(x, None, 1, 1, 70000, q.PER_TENSOR, q.ASYM_U8, q.PERCENTILE, 0.999,
                                          flags=q.STORE_CODES),
                              q.make_desc(w, None, 1, 32, 300, q.PER_CHANNEL, q.SYM_I8, flags=q.STORE_CODES)])
        cal = ctx.calibrate(descs)
        codes = [torch.zeros(70000, dtype=torch.uint8, device="cuda"), torch.zeros(9600, dtype=torch.uint8, device="cuda")]
        met0 = ctx.quant_metrics(descs, cal.step, cal.inv, cal.offset, codes)
        torch.cuda.synchronize()
        s0, l0 = ctx.syncs, ctx.launches
        for it in range(6):                               # more rounds than staging areas for the pointers
            cal = ctx.calibrate(descs)
            other = [torch.zeros_like(c) for c in codes]
            met = ctx.quant_metrics(descs, cal.step, cal.inv, cal.offset, other if it % 2 else codes)
            met_plain = ctx.quant_metrics(descs, cal.step, cal.inv, cal.offset)
        assert ctx.syncs == s0, "a steady-state call synchronised the stream"
        assert ctx.launches - l0 == 6 * (2 + 1 + 1) * per_phase
        torch.cuda.synchronize()
        assert torch.equal(other[0], codes[0]) and torch.equal(other[1], codes[1]) and int(codes[0].max()) > 0
        assert torch.equal(met.sse.view(torch.int64), met0.sse.view(torch.int64))
        assert torch.equal(met_plain.sse.view(torch.int64), met0.sse.view(torch.int64))
        ref = oracle.sweep_tensor(x.cpu().numpy(), None, 1, 1, 70000, False, True, 0.999, want_codes=True)
        assert np.array_equal(codes[0].cpu().numpy(), ref.codes.view(np.uint8))
    finally:
        ctx.close()


def test_captured_pass_pins_the_plan_of_its_context():
    """While a captured pass lives, a call with another descriptor set is refused (it would
    overwrite the tile tables the graph replays) and the replay still gives the same bits."""
    s = torch.cuda.Stream()
    ctx = q.Context(0, stream=s)
    try:
        model = gen.make_model("squeezenet", seed=4, device="cuda", batch=1, layer_indices=range(6))
        md = q.model_descs(model)
        cfg = q.default_rank_cfg(select_mode=q.BY_BOPS_RATE, rate_permyriad=md.rate_permyriad)
        torch.cuda.synchronize()
        with torch.cuda.stream(s):
            sb, t = ctx.alloc_sweep_buffers(md.descs, md.n_layers)
            gr = ctx.sweep_graph(md.descs, md.n_layers, md.macs, None, cfg, sb)
            gr.launch(); s.synchronize()
            ref = {k: v.clone() for k, v in t.items() if v is not None}
            other = torch.randn(300000, device="cuda")
            od = q.desc_array([q.make_desc(other, None, 1, 1, other.numel(), q.PER_TENSOR, q.SYM_I8)])
            with pytest.raises(q.binding.Qv2Error) as e:
                ctx.calibrate(od)
            assert e.value.status == -8
            with pytest.raises(q.binding.Qv2Error) as e:
                ctx.set_schedule(q.SCHEDULE_L2_CHUNKED)
            assert e.value.status == -8
            cal = ctx.calibrate(md.descs)                 # the captured set itself is welcome
            for k in ("mse", "sqnr_db", "order", "step"):
                t[k].zero_()
            gr.launch(); s.synchronize()
            for k, v in ref.items():
                assert torch.equal(t[k].view(torch.uint8), v.view(torch.uint8)), k
            assert torch.equal(cal.step.view(torch.int32), t["step"].view(torch.int32)[: cal.step.numel()])
            gr.close()
            ctx.calibrate(od)                             # allowed again once the graph is gone
            s.synchronize()
    finally:
        ctx.close()


def test_rank_literal_outlier_order_is_bit_exact():
    ctx = q.Context(0)
    try:
        rng = np.random.default_rng(11)
        dv = lambda a: torch.from_numpy(np.asarray(a)).cuda()
        for trial in range(40):
            n = int(rng.integers(1, 90)) if trial < 36 else (512, 513, 700, 1500)[trial - 36]
            sw = rng.uniform(-5, 60, n).round(1); sa = rng.uniform(-5, 60, n).round(1)
            mw = rng.choice([1e-6, 1e-6, 1e-6, 1e-6, 3e-4, 2e-3], n); ma = rng.choice([1e-3, 1e-3, 1e-3, 9e-2, 0.5], n)
            macs = rng.integers(0, 10 ** 9, n).astype(np.uint64)
            fg = None
            if trial % 3 == 0:
                fg = rng.integers(0, max(2, n // 3), n).astype(np.uint32)
                fg[rng.random(n) < 0.4] = 0xFFFFFFFF
            mode = trial % 2
            rate = int(rng.integers(0, 10001)); kc = int(rng.integers(0, n + 2))
            ro, rk, rn = oracle.rank_layers_fused(sw, mw, sa, ma, fg, macs=macs, select_mode=mode, keep_count=kc,
                                                  rate_permyriad=rate, outlier_order=1)
            cfg = q.default_rank_cfg(select_mode=mode, keep_count=kc, rate_permyriad=rate,
                                     outlier_order=q.OUTLIERS_LITERAL)
            o, k, nk = ctx.rank_layers(dv(sw), dv(mw), dv(sa), dv(ma), dv(macs.view(np.int64)), None, cfg,
                                       fuse_group=None if fg is None else dv(fg.view(np.int32)))
            torch.cuda.synchronize()
            assert o.cpu().numpy().view(np.uint32).tolist() == ro.tolist(), trial
            assert k.cpu().numpy().tolist() == rk.tolist() and int(nk) == rn
        bad = q.default_rank_cfg(outlier_order=5)
        with pytest.raises(q.binding.Qv2Error):
            ctx.rank_layers(dv(np.ones(3)), dv(np.ones(3)), dv(np.ones(3)), dv(np.ones(3)), None, None, bad)
    finally:
        ctx.close()


@pytest.mark.parametrize("c,k,mis", [(64, 576, 0), (37, 1153, 0), (16, 64, 1)])
def test_fold_batchnorm_in_place(c, k, mis):
    from parity import to_dev
    g = torch.Generator(); g.manual_seed(c + k)
    w = torch.randn(c, k, generator=g); b = torch.randn(c, generator=g)
    gamma = torch.rand(c, generator=g) * 1.5 + 0.5; beta = torch.randn(c, generator=g)
    mean = torch.randn(c, generator=g); var = torch.rand(c, generator=g) * 3 + 0.05
    ra, rc = oracle.fold_batchnorm(w.numpy(), b.numpy(), gamma.numpy(), beta.numpy(), mean.numpy(), var.numpy())
    ctx = q.Context(0)
    try:
        dw = to_dev(w, mis).view(c, k)
        a, cc = ctx.fold_batchnorm(dw, b.cuda(), gamma.cuda(), beta.cuda(), mean.cuda(), var.cuda(), inplace=True)
        torch.cuda.synchronize()
        assert a.data_ptr() == dw.data_ptr()
        assert np.array_equal(dw.cpu().numpy().view(np.uint32), ra.view(np.uint32))
        assert np.array_equal(cc.cpu().numpy().view(np.uint32), rc.view(np.uint32))
        # a partial overlap of input and output is refused before anything runs
        buf = torch.zeros(2 * c * k, device="cuda")
        st = q.lib().qv2_fold_batchnorm(ctx._h, buf.data_ptr(), None, gamma.cuda().data_ptr(), beta.cuda().data_ptr(),
                                        mean.cuda().data_ptr(), var.cuda().data_ptr(), c, k, buf.data_ptr() + 4 * k, None)
        assert st == -1
    finally:
        ctx.close()
