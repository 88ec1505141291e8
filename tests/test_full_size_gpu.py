"""GPU parity at the benchmark configurations' full sizes, in the launch configuration
bench.py times.  Small configs are compared element by element; for the large ones the CUDA
path runs the full problem and the oracle recomputes a seeded sample of (batch, head) rows and
output columns from the same inputs -- legitimate because every output column is an independent
recurrence (Sec. 3.1), which tests/test_oracle_pins.py::test_column_independence pins."""
import pytest
import torch

from paper_2609_39034_b200 import workloads as wl
from tests._gpu_util import TOL_BF16_O, TOL_FP32, TOL_STATE, assert_close, gpu_forward, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def binding():
    assert torch.cuda.is_available()
    from paper_2609_39034_b200 import binding as b

    return b


def _sample(w, n_bh, n_cols, seed):
    g = torch.Generator().manual_seed(seed)
    bh = torch.randperm(w.B * w.H, generator=g)[:n_bh].sort().values
    cols = torch.randperm(w.Dv, generator=g)[:n_cols].sort().values
    return bh, cols


def _check_sample(w, oracle, inp_dev, got_o, got_W, bh, cols, what):
    sub = wl.slice_rows({n: (x if x is not None else None) for n, x in inp_dev.items()}, bh.cuda(), cols.cuda())
    sub = {n: (x.cpu() if x is not None else None) for n, x in sub.items()}
    ref = oracle.forward_inputs(sub)
    o = got_o.reshape(w.B * w.H, w.T, w.Dv)[bh.cuda()][..., cols.cuda()].unsqueeze(1).cpu()
    W = got_W.reshape(w.B * w.H, w.J, w.Dv, w.Dk)[bh.cuda()][:, :, cols.cuda()].unsqueeze(1).cpu()
    tol_o = TOL_BF16_O if w.io_dtype == "bf16" else TOL_FP32
    e_o, e_w = wl.rel_err(o, torch.from_numpy(ref["o"])), wl.rel_err(W, torch.from_numpy(ref["W"]))
    assert e_o < tol_o and e_w < TOL_STATE, (what, e_o, e_w)


@pytest.mark.parametrize("cfg", [0, 1])
@pytest.mark.parametrize("stress", [False, True], ids=["calm", "stress"])
def test_small_configs_full_comparison(binding, oracle, cfg, stress):
    w = wl.CONFIGS[cfg]
    inp = wl.make_inputs(w, stress=stress)
    ref = oracle.forward_inputs(inp)
    got = gpu_forward(binding, w, to_dev(inp))
    assert_close(w, got, ref, w.name)


@pytest.mark.parametrize("cfg,n_bh,n_cols", [(2, 6, 12), (3, 24, 64)])
@pytest.mark.parametrize("stress", [False, True], ids=["calm", "stress"])
def test_large_prefill_configs_sampled(binding, oracle, cfg, n_bh, n_cols, stress):
    w = wl.CONFIGS[cfg]
    inp = wl.make_inputs(w, device="cuda", stress=stress)
    st = binding.state_alloc(w, init=False)
    o = binding.swila_forward(w, inp, state_in={"W": inp["W0"]}, state_out=st)
    torch.cuda.synchronize()
    assert bool(torch.isfinite(o.float()).all()) and bool(torch.isfinite(st["W"]).all())
    bh, cols = _sample(w, n_bh, n_cols, seed=cfg)
    _check_sample(w, oracle, inp, o, st["W"], bh, cols, w.name)


def test_batched_decode_config_sampled(binding, oracle):
    """Config 4 at full batch: 4096-token prefill fed as 16 chunks with carried state, then
    all 1024 single-token decode steps with fresh inputs; a sample of streams is replayed by the oracle
    over the whole 4096 + 1024 token history; the output of every step and the final state are compared."""
    w = wl.CONFIGS[4]
    n_decode = wl.DECODE_STEPS
    bh, cols = _sample(w, 12, 8, seed=4)
    st = binding.state_alloc(w)
    chunk = wl.DECODE_PREFILL_CHUNK
    hist, outs = [], []
    for c in range(w.T // chunk):
        wc = w.with_(T=chunk)
        inp = wl.make_inputs(wc, device="cuda", seed_offset=1 + c)
        o = binding.swila_forward(w, inp, state_in=st, state_out=st)
        sub = wl.slice_rows(inp, bh.cuda(), cols.cuda())
        hist.append({n: (x.cpu() if x is not None else None) for n, x in sub.items()})
        outs.append(o.reshape(w.B * w.H, chunk, w.Dv)[bh.cuda()][..., cols.cuda()].cpu())
        del inp, o
    for s in range(n_decode):
        inp = wl.decode_step_inputs(w, s, device="cuda")
        o = binding.swila_decode_step(w, inp, st)
        sub = wl.slice_rows(inp, bh.cuda(), cols.cuda())
        hist.append({n: (x.cpu() if x is not None else None) for n, x in sub.items()})
        outs.append(o.reshape(w.B * w.H, 1, w.Dv)[bh.cuda()][..., cols.cuda()].cpu())
    torch.cuda.synchronize()
    names = ("q", "k", "v", "beta_logit", "pik_logit", "piq_logit")
    full = {n: torch.cat([h[n] for h in hist], dim=2) for n in names}
    ref = oracle.forward(full["q"], full["k"], full["v"], full["beta_logit"], full["pik_logit"], full["piq_logit"])
    o = torch.cat(outs, dim=1).unsqueeze(1)
    W = st["W"].reshape(w.B * w.H, w.J, w.Dv, w.Dk)[bh.cuda()][:, :, cols.cuda()].unsqueeze(1).cpu()
    e_o, e_w = wl.rel_err(o, torch.from_numpy(ref["o"])), wl.rel_err(W, torch.from_numpy(ref["W"]))
    # decode outputs alone (the last n_decode tokens)
    e_dec = wl.rel_err(o[:, :, -n_decode:], torch.from_numpy(ref["o"][:, :, -n_decode:]))
    assert e_o < TOL_BF16_O and e_dec < TOL_BF16_O and e_w < TOL_STATE, (e_o, e_dec, e_w)


def test_paper_native_shapes(binding, oracle):
    """Shapes the paper itself quotes: the 374M language-model layer (H=8, J=4, D=64) at B=16, T=4096
    (App. C), and the generation protocol of App. D.4 -- a 2048-token prompt followed by 128 decoded
    tokens -- at batch 8.  Sampled rows are replayed by the oracle."""
    lm = wl.CONFIGS[1].with_(name="lm374m_layer", B=16, H=8, T=4096)
    inp = wl.make_inputs(lm, device="cuda", stress=True)
    st = binding.state_alloc(lm, init=False)
    o = binding.swila_forward(lm, inp, state_in={"W": inp["W0"]}, state_out=st)
    torch.cuda.synchronize()
    bh, cols = _sample(lm, 8, 16, seed=11)
    _check_sample(lm, oracle, inp, o, st["W"], bh, cols, lm.name)

    # the component-count ablation of Sec. 5: the same layer with J = 16 (chunked kernel, outputs formed per thread)
    abl = lm.with_(name="lm374m_layer_j16", J=16)
    inp = wl.make_inputs(abl, device="cuda", stress=True)
    st = binding.state_alloc(abl, init=False)
    o = binding.swila_forward(abl, inp, state_in={"W": inp["W0"]}, state_out=st)
    torch.cuda.synchronize()
    binding.device_status()
    bh, cols = _sample(abl, 6, 12, seed=13)
    _check_sample(abl, oracle, inp, o, st["W"], bh, cols, abl.name)
    del inp, st, o

    gen = wl.CONFIGS[1].with_(name="generation", B=8, H=8, T=2048)
    bh, cols = _sample(gen, 8, 8, seed=12)
    prompt = wl.make_inputs(gen, device="cuda")
    st = binding.state_alloc(gen)
    outs = [binding.swila_forward(gen, prompt, state_in=st, state_out=st)]
    hist = [wl.slice_rows(prompt, bh.cuda(), cols.cuda())]
    for s in range(128):
        step = wl.decode_step_inputs(gen, s, device="cuda")
        outs.append(binding.swila_decode_step(gen, step, st))
        hist.append(wl.slice_rows(step, bh.cuda(), cols.cuda()))
    torch.cuda.synchronize()
    names = ("q", "k", "v", "beta_logit", "pik_logit", "piq_logit")
    full = {n: torch.cat([h[n].cpu() for h in hist], dim=2) for n in names}
    ref = oracle.forward(full["q"], full["k"], full["v"], full["beta_logit"], full["pik_logit"], full["piq_logit"])
    o = torch.cat(outs, dim=2).reshape(gen.B * gen.H, -1, gen.Dv)[bh.cuda()][..., cols.cuda()].unsqueeze(1).cpu()
    W = st["W"].reshape(gen.B * gen.H, gen.J, gen.Dv, gen.Dk)[bh.cuda()][:, :, cols.cuda()].unsqueeze(1).cpu()
    assert wl.rel_err(o, torch.from_numpy(ref["o"])) < TOL_BF16_O
    assert wl.rel_err(W, torch.from_numpy(ref["W"])) < TOL_STATE


def test_balanced_schedule_matches_one_tile_per_block(binding):
    """More tiles than SMs and not a whole number of waves: with a state output the chunked kernel cuts the
    chunk sequence into equal runs per SM and hands split tiles' states over between blocks; without one it
    runs one tile per block.  Both must give the same outputs, and the state must match the scan kernel's."""
    w = wl.CONFIGS[2].with_(B=2, H=20, T=1024)  # 160 tiles of 32 chunks
    inp = wl.make_inputs(w, device="cuda")
    st = binding.state_alloc(w, init=False)
    o_split = binding.swila_forward(w, inp, state_in={"W": inp["W0"]}, state_out=st, algo=binding.ALGO_CHUNK)
    o_plain = binding.swila_forward(w, inp, state_in={"W": inp["W0"]}, state_out=None, algo=binding.ALGO_CHUNK)
    st_scan = binding.state_alloc(w, init=False)
    o_scan = binding.swila_forward(w, inp, state_in={"W": inp["W0"]}, state_out=st_scan, algo=binding.ALGO_SCAN)
    torch.cuda.synchronize()
    binding.device_status()
    # a split tile restarts from the fully updated state instead of adding the cross-chunk term: the
    # arithmetic differs in the last bits only, far below one bf16 rounding step of the outputs
    assert wl.rel_err(o_split.float().cpu(), o_plain.float().cpu()) < 1e-2
    assert wl.rel_err(o_split.float().cpu(), o_scan.float().cpu()) < 1e-2
    assert wl.rel_err(st["W"].cpu(), st_scan["W"].cpu()) < TOL_STATE


@pytest.mark.parametrize("algo", ["chunk", "scan"])
def test_long_sequence_from_zero_state(binding, oracle, algo):
    """One (batch, head) pair, 8192 tokens from a zero state with near-uniform gates, every column compared.
    The J components start identical and separate only through the feedback of the E-step (Eq. 3.4) on their
    own updates, so rounding of the rank-one updates (Eq. 3.3) is carried and amplified along the whole
    sequence: the least forgiving input found for the state tolerance, and the one that fixes how many bits
    of the update coefficients the chunked kernel hands to the tensor cores (24; with 16 it fails here)."""
    w = wl.CONFIGS[2].with_(B=1, H=1, T=8192, recipe="gauss")
    inp = wl.make_inputs(w)
    ref = oracle.forward_inputs(inp)
    got = gpu_forward(binding, w, to_dev(inp), algo=getattr(binding, "ALGO_" + algo.upper()))
    assert wl.rel_err(got["o"], torch.from_numpy(ref["o"])) < TOL_BF16_O
    assert wl.rel_err(got["W"], torch.from_numpy(ref["W"])) < TOL_STATE


@pytest.mark.parametrize("temporal,gated", [(False, False), (True, False), (False, True)], ids=["vanilla", "temporal", "gated_rows"])
def test_calls_replay_from_a_cuda_graph(binding, temporal, gated):
    """A prefill on the balanced schedule (cooperative launch, state handed over between blocks through flags that
    carry the launch's epoch) and a decode step, captured once in a CUDA graph and replayed on fresh inputs: every
    replay must equal the eager call on the same inputs.  A replay reuses the captured epoch, so the hand-over flags
    must not keep last replay's value."""
    w = wl.CONFIGS[2].with_(B=2, H=20, T=1024).variant(temporal=temporal, gated=gated, granularity=wl.GRAN_PER_OUT)
    inp = wl.make_inputs(w, device="cuda", stress=True)
    st = binding.state_alloc(w, init=False)
    o = torch.empty((w.B, w.H, w.T, w.Dv), device="cuda", dtype=w.torch_io_dtype)
    w1 = w.with_(T=1)
    sin = {"W": inp["W0"], "r_prev": inp.get("r0"), "rho_prev": inp.get("rho0")}
    step = wl.decode_step_inputs(w, 0, device="cuda")
    o1 = torch.empty((w.B, w.H, 1, w.Dv), device="cuda", dtype=w.torch_io_dtype)

    def call():
        binding.swila_forward(w, inp, state_in=sin, state_out=st, o=o, algo=binding.ALGO_CHUNK)
        binding.swila_decode_step(w1, step, st, o=o1)

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        call()  # everything lazy (function attributes, module loading) happens outside the capture
    torch.cuda.current_stream().wait_stream(side)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        call()
    names = ("q", "k", "v", "beta_logit", "pik_logit", "piq_logit") + (("gk_logit", "gq_logit") if temporal else ()) + (
        ("alpha",) if gated else ())
    for rep in range(3):
        fresh = wl.make_inputs(w, device="cuda", seed_offset=rep + 1, stress=True)
        fresh_step = wl.decode_step_inputs(w, rep + 1, device="cuda")
        for n in names:
            inp[n].copy_(fresh[n])
            step[n].copy_(fresh_step[n])
        inp["W0"].copy_(fresh["W0"])
        if temporal:
            inp["r0"].copy_(fresh["r0"])
            inp["rho0"].copy_(fresh["rho0"])
        graph.replay()
        torch.cuda.synchronize()
        got = (o.clone(), o1.clone(), st["W"].clone()) + ((st["r_prev"].clone(), st["rho_prev"].clone()) if temporal else ())
        call()
        torch.cuda.synchronize()
        binding.device_status()
        assert torch.equal(got[0], o) and torch.equal(got[1], o1) and torch.equal(got[2], st["W"]), rep
        if temporal:
            assert torch.equal(got[3], st["r_prev"]) and torch.equal(got[4], st["rho_prev"]), rep


@pytest.mark.parametrize("shape", ["headline", "more_tiles_than_sms"])
def test_temporal_prefill_sampled(binding, oracle, shape):
    """Temporal SwiLA (App. B.3) at full size through the default dispatch (chunked kernel): the LM-shaped
    configuration, and a shape whose tiles are split between blocks, so that W, r_prev and rho_prev of a split tile
    travel through the state output and the hand-over flag.  Sampled rows are replayed by the oracle; the whole
    state is compared with the scan kernel's."""
    base = wl.CONFIGS[2] if shape == "headline" else wl.CONFIGS[2].with_(B=2, H=20, T=1024)
    w = base.variant(temporal=True)
    inp = wl.make_inputs(w, device="cuda", stress=True)
    sin = {"W": inp["W0"], "r_prev": inp["r0"], "rho_prev": inp["rho0"]}
    st = binding.state_alloc(w, init=False)
    o = binding.swila_forward(w, inp, state_in=sin, state_out=st)
    st_scan = binding.state_alloc(w, init=False)
    o_scan = binding.swila_forward(w, inp, state_in=sin, state_out=st_scan, algo=binding.ALGO_SCAN)
    torch.cuda.synchronize()
    binding.device_status()
    assert wl.rel_err(o.float().cpu(), o_scan.float().cpu()) < TOL_BF16_O
    for name in ("W", "r_prev", "rho_prev"):
        # two kernels, each held to the tolerance against the oracle below: against each other, twice that
        assert wl.rel_err(st[name].cpu(), st_scan[name].cpu()) < 2 * TOL_STATE, name
    bh, cols = _sample(w, 4, 8, seed=21)
    sub = wl.slice_rows(inp, bh.cuda(), cols.cuda())
    ref = oracle.forward_inputs({n: (x.cpu() if x is not None else None) for n, x in sub.items()}, flags=w.flags)
    pick = lambda x: x.reshape((w.B * w.H,) + tuple(x.shape[2:]))[bh.cuda()]  # noqa: E731
    assert wl.rel_err(pick(o)[..., cols.cuda()].unsqueeze(1).cpu(), torch.from_numpy(ref["o"])) < TOL_BF16_O
    assert wl.rel_err(pick(st["W"])[:, :, cols.cuda()].unsqueeze(1).cpu(), torch.from_numpy(ref["W"])) < TOL_STATE
    for name in ("r_prev", "rho_prev"):
        assert wl.rel_err(pick(st[name])[..., cols.cuda()].unsqueeze(1).cpu(), torch.from_numpy(ref[name])) < TOL_STATE, name


@pytest.mark.parametrize("shape,gran,post", [("headline", wl.GRAN_PER_OUT, False), ("more_tiles_than_sms", wl.GRAN_SCALAR, True),
                                             ("more_tiles_than_sms", wl.GRAN_PER_OUT, False)],
                         ids=["headline_out_pre", "split_scalar_post", "split_out_pre"])
def test_gated_rows_prefill_sampled(binding, oracle, shape, gran, post):
    """Gated SwiLA with one decay per state row (Eqs. 3.7 / 3.8 as printed) at full size through the default dispatch
    (guard pass, chunked kernel, scan kernel standing by): the LM-shaped configuration, and a shape whose tiles are
    split between blocks (tail pieces wait for their state, which is where the decay warp once ran ahead of the
    helpers).  Sampled rows are replayed by the oracle; the whole state is compared with the scan kernel's."""
    base = wl.CONFIGS[2] if shape == "headline" else wl.CONFIGS[2].with_(B=2, H=20, T=1024)
    w = base.variant(gated=True, granularity=gran, post_decay=post)
    assert binding.auto_algo(w) == binding.ALGO_CHUNK
    inp = wl.make_inputs(w, device="cuda", stress=True)
    sin = {"W": inp["W0"]}
    st = binding.state_alloc(w, init=False)
    o = binding.swila_forward(w, inp, state_in=sin, state_out=st)
    st_scan = binding.state_alloc(w, init=False)
    o_scan = binding.swila_forward(w, inp, state_in=sin, state_out=st_scan, algo=binding.ALGO_SCAN)
    torch.cuda.synchronize()
    binding.device_status()
    assert not torch.equal(st["W"], st_scan["W"])  # two kernels
    assert wl.rel_err(o.float().cpu(), o_scan.float().cpu()) < TOL_BF16_O
    assert wl.rel_err(st["W"].cpu(), st_scan["W"].cpu()) < 2 * TOL_STATE
    bh, cols = _sample(w, 4, 8, seed=31)
    sub = wl.slice_rows(inp, bh.cuda(), cols.cuda(), gran=gran)
    ref = oracle.forward_inputs({n: (x.cpu() if x is not None else None) for n, x in sub.items()}, flags=w.flags, gran=gran)
    pick = lambda x: x.reshape((w.B * w.H,) + tuple(x.shape[2:]))[bh.cuda()]  # noqa: E731
    assert wl.rel_err(pick(o)[..., cols.cuda()].unsqueeze(1).cpu(), torch.from_numpy(ref["o"])) < TOL_BF16_O
    assert wl.rel_err(pick(st["W"])[:, :, cols.cuda()].unsqueeze(1).cpu(), torch.from_numpy(ref["W"])) < TOL_STATE
