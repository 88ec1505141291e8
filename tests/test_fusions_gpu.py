"""GPU parity of the steps either side of the recurrence against the fp64 oracle: in-kernel q/k/v activation
(SWILA_QKV_ACT: App. B.2, App. D.1), sums over time of the mixture weights (swila_forward_stats: Sec. 3.5,
App. D.5) and the output RMSNorm (swila_output_norm: App. D.1).  All calls go through the C ABI."""
import numpy as np
import pytest
import torch

from paper_2609_39034_b200 import workloads as wl
from tests._gpu_util import TOL_BF16_O, TOL_FP32, TOL_STATE, gpu_forward, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def binding():
    from paper_2609_39034_b200 import binding as b
    return b


@pytest.fixture(scope="module")
def oracle():
    from oracle import swila_oracle
    return swila_oracle


@pytest.fixture(scope="module")
def fus():
    from oracle import swila_fusions
    return swila_fusions


def _raw_qkv(w, inp, seed):
    """Replace the generator's (already normalised) q, k, v by raw projections: unit-variance values with a
    per-token scale spread, rounded to the io dtype like every other input."""
    g = torch.Generator().manual_seed(seed)
    out = dict(inp)
    for name, width in (("q", w.Dk), ("k", w.Dk), ("v", w.Dv)):
        x = torch.randn((w.B, w.H, w.T, width), generator=g) * torch.exp(0.5 * torch.randn((w.B, w.H, w.T, 1), generator=g))
        out[name] = x.to(w.torch_io_dtype).contiguous()
    return out


SHAPES = [
    pytest.param(wl.CONFIGS[0].with_(T=67), id="c0_fp32_dk16"),
    pytest.param(wl.CONFIGS[1].with_(B=1, H=2, T=150), id="c1_bf16_dk64"),
    pytest.param(wl.CONFIGS[2].with_(B=1, H=1, T=70, recipe="gauss"), id="c2_bf16_dk128"),
    pytest.param(wl.CONFIGS[3].with_(B=1, H=2, T=45, recipe="gauss"), id="c3_fp32_j8"),
    pytest.param(wl.CONFIGS[1].with_(B=1, H=1, T=40, Dv=24), id="ragged_columns"),
]


@pytest.mark.parametrize("w", SHAPES)
@pytest.mark.parametrize("variant", ["vanilla", "temporal", "gated"])
def test_qkv_activation_in_kernel(binding, oracle, fus, w, variant):
    wv = w.variant(temporal=variant == "temporal", gated=variant == "gated")
    inp = _raw_qkv(wv, wl.make_inputs(wv, stress=True), seed=7)
    qa, ka, va = fus.qkv_activation(inp["q"], inp["k"], inp["v"])
    ref_in = dict(inp, q=qa, k=ka, v=va)
    ref = oracle.forward_inputs(ref_in, flags=wv.flags, gran=wv.gate_granularity)
    wa = wv.with_(flags=wv.flags | wl.FLAG_QKV_ACT)
    got = gpu_forward(binding, wa, to_dev(inp))
    tol_o = TOL_BF16_O if w.io_dtype == "bf16" else TOL_FP32
    assert wl.rel_err(got["o"], torch.from_numpy(ref["o"])) < tol_o
    assert wl.rel_err(got["W"], torch.from_numpy(ref["W"])) < TOL_STATE
    # decode steps with the flag continue the same sequence: one more token on the carried state
    st = {"W": got["W"].cuda(), "r_prev": got["r_prev"].cuda() if wv.temporal else None,
          "rho_prev": got["rho_prev"].cuda() if wv.temporal else None}
    step = {k: (v[:, :, :1].contiguous() if v is not None and k not in ("W0", "r0", "rho0") else v) for k, v in to_dev(inp).items()}
    o1 = binding.swila_decode_step(wa, step, st)
    torch.cuda.synchronize()
    ref1 = oracle.forward_inputs({k: (v[:, :, :1] if v is not None and k not in ("W0", "r0", "rho0") else v) for k, v in ref_in.items()},
                                 flags=wv.flags, gran=wv.gate_granularity,
                                 state={"W": ref["W"], "r_prev": ref.get("r_prev"), "rho_prev": ref.get("rho_prev")})
    assert wl.rel_err(o1.cpu(), torch.from_numpy(ref1["o"])) < tol_o
    assert wl.rel_err(st["W"].cpu(), torch.from_numpy(ref1["W"])) < TOL_STATE


def test_qkv_activation_is_refused_by_the_chunked_kernel(binding):
    w = wl.CONFIGS[1].with_(B=1, H=1, T=64, flags=wl.FLAG_QKV_ACT)
    inp = wl.make_inputs(w, device="cuda")
    with pytest.raises(binding.SwilaError) as e:
        binding.swila_forward(w, inp, algo=binding.ALGO_CHUNK)
    assert e.value.status == binding.ERR_UNSUPPORTED


@pytest.mark.parametrize("w", SHAPES)
@pytest.mark.parametrize("temporal,algo", [(False, "scan"), (True, "scan"), (False, "auto"), (True, "auto")],
                         ids=["vanilla_scan", "temporal_scan", "vanilla_auto", "temporal_auto"])
def test_statistics_match_the_oracle(binding, oracle, fus, w, temporal, algo):
    """`auto` takes the chunked tensor-core kernel for the bf16 shapes of 64 tokens and more."""
    algo = getattr(binding, "ALGO_" + algo.upper())
    wv = w.variant(temporal=temporal)
    inp = wl.make_inputs(wv, stress=True)
    ref = oracle.forward_inputs(inp, flags=wv.flags, want_r=True)
    rho = fus.readout_weights(inp["piq_logit"], inp.get("gq_logit") if temporal else None, inp.get("rho0") if temporal else None)
    want = fus.responsibility_stats(ref["r"], rho)
    dev = to_dev(inp)
    stats = binding.stats_alloc(wv)
    st_out = binding.state_alloc(wv, init=False)
    sin = {"W": dev["W0"], "r_prev": dev.get("r0"), "rho_prev": dev.get("rho0")}
    o = binding.swila_forward_stats(wv, dev, stats, state_in=sin, state_out=st_out, algo=algo)
    torch.cuda.synchronize()
    # sums of T values in [0, 1] (entropies in [0, ln J]) accumulated in FP32 from FP32 responsibilities
    for name in ("r_sum", "r_ent", "rho_sum", "rho_ent"):
        assert wl.rel_err(stats[name].cpu(), torch.from_numpy(want[name])) < 1e-4, name
    # outputs and state are those of the plain call, bit for bit
    st2 = binding.state_alloc(wv, init=False)
    o2 = binding.swila_forward(wv, dev, state_in=sin, state_out=st2, algo=algo)
    torch.cuda.synchronize()
    assert torch.equal(o, o2) and torch.equal(st_out["W"], st2["W"])
    # a second call ADDS to the buffers; a sequence fed in two pieces accumulates to the same sums
    stats2 = binding.stats_alloc(wv)
    half = wv.T // 2
    first = {k: (v[:, :, :half].contiguous() if v is not None and k not in ("W0", "r0", "rho0") else v) for k, v in dev.items()}
    second = {k: (v[:, :, half:].contiguous() if v is not None and k not in ("W0", "r0", "rho0") else v) for k, v in dev.items()}
    carry = binding.state_alloc(wv, init=False)
    binding.swila_forward_stats(wv, first, stats2, state_in=sin, state_out=carry, algo=algo)
    binding.swila_forward_stats(wv, second, stats2, state_in=carry, state_out=carry, algo=algo)
    torch.cuda.synchronize()
    for name in ("r_sum", "r_ent", "rho_sum", "rho_ent"):
        assert wl.rel_err(stats2[name].cpu(), stats[name].cpu()) < 2e-5, name
    # mutual information of Sec. 3.5 from the sums: the quantity the loss is built from
    mi = fus.mutual_information(stats["r_sum"].cpu().numpy(), stats["r_ent"].cpu().numpy(), wv.T)
    mi_ref = fus.mutual_information(want["r_sum"], want["r_ent"], wv.T)
    assert np.max(np.abs(mi - mi_ref)) < 1e-4


@pytest.mark.parametrize("algo", ["scan", "chunk"])
def test_statistics_members_are_optional(binding, algo):
    algo = getattr(binding, "ALGO_" + algo.upper())
    w = wl.CONFIGS[1].with_(B=1, H=1, T=96)
    inp = wl.make_inputs(w, device="cuda")
    full = binding.stats_alloc(w)
    binding.swila_forward_stats(w, inp, full, algo=algo)
    only = {"r_sum": torch.zeros_like(full["r_sum"])}
    binding.swila_forward_stats(w, inp, only, algo=algo)
    torch.cuda.synchronize()
    assert torch.equal(only["r_sum"], full["r_sum"])  # one piece per tile here: a single addition per element


@pytest.mark.parametrize("temporal", [False, True], ids=["plain", "temporal"])
def test_statistics_on_the_balanced_schedule(binding, oracle, fus, temporal):
    """More tiles than SMs: the chunked kernel cuts sequences into pieces that run in different blocks, whose sums
    meet in the caller's buffers through atomic additions.  Checked against the scan kernel's sums and, on sampled
    rows, against the oracle."""
    w = wl.CONFIGS[2].with_(B=2, H=20, T=1024).variant(temporal=temporal)
    inp = wl.make_inputs(w, device="cuda", stress=True)
    sin = {"W": inp["W0"], "r_prev": inp.get("r0"), "rho_prev": inp.get("rho0")}
    got, ref = binding.stats_alloc(w), binding.stats_alloc(w)
    st = binding.state_alloc(w, init=False)
    binding.swila_forward_stats(w, inp, got, state_in=sin, state_out=st, algo=binding.ALGO_CHUNK)
    binding.swila_forward_stats(w, inp, ref, state_in=sin, state_out=st, algo=binding.ALGO_SCAN)
    torch.cuda.synchronize()
    binding.device_status()
    for name in ("r_sum", "r_ent", "rho_sum", "rho_ent"):
        assert wl.rel_err(got[name].cpu(), ref[name].cpu()) < 1e-4, name
    bh = torch.tensor([3, 17, 38])
    cols = torch.tensor([0, 31, 32, 77, 127])
    rows = {k: (v.cpu() if v is not None else None) for k, v in wl.slice_rows(inp, bh.cuda(), cols.cuda()).items()}
    o_ref = oracle.forward_inputs(rows, flags=w.flags, want_r=True)
    want = fus.responsibility_stats(o_ref["r"], fus.readout_weights(rows["piq_logit"], rows.get("gq_logit") if temporal else None,
                                                                    rows.get("rho0") if temporal else None))
    for name in ("r_sum", "rho_sum"):
        g = got[name].reshape(w.B * w.H, w.J, w.Dv)[bh.cuda()][:, :, cols.cuda()].unsqueeze(1).cpu()
        assert wl.rel_err(g, torch.from_numpy(want[name])) < 1e-4, name
    for name in ("r_ent", "rho_ent"):
        g = got[name].reshape(w.B * w.H, w.Dv)[bh.cuda()][:, cols.cuda()].unsqueeze(1).cpu()
        assert wl.rel_err(g, torch.from_numpy(want[name])) < 1e-4, name


@pytest.mark.parametrize("io,Dv,T", [("bf16", 128, 1000), ("bf16", 64, 77), ("fp32", 16, 50), ("fp32", 256, 33), ("bf16", 512, 9)])
@pytest.mark.parametrize("with_weight", [False, True])
def test_output_rmsnorm(binding, fus, io, Dv, T, with_weight):
    w = wl.CONFIGS[1].with_(B=2, H=3, T=T, Dv=Dv, io_dtype=io)
    g = torch.Generator().manual_seed(Dv + T)
    o = (torch.randn((w.B, w.H, T, Dv), generator=g) * torch.exp(torch.randn((w.B, w.H, T, 1), generator=g))).to(w.torch_io_dtype)
    wgt = (1.0 + 0.1 * torch.randn(Dv, generator=g)) if with_weight else None
    want = fus.output_rmsnorm(o, wgt.numpy() if with_weight else None, eps=1e-6)
    got = binding.swila_output_norm(w, o.cuda(), wgt.cuda() if with_weight else None, eps=1e-6)
    torch.cuda.synchronize()
    tol = TOL_BF16_O if io == "bf16" else 1e-5
    assert wl.rel_err(got.cpu(), torch.from_numpy(want)) < tol


def test_output_rmsnorm_rejects_bad_arguments(binding):
    w = wl.CONFIGS[1].with_(B=1, H=1, T=4)
    o = torch.zeros((1, 1, 4, w.Dv), device="cuda", dtype=torch.bfloat16)
    with pytest.raises(binding.SwilaError) as e:
        binding.swila_output_norm(w, o, eps=-1.0)
    assert e.value.status == binding.ERR_SHAPE
    import ctypes
    sh = binding.make_shape(w, T=0)  # no rows: nothing to do, nothing touched
    assert binding.lib.swila_output_norm(ctypes.byref(sh), ctypes.c_void_p(o.data_ptr()), None, ctypes.c_float(1e-6), None) == 0
    assert binding.lib.swila_output_norm(ctypes.byref(sh), None, None, ctypes.c_float(1e-6), None) == binding.ERR_NULL
