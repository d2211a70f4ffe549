"""GPU parity of the accumulated broadcast (persistent pair stream) against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import nested_pair_oracle as orc
from paper_2609_30379_b200 import workloads as wl
from tests.parity_utils import check, ln0

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def nt():
    from paper_2609_30379_b200 import binding
    return binding


def host(t):
    return t.detach().to(torch.float32).cpu().numpy().astype(np.float64)


@pytest.mark.parametrize("dtype,generic,lengths,c_z", [("f32", False, (5, 9, 13, 16), 16), ("bf16", False, (0, 1, 7, 64, 65, 130), 128),
                                                        ("bf16", True, (3, 70), 128), ("bf16", False, (40, 9), 64)])
def test_pair_broadcast_add(nt, dtype, generic, lengths, c_z):
    from paper_2609_30379_b200 import runner
    cfg = wl.Config("stream", dtype, lengths, c_s=32, c_z=c_z, c_h=c_z, H=2, d=c_z // 2 if c_z <= 32 else 32, blocks=1, seed=81)
    inp = wl.make_inputs(cfg)
    prev = nt.nt_force_generic(generic)
    try:
        st = runner.PairStack(cfg, cfg.lengths, inp["blocks"])
        rng = np.random.default_rng(82)
        zp = rng.standard_normal((cfg.T2, cfg.c_z)).astype(np.float32)
        if dtype == "bf16":
            zp = wl.round_to_bf16(zp)
        st.z.copy_(torch.from_numpy(zp).to("cuda", st.dtype))
        x_d = runner.to_device(inp["x"], st.dtype)
        b = st.W[0]["broadcast"]
        nt.nt_pair_broadcast_add(st.L, x_d, b["W_a"], b["W_b"], b["ln_gamma"], b["ln_beta"], 1e-5, st.z, st.workspace)
        torch.cuda.synchronize()
        assert st.L.device_status() == 0
        ref = orc.pair_broadcast_add(zp, inp["x"], cfg.lengths, **inp["blocks"][0]["broadcast"])
        check(cfg.dtype, host(st.z), ref, "accumulated broadcast")
    finally:
        nt.nt_force_generic(prev)


def test_cfg2_sampled_rows_and_two_block_stream(nt):
    from paper_2609_30379_b200 import runner
    # the bench workload's shapes, one accumulated broadcast, checked on whole samples (the oracle's broadcast is cheap)
    cfg = wl.CONFIGS["cfg2"]
    inp = wl.make_inputs(cfg)
    st = runner.PairStack(cfg, cfg.lengths, inp["blocks"][:1])
    x_d = runner.to_device(inp["x"], st.dtype)
    b = st.W[0]["broadcast"]
    nt.nt_pair_broadcast(st.L, x_d, b["W_a"], b["W_b"], b["ln_gamma"], b["ln_beta"], 1e-5, st.z, st.workspace)
    z0 = host(st.z)
    nt.nt_pair_broadcast_add(st.L, x_d, b["W_a"], b["W_b"], b["ln_gamma"], b["ln_beta"], 1e-5, st.z, st.workspace)
    torch.cuda.synchronize()
    ref = orc.pair_broadcast_add(z0, inp["x"], cfg.lengths, **inp["blocks"][0]["broadcast"])
    check("bf16", host(st.z), ref, "accumulated broadcast, bench workload")
    # two stacked blocks with a persistent pair state: drift against the oracle (no teacher forcing), loose guard
    cfg2 = wl.Config("stream2", "bf16", (40, 72, 9), c_s=128, c_z=128, c_h=128, H=4, d=32, blocks=2, seed=83)
    inp2 = wl.make_inputs(cfg2)
    st2 = runner.PairStack(cfg2, cfg2.lengths, inp2["blocks"])
    x2 = runner.to_device(inp2["x"], st2.dtype)
    x_out, z = st2.forward(x2, persistent=True)
    rx, rz = orc.stack_forward(inp2["x"], cfg2.lengths, inp2["blocks"], cfg2.H, cfg2.d, persistent=True)
    dz = float(np.abs(ln0(host(z)) - ln0(rz)).max())
    dx = float(np.abs(ln0(host(x_out)) - ln0(rx)).max())
    assert dz < 0.25 and dx < 0.25, (dz, dx)
