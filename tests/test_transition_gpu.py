"""GPU parity of the SwiGLU pair transition (Eq. 1 line 2) against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import nested_pair_oracle as orc
from paper_2609_30379_b200 import workloads as wl
from tests.parity_utils import check

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def nt():
    from paper_2609_30379_b200 import binding
    return binding


def host(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def _run(nt, dtype, rows, c, seed, force_generic=False, expansion=4):
    cfg = wl.Config("tr", dtype, (3,), c_s=8, c_z=c, c_h=8, H=2, d=c // 2, blocks=1, seed=seed)
    W = wl.make_transition_weights(cfg, expansion=expansion)
    rng = np.random.default_rng(seed + 1)
    z = rng.standard_normal((rows, c)).astype(np.float32) * 2.0 + 0.5
    if dtype == "bf16":
        z = wl.round_to_bf16(z)
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    z_d = torch.from_numpy(z).to("cuda", tdt)
    W_d = {k: torch.from_numpy(np.ascontiguousarray(v)).to("cuda", tdt) for k, v in W.items()}
    hidden = W["W_a"].shape[0]
    ws = torch.empty(nt.nt_transition_workspace_bytes(tdt, c, hidden, max(rows, 1)) or 256, dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    prev = nt.nt_force_generic(force_generic)
    try:
        nt.nt_pair_transition(W_d, 1e-5, z_d, ws, status)
        torch.cuda.synchronize()
    finally:
        nt.nt_force_generic(prev)
    assert int(status.item()) == 0
    return host(z_d), orc.pair_transition(z, W)


@pytest.mark.parametrize("rows,c", [(1, 8), (37, 16), (300, 64), (1000, 128)])
def test_transition_f32(nt, rows, c):
    got, ref = _run(nt, "f32", rows, c, seed=rows)
    check("f32", got, ref, f"transition f32 rows={rows} c={c}")


@pytest.mark.parametrize("rows,c", [(1, 64), (129, 64), (700, 128), (5000, 128), (70000, 128)])
def test_transition_bf16(nt, rows, c):
    got, ref = _run(nt, "bf16", rows, c, seed=rows)
    check("bf16", got, ref, f"transition bf16 rows={rows} c={c}")


@pytest.mark.parametrize("rows,c", [(333, 128), (66000, 64)])
def test_transition_bf16_generic_kernels(nt, rows, c):
    got, ref = _run(nt, "bf16", rows, c, seed=rows, force_generic=True)
    check("bf16", got, ref, f"transition bf16 generic rows={rows} c={c}")


def test_transition_empty_and_arguments(nt):
    z = torch.empty((0, 128), dtype=torch.bfloat16, device="cuda")
    cfg = wl.Config("tr", "bf16", (3,), c_s=8, c_z=128, c_h=8, H=2, d=64, blocks=1, seed=1)
    W_d = {k: torch.from_numpy(np.ascontiguousarray(v)).to("cuda", torch.bfloat16)
           for k, v in wl.make_transition_weights(cfg).items()}
    ws = torch.empty(1 << 21, dtype=torch.uint8, device="cuda")
    nt.nt_pair_transition(W_d, 1e-5, z, ws)                      # no rows: nothing to do
    z1 = torch.zeros((4, 128), dtype=torch.bfloat16, device="cuda")
    small = torch.empty(16, dtype=torch.uint8, device="cuda")
    with pytest.raises(nt.NtError) as e:
        nt.nt_pair_transition(W_d, 1e-5, z1, small)
    assert e.value.status == 3      # NT_ERR_WORKSPACE


def test_transition_cfg2_sampled(nt):
    """Full cfg2 pair state (368 250 positions, c = 128, hidden = 512): the update is position-wise, so the oracle
    checks a sample of the positions one by one."""
    cfg = wl.CONFIGS["cfg2"] if isinstance(wl.CONFIGS, dict) else [c for c in wl.CONFIGS if c.name == "cfg2"][0]
    W = wl.make_transition_weights(cfg)
    rows, c = cfg.T2, cfg.c_z
    rng = np.random.default_rng(5)
    z = wl.round_to_bf16(rng.standard_normal((rows, c)).astype(np.float32) * 2.0)
    z_d = torch.from_numpy(z).to("cuda", torch.bfloat16)
    W_d = {k: torch.from_numpy(np.ascontiguousarray(v)).to("cuda", torch.bfloat16) for k, v in W.items()}
    ws = torch.empty(nt.nt_transition_workspace_bytes(torch.bfloat16, c, W["W_a"].shape[0], rows), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    nt.nt_pair_transition(W_d, 1e-5, z_d, ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    idx = np.unique(np.concatenate([np.arange(0, 300), rng.integers(0, rows, 3000), np.arange(rows - 300, rows)]))
    got = host(z_d[torch.from_numpy(idx).cuda()])
    check("bf16", got, orc.pair_transition(z[idx], W), "transition cfg2 sampled")
