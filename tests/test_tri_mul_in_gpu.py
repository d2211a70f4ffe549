"""GPU parity of the incoming triangle update (contraction over the first pair index) against the CPU oracle,
through the C ABI.  The state it acts on is the one the block's broadcast produces from the seeded tokens."""
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
    return t.detach().to(torch.float32).cpu().numpy().astype(np.float64)


def _state_and_call(nt, cfg, force_generic=False):
    """Broadcast (checked elsewhere) then nt_tri_mul_in; returns the state before and after, on the device."""
    from paper_2609_30379_b200 import runner
    inp = wl.make_inputs(cfg)
    prev = nt.nt_force_generic(force_generic)
    try:
        st = runner.PairStack(cfg, cfg.lengths, inp["blocks"][:1])
        w_d = st.W[0]
        x_d = runner.to_device(inp["x"], st.dtype)
        b = w_d["broadcast"]
        nt.nt_pair_broadcast(st.L, x_d, b["W_a"], b["W_b"], b["ln_gamma"], b["ln_beta"], 1e-5, st.z, st.workspace)
        z0 = st.z.clone()
        nt.nt_tri_mul_in(st.L, w_d["trimul"], 1e-5, st.z, st.workspace)
        torch.cuda.synchronize()
        assert st.L.device_status() == 0
        return z0, st.z.clone(), inp["blocks"][0]["trimul"]
    finally:
        nt.nt_force_generic(prev)


def _check_full(cfg, z0, z1, W, samples):
    po = np.concatenate([[0], np.cumsum(np.asarray(cfg.lengths, dtype=np.int64) ** 2)])
    for s in samples:
        n = cfg.lengths[s]
        if n == 0:
            continue
        ref = orc.tri_mul_in(host(z0[po[s]:po[s + 1]]), (n,), W)
        check(cfg.dtype, host(z1[po[s]:po[s + 1]]), ref, f"tri_mul_in s={s} n={n}")


def _check_sampled(cfg, z0, z1, W, samples, npos, seed):
    po = np.concatenate([[0], np.cumsum(np.asarray(cfg.lengths, dtype=np.int64) ** 2)])
    rng = np.random.default_rng(seed)
    for s in samples:
        n = cfg.lengths[s]
        pos = [(int(a), int(b)) for a, b in zip(rng.integers(0, n, npos), rng.integers(0, n, npos))]
        pos += [(0, 0), (n - 1, n - 1), (0, n - 1), (n - 1, 0)]
        cols = sorted({i for i, _ in pos} | {j for _, j in pos})
        # only the needed columns of the sample's state cross to the host: zs[:, i] for the listed i
        zs_d = z0[po[s]:po[s + 1]].view(n, n, -1)
        fetched = {c: host(zs_d[:, c]) for c in cols}

        class Cols:
            def __getitem__(self, key):
                return fetched[key[1]]

        ref = orc.tri_mul_in_at(Cols(), W, pos)
        got = host(z1[torch.as_tensor([po[s] + i * n + j for i, j in pos], device=z1.device)])
        check(cfg.dtype, got, ref, f"tri_mul_in sampled s={s} n={n}")


def test_tri_mul_in_cfg1_f32(nt):
    cfg = wl.CONFIGS["cfg1"]
    z0, z1, W = _state_and_call(nt, cfg)
    _check_full(cfg, z0, z1, W, range(cfg.B))


@pytest.mark.parametrize("generic", [False, True])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_tri_mul_in_edge_lengths(nt, dtype, generic):
    # empty samples, one token, ragged tails around the 64 / 128 tile edges, several 128-row blocks
    cfg = wl.Config("edge_in", dtype, (0, 1, 7, 63, 64, 65, 0, 129, 200), c_s=32, c_z=128 if dtype == "bf16" else 16,
                    c_h=128 if dtype == "bf16" else 16, H=4 if dtype == "bf16" else 2, d=32 if dtype == "bf16" else 8,
                    blocks=1, seed=21)
    z0, z1, W = _state_and_call(nt, cfg, force_generic=generic)
    _check_full(cfg, z0, z1, W, range(cfg.B))
    # samples are independent: nothing outside the packed size was touched and empty samples add nothing
    assert z1.shape == z0.shape and torch.isfinite(z1.float()).all()


def test_tri_mul_in_c64(nt):
    cfg = wl.Config("in64", "bf16", (50, 131, 17), c_s=32, c_z=64, c_h=64, H=4, d=16, blocks=1, seed=22)
    z0, z1, W = _state_and_call(nt, cfg)
    _check_full(cfg, z0, z1, W, range(cfg.B))


def test_tri_mul_in_wide_sample_column_blocks(nt):
    # one sample wider than a 256-column block and not a multiple of 16
    cfg = wl.Config("in300", "bf16", (301, 12), c_s=32, c_z=128, c_h=128, H=4, d=32, blocks=1, seed=23)
    z0, z1, W = _state_and_call(nt, cfg)
    _check_full(cfg, z0, z1, W, [1])
    _check_sampled(cfg, z0, z1, W, [0], 24, seed=1)


def test_tri_mul_in_cfg2_sampled(nt):
    """The bench workload in the launch configuration bench.py times, at sampled positions."""
    cfg = wl.CONFIGS["cfg2"]
    z0, z1, W = _state_and_call(nt, cfg)
    _check_sampled(cfg, z0, z1, W, range(cfg.B), 12, seed=2)


def test_tri_mul_in_differs_from_out_and_is_deterministic(nt):
    from paper_2609_30379_b200 import runner
    cfg = wl.Config("in_det", "bf16", (40, 72), c_s=32, c_z=128, c_h=128, H=4, d=32, blocks=1, seed=24)
    z0, z1, W = _state_and_call(nt, cfg)
    z0b, z1b, _ = _state_and_call(nt, cfg)
    assert torch.equal(z0, z0b) and torch.equal(z1, z1b)
    inp = wl.make_inputs(cfg)
    st = runner.PairStack(cfg, cfg.lengths, inp["blocks"][:1])
    st.z.copy_(z0)
    nt.nt_tri_mul_out(st.L, st.W[0]["trimul"], 1e-5, st.z, st.workspace)
    torch.cuda.synchronize()
    assert not torch.equal(st.z, z1)
