"""GPU parity of the column-wise ("ending node") pair-biased attention against the CPU oracle, through the C ABI.
The state it acts on is the one the block's broadcast produces from the seeded tokens."""
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
        nt.nt_col_attn_pairbias(st.L, w_d["attn"], cfg.H, cfg.d, 1e-5, st.z, st.workspace)
        torch.cuda.synchronize()
        assert st.L.device_status() == 0
        return z0, st.z.clone(), inp["blocks"][0]["attn"], st
    finally:
        nt.nt_force_generic(prev)


def _po(cfg):
    return np.concatenate([[0], np.cumsum(np.asarray(cfg.lengths, dtype=np.int64) ** 2)])


def _check_full(cfg, z0, z1, W, samples):
    po = _po(cfg)
    for s in samples:
        n = cfg.lengths[s]
        if n == 0:
            continue
        ref = orc.col_attn_pairbias(host(z0[po[s]:po[s + 1]]), (n,), W, cfg.H, cfg.d)
        check(cfg.dtype, host(z1[po[s]:po[s + 1]]), ref, f"col_attn s={s} n={n}")


def _check_sampled(cfg, z0, z1, W, samples, npos, seed):
    po = _po(cfg)
    rng = np.random.default_rng(seed)
    for s in samples:
        n = cfg.lengths[s]
        pos = [(int(a), int(b)) for a, b in zip(rng.integers(0, n, npos), rng.integers(0, n, npos))]
        pos += [(0, 0), (n - 1, n - 1), (0, n - 1), (n - 1, 0)]
        cols = sorted({i for i, _ in pos} | {j for _, j in pos})
        zs_d = z0[po[s]:po[s + 1]].view(n, n, -1)
        fetched = {c: host(zs_d[:, c]) for c in cols}

        class Cols:
            def __getitem__(self, key):
                return fetched[key[1]]

        ref = orc.col_attn_pairbias_at(Cols(), W, cfg.H, cfg.d, pos)
        got = host(z1[torch.as_tensor([po[s] + i * n + j for i, j in pos], device=z1.device)])
        check(cfg.dtype, got, ref, f"col_attn sampled s={s} n={n}")


def test_col_attn_cfg1_f32(nt):
    cfg = wl.CONFIGS["cfg1"]
    z0, z1, W, _ = _state_and_call(nt, cfg)
    _check_full(cfg, z0, z1, W, range(cfg.B))


@pytest.mark.parametrize("generic", [False, True])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_col_attn_edge_lengths(nt, dtype, generic):
    # empty samples, one token, ragged tails around the 16 / 32 / 128 edges, two query blocks
    bf = dtype == "bf16"
    cfg = wl.Config("edge_col", dtype, (0, 1, 7, 31, 33, 64, 0, 129, 200), c_s=32, c_z=128 if bf else 16,
                    c_h=128 if bf else 16, H=4 if bf else 2, d=32 if bf else 8, blocks=1, seed=41)
    z0, z1, W, _ = _state_and_call(nt, cfg, force_generic=generic)
    _check_full(cfg, z0, z1, W, range(cfg.B))
    assert torch.isfinite(z1.float()).all()


def test_col_attn_d16(nt):
    cfg = wl.Config("col16", "bf16", (50, 131, 17), c_s=32, c_z=64, c_h=64, H=4, d=16, blocks=1, seed=42)
    z0, z1, W, _ = _state_and_call(nt, cfg)
    _check_full(cfg, z0, z1, W, range(cfg.B))


def test_col_attn_sample_beyond_the_accumulator(nt):
    # 300 keys do not fit the tensor-core kernel's accumulator: that sample takes the shape-generic core,
    # the short one beside it the tcgen05 core, in one call
    cfg = wl.Config("col300", "bf16", (300, 40), c_s=32, c_z=128, c_h=128, H=4, d=32, blocks=1, seed=43)
    z0, z1, W, _ = _state_and_call(nt, cfg)
    _check_full(cfg, z0, z1, W, [1])
    _check_sampled(cfg, z0, z1, W, [0], 16, seed=3)


def test_col_attn_cfg2_sampled(nt):
    """The bench workload in the launch configuration bench.py times, at sampled positions."""
    cfg = wl.CONFIGS["cfg2"]
    z0, z1, W, _ = _state_and_call(nt, cfg)
    _check_sampled(cfg, z0, z1, W, range(cfg.B), 10, seed=4)


def test_col_attn_is_transposed_row_attn_on_device(nt):
    """Column attention of a state equals the transpose of row attention of the transposed state (both on the GPU)."""
    cfg = wl.Config("colT", "bf16", (37, 90), c_s=32, c_z=128, c_h=128, H=4, d=32, blocks=1, seed=44)
    z0, z1, W, st = _state_and_call(nt, cfg)
    po = _po(cfg)
    zT = torch.empty_like(z0)
    for s, n in enumerate(cfg.lengths):
        zT[po[s]:po[s + 1]] = z0[po[s]:po[s + 1]].view(n, n, -1).transpose(0, 1).reshape(n * n, -1)
    st.z.copy_(zT)
    nt.nt_row_attn_pairbias(st.L, nt.NT_ORDER_PAIR_IJC, st.W[0]["attn"], cfg.H, cfg.d, 1e-5, st.z, st.workspace)
    torch.cuda.synchronize()
    back = torch.empty_like(z0)
    for s, n in enumerate(cfg.lengths):
        back[po[s]:po[s + 1]] = st.z[po[s]:po[s + 1]].view(n, n, -1).transpose(0, 1).reshape(n * n, -1)
    # two independently rounded bf16 results, each within the tolerance of the exact value: twice the tolerance apart at most
    from tests.parity_utils import ln0, BF16_ATOL_AFTER_LN
    worst = float(np.abs(ln0(host(z1)) - ln0(host(back))).max())
    assert worst <= 2 * BF16_ATOL_AFTER_LN, worst
