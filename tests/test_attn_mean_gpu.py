"""GPU parity of the fused call (row-wise pair-biased attention followed by the mean over j of the updated state)
against the CPU oracle and against the two separate calls, through the C ABI."""
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


def _run(nt, cfg, force_generic=False):
    """Broadcast (checked elsewhere), then the fused call on one copy of the state and the two calls on another."""
    from paper_2609_30379_b200 import runner
    inp = wl.make_inputs(cfg)
    prev = nt.nt_force_generic(force_generic)
    try:
        st = runner.PairStack(cfg, cfg.lengths, inp["blocks"][:1])
        w = st.W[0]
        x = runner.to_device(inp["x"], st.dtype)
        b = w["broadcast"]
        nt.nt_pair_broadcast(st.L, x, b["W_a"], b["W_b"], b["ln_gamma"], b["ln_beta"], 1e-5, st.z, st.workspace)
        z0 = st.z.clone()
        m_f = torch.full_like(st.m, float("nan"))
        nt.nt_row_attn_pairbias_mean(st.L, w["attn"], cfg.H, cfg.d, 1e-5, st.z, m_f, st.workspace)
        z_f = st.z.clone()
        st.z.copy_(z0)
        m_s = torch.full_like(st.m, float("nan"))
        nt.nt_row_attn_pairbias(st.L, nt.NT_ORDER_PAIR_IJC, w["attn"], cfg.H, cfg.d, 1e-5, st.z, st.workspace)
        nt.nt_segment_reduce(nt.NT_REDUCE_MEAN, st.L.row_splits, st.z, m_s, st.L.status)
        torch.cuda.synchronize()
        assert st.L.device_status() == 0
        return z0, z_f, m_f, st.z.clone(), m_s, inp["blocks"][0]["attn"]
    finally:
        nt.nt_force_generic(prev)


def _check_against_oracle(cfg, z0, z_f, m_f, W, samples):
    n_all = np.asarray(cfg.lengths, dtype=np.int64)
    po = np.concatenate([[0], np.cumsum(n_all ** 2)])
    to = np.concatenate([[0], np.cumsum(n_all)])
    for s in samples:
        n = cfg.lengths[s]
        if n == 0:
            continue
        ref = orc.row_attn_pairbias(host(z0[po[s]:po[s + 1]]), (n,), W, cfg.H, cfg.d)
        check(cfg.dtype, host(z_f[po[s]:po[s + 1]]), ref, f"fused attention state s={s} n={n}")
        ref_m = ref.reshape(n, n, -1).mean(axis=1)
        check(cfg.dtype, host(m_f[to[s]:to[s + 1]]), ref_m, f"fused mean s={s} n={n}")


@pytest.mark.parametrize("lengths", [(40, 72, 0, 33), (32, 129, 64), (0, 0, 97)])
def test_fused_mean_matches_oracle_and_separate_calls(nt, lengths):
    cfg = wl.Config("fm", "bf16", lengths, c_s=32, c_z=128, c_h=128, H=4, d=32, blocks=1, seed=41)
    z0, z_f, m_f, z_s, m_s, W = _run(nt, cfg)
    assert torch.equal(z_f, z_s)                       # the state is what the attention alone leaves
    assert torch.isfinite(m_f.float()).all()
    # same sums in another order, then one rounding to bf16: at most one unit in the last place apart
    assert (m_f.float() - m_s.float()).abs().max().item() <= 2.0 ** -7 * max(1.0, m_s.float().abs().max().item())
    _check_against_oracle(cfg, z0, z_f, m_f, W, range(cfg.B))


def test_fused_mean_short_samples_take_the_separate_reduction(nt):
    # a sample shorter than 32 switches the fused column sums off; the call still returns the mean
    cfg = wl.Config("fm_short", "bf16", (7, 50, 1, 31), c_s=32, c_z=128, c_h=128, H=4, d=32, blocks=1, seed=42)
    z0, z_f, m_f, z_s, m_s, W = _run(nt, cfg)
    assert torch.equal(z_f, z_s) and torch.equal(m_f, m_s)
    _check_against_oracle(cfg, z0, z_f, m_f, W, range(cfg.B))


@pytest.mark.parametrize("dtype,generic", [("f32", False), ("bf16", True)])
def test_fused_mean_generic_paths(nt, dtype, generic):
    cfg = wl.Config("fm_gen", dtype, (40, 0, 35), c_s=32, c_z=16 if dtype == "f32" else 128, c_h=16, H=2 if dtype == "f32" else 4,
                    d=8 if dtype == "f32" else 32, blocks=1, seed=43)
    z0, z_f, m_f, z_s, m_s, W = _run(nt, cfg, force_generic=generic)
    assert torch.equal(z_f, z_s) and torch.equal(m_f, m_s)
    _check_against_oracle(cfg, z0, z_f, m_f, W, range(cfg.B))


def test_fused_mean_c64(nt):
    cfg = wl.Config("fm64", "bf16", (50, 131, 36), c_s=32, c_z=64, c_h=64, H=4, d=16, blocks=1, seed=44)
    z0, z_f, m_f, z_s, m_s, W = _run(nt, cfg)
    assert torch.equal(z_f, z_s)
    _check_against_oracle(cfg, z0, z_f, m_f, W, range(cfg.B))


def test_fused_mean_many_samples_cross_group_boundaries(nt):
    # more samples than one kernel group takes: the partial sums restart with every group
    rng = np.random.default_rng(5)
    lengths = tuple(int(v) for v in rng.integers(32, 41, 70))
    cfg = wl.Config("fm_many", "bf16", lengths, c_s=32, c_z=128, c_h=128, H=4, d=32, blocks=1, seed=45)
    z0, z_f, m_f, z_s, m_s, W = _run(nt, cfg)
    assert torch.equal(z_f, z_s)
    assert (m_f.float() - m_s.float()).abs().max().item() <= 2.0 ** -7 * max(1.0, m_s.float().abs().max().item())
    _check_against_oracle(cfg, z0, z_f, m_f, W, [0, 1, 63, 64, 69])


def test_fused_mean_cfg2_sampled_rows(nt):
    """The bench workload: the fused mean of sampled pair rows against the float mean of the library's own final state
    (the state itself is checked against the oracle by the attention parity tests)."""
    cfg = wl.CONFIGS["cfg2"]
    z0, z_f, m_f, z_s, m_s, W = _run(nt, cfg)
    assert torch.equal(z_f, z_s)
    n_all = np.asarray(cfg.lengths, dtype=np.int64)
    po = np.concatenate([[0], np.cumsum(n_all ** 2)])
    to = np.concatenate([[0], np.cumsum(n_all)])
    rng = np.random.default_rng(3)
    for s in range(cfg.B):
        n = cfg.lengths[s]
        for i in [0, n - 1] + [int(v) for v in rng.integers(0, n, 6)]:
            ref = host(z_f[po[s] + i * n: po[s] + (i + 1) * n]).mean(axis=0)
            got = host(m_f[to[s] + i])
            assert np.abs(got - ref).max() <= 2.0 ** -8 * max(1.0, np.abs(ref).max()), (s, i)
