"""The block is capturable in a CUDA graph as it stands (no call allocates or synchronises); a replay gives what the
host-launched sequence gives."""
import pytest
import torch

from paper_2609_30379_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def test_captured_stack_replays_to_the_same_result():
    from paper_2609_30379_b200 import runner
    cfg = wl.Config("graph", "bf16", (40, 0, 72, 33), c_s=64, c_z=128, c_h=128, H=4, d=32, blocks=2, seed=51)
    inp = wl.make_inputs(cfg)
    st = runner.PairStack(cfg, cfg.lengths, inp["blocks"])
    x0 = runner.to_device(inp["x"], st.dtype)
    x = x0.clone()
    st.forward(x)
    torch.cuda.synchronize()
    want_x, want_z = x.clone(), st.z.clone()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        x.copy_(x0)
        graph = st.capture(x)
    torch.cuda.current_stream().wait_stream(side)
    for _ in range(2):                      # the second replay starts from the same tokens again
        x.copy_(x0)
        st.z.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(x, want_x) and torch.equal(st.z, want_z)
    assert st.L.device_status() == 0
