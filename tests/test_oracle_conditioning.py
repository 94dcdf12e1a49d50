"""Why gradient tolerances on deep networks cannot be 1e-4 in fp32: the oracle run in
float32 against the oracle run in float64 on the same inputs.  The forward pass agrees
to ~1e-6, the gradient only to ~1e-2, because rounding flips a few ReLU gates and each
flip moves its gradient element by O(1)."""
import numpy as np

import fdg_synth as S
from oracle import fdg, nets


def test_fp32_vs_fp64_gradient_gap_on_a_deep_network():
    arch = nets.Arch(n_per_stage=9, batch=4)          # ResNet-56 layers, small batch to stay fast
    out = []
    for dt in (np.float64, np.float32):
        o = fdg.FDGOracle(arch, fdg.FDGConfig(K=1, split_after_block=(), lr=0.0), dtype=dt)
        o.set_params(1, S.init_params(0, 1, o.param_spec(1)))
        loss = o.step(S.images(0, 1, 4, 32, 32, 3), S.labels(0, 1, 4, 10))
        out.append((loss, o.get_grads(1).astype(np.float64)))
    (l64, g64), (l32, g32) = out
    assert abs(l32 - l64) / l64 < 1e-5
    gap = np.linalg.norm(g32 - g64) / np.linalg.norm(g64)
    assert 1e-4 < gap < 0.3, gap
