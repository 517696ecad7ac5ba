"""Timing claims of the paper on this kernel.  Not part of the parity gate: these assert on measured times on a
shared machine, so they carry their own marker (`pytest -m timing` on a GPU machine) instead of `gpu`."""
import pytest
import torch

import bench

pytestmark = [pytest.mark.timing, pytest.mark.skipif(not torch.cuda.is_available(), reason="needs a CUDA device")]


@pytest.fixture(scope="module")
def ck():
    import paper_2608_30295_b200 as pkg
    return pkg.binding


def test_decode_time_follows_the_papers_efficiency_claims(ck):
    # Sections 4.4.1-4.4.3: latency grows linearly with the share of adaptive heads and with their retained
    # fraction, and the consistent heads' budget hardly matters.  Wide margins: this is a timing test.
    lin = bench.time_linearity(ck, "cuda")
    assert lin["r2_vs_r"] >= 0.99, lin
    assert lin["r2_vs_eta"] >= 0.99, lin
    t = lin["us_per_layer_step_vs_budget"]
    assert max(t) / min(t) <= 1.15, lin
    assert lin["us_per_layer_step_vs_r"][-1] > 3.0 * lin["us_per_layer_step_vs_r"][0], lin
