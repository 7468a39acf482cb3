"""The library's two diagnostic exports through the C ABI: the bounded wait that every tensor-core kernel relies on must give
up, report JANUS_DEV_WAIT_TIMEOUT and leave the context usable (the time-out path is otherwise never taken by a healthy
pipeline), and the dense FP8 tensor-rate probe must run clean and land in a plausible range."""
import numpy as np
import pytest
import torch

from oracle import janus_oracle as O
from paper_2609_36938_b200 import binding as B
from paper_2609_36938_b200 import build
from paper_2609_36938_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build()
    B.load()
    yield
    B.check_dev_status()


def test_bounded_wait_gives_up_reports_and_leaves_the_context_usable():
    status, seconds = B.janus_selftest_bounded_wait(256)
    assert status == 103                       # JANUS_DEV_WAIT_TIMEOUT
    assert seconds < 0.05, f"256 polls took {seconds * 1e3:.1f} ms"
    status2, seconds2 = B.janus_selftest_bounded_wait(2048)
    assert status2 == 103 and seconds2 < 0.25
    per_poll = (seconds2 - seconds) / (2048 - 256)
    print(f"bounded wait: {seconds * 1e6:.0f} us for 256 polls, {seconds2 * 1e6:.0f} us for 2048: {per_poll * 1e9:.0f} ns per poll")
    # the production limit must stay well under a second on a pipeline that is stuck
    assert per_poll * B.MBAR_MAX_POLLS < 0.5
    # an ordinary call on the same context afterwards: tensor-core indexer + top-k against the oracle
    shp = W.config_shape(3, L=1500, M=24, k=64)
    sess = W.make_session(shp, seed=3)
    sc = B.janus_indexer_scores(B.to_device(sess["q_idx"], "fp8"), B.to_device(sess["k_idx"], "fp8"), B.to_device(sess["w"], "f32"),
                                q_scale=B.to_device(sess["q_scale"], "f32"), k_scale=B.to_device(sess["k_scale"], "f32"), q_pos0=shp.L, causal=True)
    idx, _, _ = B.janus_topk(sc, shp.S, shp.k, q_pos0=shp.L, causal=True)
    B.check_dev_status()
    ref = O.indexer_scores(sess["q_idx"], sess["k_idx"], sess["w"], dtype="fp8", q_scale=sess["q_scale"], k_scale=sess["k_scale"], q_pos0=shp.L, causal=True)
    idx_h = idx.cpu().numpy()
    for t in range(shp.M):
        ok, msg = O.topk_row_agrees(idx_h[t], ref[t], shp.L + t + 1, shp.k)
        assert ok, msg


def test_fp8_tensor_rate_probe_runs_clean():
    n_sm = torch.cuda.get_device_properties(0).multi_processor_count
    B.janus_fp8_mma_probe(n_sm, 64)             # warm-up
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    flop = B.janus_fp8_mma_probe(n_sm, 4096)
    e1.record()
    torch.cuda.synchronize()
    B.check_dev_status()
    assert flop == 2.0 * 128 * 256 * 128 * 4096 * n_sm
    rate = flop / (e0.elapsed_time(e1) * 1e-3) / 1e12
    print(f"fp8 tensor-rate probe: {rate:.0f} TFLOP/s over {e0.elapsed_time(e1):.2f} ms")
    assert 500.0 < rate < 6000.0
