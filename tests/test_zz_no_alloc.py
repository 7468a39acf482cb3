"""janus_indexer_topk_static: the one-call indexer + top-k on the scratch array built into the library, through the C ABI.
Checked against janus_indexer_topk (caller's workspace) on the same inputs, twice in a row (the second call runs on
whatever the first left in the array), on a shape that takes the candidate-list route and one that takes the two-call
route; the device's free memory must not move across the calls; a problem beyond the array is refused.
The comparator is the library's own workspace call, not the oracle: that call's oracle check lives in
tests/test_gpu_fused.py and tests/test_gpu_fullsize.py, so agreement with it carries the oracle check over to this entry.
The file name sorts last on purpose: the array has then been used by nothing, or by anything, before."""
import numpy as np
import pytest
import torch

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


def make_inputs(seed, M, L, dtype):
    rng = np.random.default_rng(seed)
    H, D, S = 64, 128, L + M
    q = rng.standard_normal((M, H, D)).astype(np.float32)
    kk = rng.standard_normal((S, D)).astype(np.float32)
    w = (rng.uniform(0.0, 1.0, (M, H)) / 8).astype(np.float32)
    if dtype == "bf16":
        return dict(q=B.to_device(W.to_bf16_bits(q), "bf16"), k=B.to_device(W.to_bf16_bits(kk), "bf16"), w=B.to_device(w, "f32"), q_scale=None,
                    k_scale=None)
    return dict(q=B.to_device(W.to_e4m3_bits(2 * q), "fp8"), k=B.to_device(W.to_e4m3_bits(2 * kk), "fp8"), w=B.to_device(w, "f32"),
                q_scale=B.to_device(np.exp2(rng.uniform(-2, 2, H)).astype(np.float32), "f32"),
                k_scale=B.to_device(np.exp2(rng.uniform(-1, 1, S)).astype(np.float32), "f32"))


def same_selection(got, want, scores, L):
    """Same counts and k-th values; the index sets may differ only among scores tied with the k-th (order is free)."""
    (idx_g, cnt_g, kth_g), (idx_w, cnt_w, kth_w) = got, want
    assert np.array_equal(cnt_g, cnt_w)
    np.testing.assert_allclose(kth_g, kth_w, rtol=1e-6, atol=0.0)
    for t in range(idx_g.shape[0]):
        a, b = idx_g[t][idx_g[t] >= 0], idx_w[t][idx_w[t] >= 0]
        assert len(a) == len(np.unique(a)) == len(b) == cnt_w[t]
        assert a.max() <= L + t
        diff = np.setxor1d(a, b)
        assert np.all(scores[t, diff] == kth_w[t]), f"row {t}: selections differ away from the k-th score"


@pytest.mark.parametrize("M,L,dtype,k", [(24, 40000, "bf16", 512), (16, 66000, "fp8", 2048), (9, 3000, "bf16", 100)])
def test_static_scratch_matches_caller_workspace_twice_in_a_row(M, L, dtype, k):
    x = make_inputs(M * L, M, L, dtype)
    kw = dict(q_scale=x["q_scale"], k_scale=x["k_scale"], q_pos0=L, causal=True)
    idx_w, cnt_w, kth_w = B.janus_indexer_topk(x["q"], x["k"], x["w"], k, **kw)
    scores = B.janus_indexer_scores(x["q"], x["k"], x["w"], **kw)[:, :L + M].cpu().numpy()
    want = (idx_w.cpu().numpy(), cnt_w.cpu().numpy(), kth_w.cpu().numpy())

    idx = torch.empty((M, k), dtype=torch.int32, device="cuda")
    cnt = torch.empty((M,), dtype=torch.int32, device="cuda")
    kth = torch.empty((M,), dtype=torch.float32, device="cuda")
    free_before = None
    for call in range(2):
        idx.fill_(-7)
        cnt.fill_(-7)
        kth.fill_(float("nan"))
        torch.cuda.synchronize()
        if call == 1:
            free_before = torch.cuda.mem_get_info()[0]
        B.janus_indexer_topk_static(x["q"], x["k"], x["w"], k, idx, count=cnt, kth=kth, **kw)
        torch.cuda.synchronize()
        if call == 1:
            assert torch.cuda.mem_get_info()[0] == free_before, "the call changed the device's free memory"
        B.check_dev_status()
        same_selection((idx.cpu().numpy(), cnt.cpu().numpy(), kth.cpu().numpy()), want, scores, L)


def test_problem_beyond_the_built_in_scratch_is_refused():
    lib = B.load()
    M, L, k = 4096, 131072, 2048
    assert lib.janus_indexer_topk_workspace_size(M, 64, 128, L + M, L, 1, 1, k) > B.STATIC_SCRATCH_BYTES
    # pointers only need to look valid: the size check comes before anything is read or launched
    dummy = torch.zeros((64,), dtype=torch.int32, device="cuda")
    p = dummy.data_ptr()
    rc = lib.janus_indexer_topk_static(p, 64 * 128, p, 128, p, p, 0, p, None, None, M, 64, 128, L + M, L, 1, 1, k, p, None, None, None, None)
    assert rc == 3                                            # JANUS_ERR_WORKSPACE_TOO_SMALL
    torch.cuda.synchronize()
    assert int(dummy.sum().item()) == 0
