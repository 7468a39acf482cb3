"""janus_indexer_topk (indexer + top-k without the score matrix) through the C ABI: against the oracle on sampled rows,
against the two-call path on all rows, on inputs built to make the sampled threshold fail (so the exact fallback runs),
and on shapes that take the internal two-call route."""
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


def dev(x, kind):
    return B.to_device(x, kind)


def sample_positions(p0: int) -> np.ndarray:
    """Key positions the library samples: 512 chunks of 8 consecutive keys spread evenly over [0, p0) (see janus.h)."""
    n8 = p0 // 8
    j = np.arange(4096)
    return 8 * ((j // 8) * (n8 - 1) // 511) + (j % 8)


def make_case(seed, M, L, H, D, dtype, bias):
    rng = np.random.default_rng(seed)
    S = L + M
    q = rng.standard_normal((M, H, D)).astype(np.float32)
    kk = rng.standard_normal((S, D)).astype(np.float32)
    c = {"w": rng.uniform(0.0, 1.0, (M, H)).astype(np.float32) / 8, "dtype": dtype, "q_scale": None, "k_scale": None, "row_bias": None,
         "col_bias": None, "L": L, "M": M}
    if dtype == "bf16":
        c["q"], c["k"] = W.to_bf16_bits(q), W.to_bf16_bits(kk)
    else:
        c["q"], c["k"] = W.to_e4m3_bits(q * 2), W.to_e4m3_bits(kk * 2)
        c["q_scale"] = np.exp2(rng.uniform(-2, 2, H)).astype(np.float32)
        c["k_scale"] = np.exp2(rng.uniform(-1, 1, S)).astype(np.float32)
    if bias:
        c["row_bias"] = rng.uniform(0.5, 2.0, M).astype(np.float32)
        c["col_bias"] = rng.uniform(0.0, 3.0, S).astype(np.float32)
    return c


def run_both(c, k, causal=True):
    kind = c["dtype"]
    args = dict(q_scale=dev(c["q_scale"], "f32"), k_scale=dev(c["k_scale"], "f32"), row_bias=dev(c["row_bias"], "f32"),
                col_bias=dev(c["col_bias"], "f32"), q_pos0=c["L"], causal=causal)
    q, kk, w = dev(c["q"], kind), dev(c["k"], kind), dev(c["w"], "f32")
    idx_f, cnt_f, kth_f = B.janus_indexer_topk(q, kk, w, k, **args)
    sc = B.janus_indexer_scores(q, kk, w, **args)
    idx_u, cnt_u, kth_u = B.janus_topk(sc, kk.shape[0], k, q_pos0=c["L"], causal=causal)
    B.check_dev_status()
    return (idx_f.cpu().numpy(), cnt_f.cpu().numpy(), kth_f.cpu().numpy()), (idx_u.cpu().numpy(), cnt_u.cpu().numpy(), kth_u.cpu().numpy()), \
        sc[:, :kk.shape[0]].cpu().numpy()


def check_against_two_call(fused, unfused, scores, k, L, causal=True):
    """Same fp32 scores feed both paths, so the k-th value is identical and the sets agree except among ties at it."""
    (idx_f, cnt_f, kth_f), (idx_u, cnt_u, kth_u) = fused, unfused
    assert np.array_equal(cnt_f, cnt_u)
    assert np.array_equal(kth_f, kth_u)
    for t in range(idx_f.shape[0]):
        n = scores.shape[1] if not causal else min(scores.shape[1], L + t + 1)
        a, b = idx_f[t][idx_f[t] >= 0], idx_u[t][idx_u[t] >= 0]
        assert len(a) == len(np.unique(a)) == len(b) and a.max() < n
        diff = np.setxor1d(a, b)
        assert np.all(scores[t, diff] == kth_u[t]), f"row {t}: sets differ away from the threshold"


@pytest.mark.parametrize("M,L,dtype,bias,k", [(40, 40000, "bf16", False, 512), (37, 70001, "fp8", True, 2048), (20, 20000, "bf16", True, 64)])
def test_fused_matches_oracle_and_two_call_path(M, L, dtype, bias, k):
    c = make_case(M + L, M, L, 64, 128, dtype, bias)
    fused, unfused, scores = run_both(c, k)
    check_against_two_call(fused, unfused, scores, k, L)
    for t in W.sample_rows(M, 4):
        t = int(t)
        ref = O.indexer_scores(c["q"][t:t + 1], c["k"], c["w"][t:t + 1], dtype=dtype, q_scale=c["q_scale"], k_scale=c["k_scale"],
                               row_bias=None if c["row_bias"] is None else c["row_bias"][t:t + 1], col_bias=c["col_bias"], q_pos0=L + t,
                               causal=True)[0]
        ok, msg = O.topk_row_agrees(fused[0][t], ref, L + t + 1, k)
        assert ok, f"row {t}: {msg}"


def test_fused_non_causal_prediction_pass():
    c = make_case(5, 24, 33000, 64, 128, "bf16", False)
    c["k"] = c["k"][:33000]                                   # history keys only, every row sees all of them
    fused, unfused, scores = run_both(c, 256, causal=False)
    check_against_two_call(fused, unfused, scores, 256, 33000, causal=False)


def test_fallback_when_the_sample_overestimates_the_threshold():
    # only the sampled keys are large: the threshold lands far above the row's true k-th score, too few candidates are kept,
    # and every row must be recomputed exactly
    M, L, k = 6, 30000, 512
    c = make_case(11, M, L, 64, 128, "bf16", False)
    kk = O.decode_bf16(c["k"]).astype(np.float32)
    pos = sample_positions(L + 1)
    kk[pos] *= 6.0
    c["k"] = W.to_bf16_bits(kk)
    fused, unfused, scores = run_both(c, k)
    # the fallback recomputes the rows on the fp32 ALUs (another summation order than the tensor-core kernel), so it is
    # compared with the oracle and only approximately with the two-call path
    assert np.array_equal(fused[1], unfused[1])
    np.testing.assert_allclose(fused[2], unfused[2], rtol=1e-5)
    for t in range(M):
        ref = O.indexer_scores(c["q"][t:t + 1], c["k"], c["w"][t:t + 1], dtype="bf16", q_pos0=L + t, causal=True)[0]
        ok, msg = O.topk_row_agrees(fused[0][t], ref, L + t + 1, k)
        assert ok, f"row {t}: {msg}"


def test_fallback_when_too_many_scores_tie_at_the_threshold():
    # every key identical: all scores of a row are equal, the whole row passes the threshold and overflows the candidate list
    M, L, k = 5, 25000, 300
    c = make_case(12, M, L, 64, 128, "fp8", False)
    c["k"] = np.repeat(c["k"][:1], L + M, axis=0)
    c["k_scale"] = np.full(L + M, 0.5, np.float32)
    fused, unfused, scores = run_both(c, k)
    (idx_f, cnt_f, kth_f) = fused
    assert np.array_equal(cnt_f, np.full(M, k))
    for t in range(M):
        ok, msg = O.topk_row_agrees(idx_f[t], scores[t].astype(np.float64), L + t + 1, k)
        assert ok, msg
        assert kth_f[t] == pytest.approx(scores[t, 0], rel=1e-5)


@pytest.mark.parametrize("M,n_keys,H,D,dtype,k", [(9, 3000, 64, 128, "bf16", 100), (5, 40000, 3, 48, "bf16", 64), (7, 20000, 64, 128, "fp8", 5000)])
def test_two_call_route_inside_the_fused_entry(M, n_keys, H, D, dtype, k):
    # few keys, a head count the tensor-core kernel does not take, or k above the candidate budget
    L = n_keys - M
    c = make_case(M * n_keys, M, L, H, D, dtype, False)
    fused, unfused, scores = run_both(c, k)
    check_against_two_call(fused, unfused, scores, k, L)


def test_workspace_contract():
    lib = B.load()
    fused_bytes = lib.janus_indexer_topk_workspace_size(4096, 64, 128, 135168, 131072, 1, 1, 2048)
    two_call_bytes = 4096 * 135168 * 4
    assert 0 < fused_bytes < two_call_bytes                  # the point of the fused path: no score matrix
    c = make_case(3, 8, 20000, 64, 128, "bf16", False)
    q, kk, w = dev(c["q"], "bf16"), dev(c["k"], "bf16"), dev(c["w"], "f32")
    idx = torch.empty((8, 64), dtype=torch.int32, device="cuda")
    small = torch.empty((1024,), dtype=torch.uint8, device="cuda")
    rc = lib.janus_indexer_topk(q.data_ptr(), 64 * 128, kk.data_ptr(), 128, w.data_ptr(), None, 0, None, None, None, 8, 64, 128, 20008, 20000, 1, 0,
                                64, idx.data_ptr(), None, None, small.data_ptr(), small.numel(), None, None)
    assert rc == 3                                            # JANUS_ERR_WORKSPACE_TOO_SMALL, nothing launched
    rc = lib.janus_indexer_topk(q.data_ptr(), 64 * 128, kk.data_ptr(), 128, w.data_ptr(), None, 0, None, None, None, 8, 64, 128, 20008, 20000, 1, 0,
                                0, idx.data_ptr(), None, None, small.data_ptr(), small.numel(), None, None)
    assert rc == 1                                            # k = 0
