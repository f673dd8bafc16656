"""Per-kernel parity: each step of the path, called through the C ABI, against the CPU oracle's
definition of that step on the same seeded inputs.

Tolerances (per-tensor max|a-b| <= tol * max|b|): bf16 2e-2 is the bound for hidden states and
logits over a whole layer stack; a single step rounds once, so single steps are held to 1e-2;
fp32 mode 1e-4; Eq. 1 scores 1e-3 absolute; indices bit-exact.
"""
import numpy as np
import pytest
import torch

import lazyllm_oracle as O
from paper_2407_14057_b200 import binding as B
from paper_2407_14057_b200 import build, synth
from helpers import rel_err, to_np

pytestmark = pytest.mark.gpu

BF16_STEP_TOL = 1e-2
F32_TOL = 1e-4


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build()
    B.lib()
    yield
    B.lazy_device_status()


def _rand(shape, seed, dtype, std=1.0):
    g = torch.Generator().manual_seed(seed)
    return (torch.randn(shape, generator=g, dtype=torch.float32) * std).to(dtype)


def _tol(dtype):
    return F32_TOL if dtype == torch.float32 else BF16_STEP_TOL


# ------------------------------------------------------------------------------------------ rmsnorm
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("n,d", [(1, 256), (37, 256), (300, 4096)])
def test_rmsnorm(dtype, n, d):
    x = _rand((n, d), 1, dtype, 3.0)
    g = (1 + 0.1 * _rand((d,), 2, torch.float32)).to(dtype)
    y = B.lazy_k_rmsnorm(x.cuda(), g.cuda(), 1e-6)
    ref = O.rmsnorm(to_np(x), to_np(g), 1e-6)
    assert rel_err(to_np(y), ref) < _tol(dtype)


# ------------------------------------------------------------------------------------------ GEMM
GEMM_SHAPES = [(128, 256, 64), (1, 256, 64), (300, 512, 320), (257, 1376, 688), (129, 768, 256),
               (1000, 4096, 4096)]


@pytest.mark.parametrize("M,N,K", GEMM_SHAPES)
@pytest.mark.parametrize("residual", [False, True])
def test_gemm_bf16_tensor_core(M, N, K, residual):
    A = _rand((M, K), 3, torch.bfloat16)
    Bm = _rand((N, K), 4, torch.bfloat16, 0.05)
    R = _rand((M, N), 5, torch.bfloat16) if residual else None
    out = B.lazy_k_gemm(A.cuda(), Bm.cuda(), None if R is None else R.cuda())
    B.lazy_device_status()
    ref = O.f64(to_np(A)) @ O.f64(to_np(Bm)).T
    if residual:
        ref = ref + O.f64(to_np(R))
    assert rel_err(to_np(out), ref) < BF16_STEP_TOL
    # element-wise: bf16 rounding of the exact value, plus fp32 accumulation noise
    err = np.abs(to_np(out).astype(np.float64) - ref)
    assert np.all(err <= 2.0 ** -8 * np.abs(ref) + 1e-3 * np.max(np.abs(ref)))


@pytest.mark.parametrize("impl", [2, 3])
@pytest.mark.parametrize("M,N,K", [(130, 8, 64), (37, 72, 128), (200, 200, 256), (129, 136, 64), (300, 264, 320)])
def test_gemm_bf16_narrow_and_ragged_output_widths(M, N, K, impl):
    """Outputs narrower than one 64-column store box, or ending inside one, with row counts that end inside a
    32-row box: the epilogues stage whole boxes and rely on the store unit to drop what lies outside the
    matrix, so nothing may be written beyond it (the output sits inside a larger poisoned buffer) and every
    element inside must be right.  Both tensor-core kernels, with and without the residual."""
    A = _rand((M, K), 80, torch.bfloat16).cuda()
    Bm = _rand((N, K), 81, torch.bfloat16, 0.05).cuda()
    R = _rand((M, N), 82, torch.bfloat16).cuda()
    ws = B.lazy_k_gemm_scratch()
    ref0 = O.f64(to_np(A)) @ O.f64(to_np(Bm)).T
    for res in (None, R):
        guard = torch.full(((M + 64) * N + 256,), 777.0, dtype=torch.bfloat16, device="cuda")
        out = guard[128:128 + M * N].view(M, N)
        B.lazy_k_gemm(A, Bm, res, impl=impl, out=out, scratch=ws)
        B.lazy_device_status()
        ref = ref0 + (O.f64(to_np(res)) if res is not None else 0.0)
        assert rel_err(to_np(out), ref) < BF16_STEP_TOL
        assert torch.all(guard[:128] == 777.0) and torch.all(guard[128 + M * N:] == 777.0)


def test_gemm_bf16_in_place_residual_and_cuda_core_cross_check():
    M, N, K = 200, 512, 1408
    A = _rand((M, K), 6, torch.bfloat16).cuda()
    Bm = _rand((N, K), 7, torch.bfloat16, 0.05).cuda()
    x = _rand((M, N), 8, torch.bfloat16).cuda()
    ref = O.f64(to_np(A)) @ O.f64(to_np(Bm)).T + O.f64(to_np(x))
    simt = B.lazy_k_gemm(A, Bm, x, impl=1)
    B.lazy_k_gemm(A, Bm, x, out=x)          # x += A B^T in place
    B.lazy_device_status()
    assert rel_err(to_np(x), ref) < BF16_STEP_TOL
    assert rel_err(to_np(simt), ref) < BF16_STEP_TOL


@pytest.mark.parametrize("M,N,K", [(64, 256, 64), (70, 688, 256), (33, 256, 688)])
def test_gemm_fp32(M, N, K):
    A = _rand((M, K), 9, torch.float32)
    Bm = _rand((N, K), 10, torch.float32, 0.05)
    R = _rand((M, N), 11, torch.float32)
    out = B.lazy_k_gemm(A.cuda(), Bm.cuda(), R.cuda())
    ref = O.f64(to_np(A)) @ O.f64(to_np(Bm)).T + O.f64(to_np(R))
    assert rel_err(to_np(out), ref) < F32_TOL


@pytest.mark.parametrize("M,N,K", [(129, 256, 64), (256, 512, 128), (300, 1376, 688), (513, 4096, 4096),
                                   (3376, 768, 4096), (1013, 4096, 11008),
                                   (13000, 512, 4096), (4600, 768, 11008)])   # A beyond 96 MiB: banded tile order
def test_gemm_bf16_cta_pair_kernel_against_one_cta_kernel_and_oracle(M, N, K):
    """Above 128 rows a product runs on CTA pairs (256x256 tiles over two SMs, impl=3) or with one CTA per
    128x256 tile (impl=2), whichever is faster for the shape.  Both accumulate a tile's K range in the same
    order in fp32, so they agree to the last bit, and both match the fp64 product."""
    A = _rand((M, K), 21, torch.bfloat16).cuda()
    Bm = _rand((N, K), 22, torch.bfloat16, 0.05).cuda()
    R = _rand((M, N), 23, torch.bfloat16).cuda()
    pair = B.lazy_k_gemm(A, Bm, R, impl=3)
    one = B.lazy_k_gemm(A, Bm, R, impl=2)
    auto = B.lazy_k_gemm(A, Bm, R)
    B.lazy_device_status()
    ref = O.f64(to_np(A)) @ O.f64(to_np(Bm)).T + O.f64(to_np(R))
    assert rel_err(to_np(pair), ref) < BF16_STEP_TOL
    assert rel_err(to_np(one), ref) < BF16_STEP_TOL
    assert torch.equal(pair, one) and torch.equal(auto, one)
    F = min(N, 1408)
    g_pair = B.lazy_k_gemm_swiglu(A, Bm[:F // 2].contiguous(), Bm[F // 2:F].contiguous(), impl=3)
    g_one = B.lazy_k_gemm_swiglu(A, Bm[:F // 2].contiguous(), Bm[F // 2:F].contiguous(), impl=2)
    B.lazy_device_status()
    a = O.f64(to_np(A))
    ref = O.silu(a @ O.f64(to_np(Bm[:F // 2])).T) * (a @ O.f64(to_np(Bm[F // 2:F])).T)
    assert rel_err(to_np(g_pair), ref) < BF16_STEP_TOL
    assert torch.equal(g_pair, g_one)


@pytest.mark.parametrize("impl", [3, 2])
@pytest.mark.parametrize("M,N,K", [(2364, 4096, 4096), (1013, 4096, 11008), (1688, 12288, 4096), (600, 2048, 1024),
                                   (130, 256, 4096), (3376, 4096, 512), (12500, 768, 4096)])
def test_gemm_bf16_split_last_wave_matches_plain_tile_loop(M, N, K, impl):
    """With a scratch the kernels cut the K loops of the last partial wave of tiles across all SMs and add
    the parts in a fixed order: same answer as without (to fp32 re-association inside split tiles), right
    against fp64, identical from run to run, and the scratch is all zero again afterwards."""
    A = _rand((M, K), 31, torch.bfloat16).cuda()
    Bm = _rand((N, K), 32, torch.bfloat16, 0.05).cuda()
    R = _rand((M, N), 33, torch.bfloat16).cuda()
    ws = B.lazy_k_gemm_scratch()
    plain = B.lazy_k_gemm(A, Bm, R, impl=impl)
    split = B.lazy_k_gemm(A, Bm, R, impl=impl, scratch=ws)
    again = B.lazy_k_gemm(A, Bm, R, impl=impl, scratch=ws)
    B.lazy_device_status()
    ref = O.f64(to_np(A)) @ O.f64(to_np(Bm)).T + O.f64(to_np(R))
    assert rel_err(to_np(split), ref) < BF16_STEP_TOL
    assert rel_err(to_np(split), to_np(plain).astype(np.float64)) < 2.0 ** -7   # one bf16 rounding flip
    assert torch.equal(split, again)
    assert int(ws[:2048].count_nonzero()) == 0   # the arrival counters (first 2 KiB) are back to zero
    F = min(N // 2, 1408)
    g_plain = B.lazy_k_gemm_swiglu(A, Bm[:F].contiguous(), Bm[F:2 * F].contiguous(), impl=impl)
    g_split = B.lazy_k_gemm_swiglu(A, Bm[:F].contiguous(), Bm[F:2 * F].contiguous(), impl=impl, scratch=ws)
    B.lazy_device_status()
    a = O.f64(to_np(A))
    ref = O.silu(a @ O.f64(to_np(Bm[:F])).T) * (a @ O.f64(to_np(Bm[F:2 * F])).T)
    assert rel_err(to_np(g_split), ref) < BF16_STEP_TOL
    assert rel_err(to_np(g_split), to_np(g_plain).astype(np.float64)) < 2.0 ** -7


@pytest.mark.parametrize("M", [1, 2, 3, 4, 5])
def test_gemm_bf16_few_rows_weight_streaming_kernel(M):
    """M <= 4 takes the weight-streaming kernel, M = 5 the tensor-core one: same answers."""
    N, K = 4096, 11008
    A = _rand((M, K), 16, torch.bfloat16)
    Bm = _rand((N, K), 17, torch.bfloat16, 0.02)
    R = _rand((M, N), 18, torch.bfloat16)
    out = B.lazy_k_gemm(A.cuda(), Bm.cuda(), R.cuda())
    B.lazy_device_status()
    ref = O.f64(to_np(A)) @ O.f64(to_np(Bm)).T + O.f64(to_np(R))
    assert rel_err(to_np(out), ref) < BF16_STEP_TOL
    g = B.lazy_k_gemm_swiglu(A.cuda(), Bm[:1024].contiguous().cuda(), Bm[1024:2048].contiguous().cuda())
    B.lazy_device_status()
    a = O.f64(to_np(A))
    ref = O.silu(a @ O.f64(to_np(Bm[:1024])).T) * (a @ O.f64(to_np(Bm[1024:2048])).T)
    assert rel_err(to_np(g), ref) < BF16_STEP_TOL


@pytest.mark.parametrize("dtype,M,F,K", [(torch.bfloat16, 300, 1408, 512), (torch.bfloat16, 128, 128, 64),
                                         (torch.bfloat16, 77, 688, 256), (torch.bfloat16, 500, 11008, 4096),
                                         (torch.float32, 70, 688, 256)])
def test_gemm_swiglu(dtype, M, F, K):
    A = _rand((M, K), 12, dtype)
    Bg = _rand((F, K), 13, dtype, 0.05)
    Bu = _rand((F, K), 14, dtype, 0.05)
    out = B.lazy_k_gemm_swiglu(A.cuda(), Bg.cuda(), Bu.cuda())
    B.lazy_device_status()
    a = O.f64(to_np(A))
    ref = O.silu(a @ O.f64(to_np(Bg)).T) * (a @ O.f64(to_np(Bu)).T)
    assert rel_err(to_np(out), ref) < _tol(dtype)


def test_gemm_empty_rows_is_a_no_op():
    A = torch.empty((0, 64), dtype=torch.bfloat16, device="cuda")
    Bm = _rand((256, 64), 1, torch.bfloat16).cuda()
    assert B.lazy_k_gemm(A, Bm).shape == (0, 256)


# ------------------------------------------------------------------- selection, threshold form
@pytest.mark.parametrize("prune_bp", [0, 3000, 5000, 9999])
def test_select_threshold_matches_oracle_bit_for_bit_with_ties(prune_bp):
    rng = np.random.default_rng(3)
    lengths = [1, 5, 1024, 1025, 4097, 300, 0, 2]
    parts = []
    for n in lengths:
        sc = rng.random(n).astype(np.float32)
        if n >= 300:
            sc[rng.integers(0, n, n // 3)] = sc[n // 2]        # plant ties, some of them at the threshold
        parts.append(sc)
    cu = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
    scores = torch.tensor(np.concatenate(parts)).cuda()
    keep, drop, counts = B.lazy_k_select_threshold(scores, torch.tensor(cu).cuda(), prune_bp)
    B.lazy_device_status()
    keep, drop, counts = to_np(keep), to_np(drop), to_np(counts)
    for s, n in enumerate(lengths):
        k_ref, d_ref = O.select_threshold(parts[s], prune_bp)
        assert counts[s] == len(k_ref)
        assert np.array_equal(keep[cu[s]:cu[s] + counts[s]] - cu[s], k_ref)
        assert np.array_equal(drop[cu[s]:cu[s] + n - counts[s]] - cu[s], d_ref)


# ------------------------------------------------------------------------------------------ RoPE
@pytest.mark.parametrize("dtype,H,dh", [(torch.float32, 4, 64), (torch.bfloat16, 4, 128)])
def test_rope_and_kv_write(dtype, H, dh):
    n, d = 50, H * dh
    qkv = _rand((n, 3 * d), 15, dtype)
    pos = torch.tensor(sorted(np.random.default_rng(0).choice(4000, n, replace=False)), dtype=torch.int32)
    dev = qkv.cuda()
    kc, vc = B.lazy_k_rope_kv(dev, pos.cuda(), H, dh, 4096, 1e4)
    B.lazy_device_status()
    x = to_np(qkv)
    q_ref = O.rope(x[:, :d].reshape(n, H, dh), to_np(pos), 1e4).reshape(n, d)
    k_ref = O.rope(x[:, d:2 * d].reshape(n, H, dh), to_np(pos), 1e4).reshape(n, d)
    got = to_np(dev)
    assert rel_err(got[:, :d], q_ref) < _tol(dtype)
    assert rel_err(to_np(kc), k_ref) < _tol(dtype)
    assert np.array_equal(to_np(vc), x[:, 2 * d:])           # v is a plain copy
    assert np.array_equal(got[:, 2 * d:], x[:, 2 * d:])


# ------------------------------------------------------------------------------------------ attention
def _attention_case(dtype, H, dh, lengths, seed):
    n = sum(lengths)
    d = H * dh
    q = _rand((n, d), seed, dtype)
    k = _rand((n, d), seed + 1, dtype)
    v = _rand((n, d), seed + 2, dtype)
    cu = np.concatenate([[0], np.cumsum(lengths)]).astype(np.int32)
    o = B.lazy_k_attention(q.cuda(), d, k.cuda(), v.cuda(), d, torch.tensor(cu).cuda(), max(lengths), n, H, dh)
    s = B.lazy_k_score(q.cuda(), d, k.cuda(), d, torch.tensor(cu).cuda(), n, H, dh)
    B.lazy_device_status()
    o_ref = np.zeros((n, d))
    s_ref = np.zeros(n)
    for a, b in zip(cu[:-1], cu[1:]):
        pos = np.arange(b - a)
        oo, ss = O.attend(to_np(q)[a:b].reshape(-1, H, dh), to_np(k)[a:b].reshape(-1, H, dh),
                          to_np(v)[a:b].reshape(-1, H, dh), pos, pos, -1)
        o_ref[a:b], s_ref[a:b] = oo, ss
    return to_np(o), o_ref, to_np(s), s_ref, cu


@pytest.mark.parametrize("dtype,H,dh,lengths", [
    (torch.float32, 4, 64, [70]), (torch.float32, 2, 64, [1, 33, 5]),
    (torch.bfloat16, 4, 128, [1]), (torch.bfloat16, 4, 128, [64]), (torch.bfloat16, 3, 128, [200]),
    (torch.bfloat16, 2, 128, [65, 1, 130, 17]), (torch.bfloat16, 2, 128, [513]),
    (torch.bfloat16, 4, 64, [45]),
])
def test_attention_and_score(dtype, H, dh, lengths):
    o, o_ref, s, s_ref, cu = _attention_case(dtype, H, dh, lengths, 20)
    assert rel_err(o, o_ref) < _tol(dtype)
    assert np.max(np.abs(s - s_ref)) < 1e-3
    assert np.max(np.abs(s - s_ref) / s_ref.clip(1e-12)) < (1e-4 if dtype == torch.float32 else 2e-2)
    for a, b in zip(cu[:-1], cu[1:]):
        assert abs(s[a:b].sum() - 1) < 1e-4


def test_attention_beyond_4096_keys():
    """One sequence longer than 4096 tokens (more than 64 key tiles per query tile, several waves of query
    tiles) next to a short one, against the explicit n x n oracle: long prompts are timed at 8k-32k tokens,
    so the kernel is also checked element by element past 4096 keys."""
    o, o_ref, s, s_ref, cu = _attention_case(torch.bfloat16, 2, 128, [4500, 300], 60)
    assert rel_err(o, o_ref) < BF16_STEP_TOL
    assert np.max(np.abs(s - s_ref)) < 1e-3
    assert np.max(np.abs(s - s_ref) / s_ref.clip(1e-12)) < 2e-2
    # rows near the end of the long sequence individually (a max over the whole tensor is set by early rows)
    for r in (4096, 4223, 4499):
        assert rel_err(o[r], o_ref[r]) < BF16_STEP_TOL


def test_attention_running_max_rescale_path():
    """Logits that keep growing with the key index force the streaming softmax to raise its running
    maximum late (the tensor-core kernel then rescales the accumulator it keeps in tensor memory)."""
    H, dh, n = 2, 128, 700
    d = H * dh
    q = _rand((n, d), 40, torch.bfloat16)
    k = (_rand((n, d), 41, torch.bfloat16).float() * torch.linspace(0.2, 12.0, n)[:, None]).to(torch.bfloat16)
    v = _rand((n, d), 42, torch.bfloat16)
    cu = torch.tensor([0, n], dtype=torch.int32).cuda()
    o = B.lazy_k_attention(q.cuda(), d, k.cuda(), v.cuda(), d, cu, n, n, H, dh)
    B.lazy_device_status()
    pos = np.arange(n)
    o_ref, _ = O.attend(to_np(q).reshape(n, H, dh), to_np(k).reshape(n, H, dh), to_np(v).reshape(n, H, dh),
                        pos, pos, -1)
    assert rel_err(to_np(o), o_ref) < BF16_STEP_TOL


# ------------------------------------------------------------------------------------------ select
def _select_case(score_list, keep_list):
    cu_in = np.concatenate([[0], np.cumsum([len(s) for s in score_list])]).astype(np.int32)
    cu_keep = np.concatenate([[0], np.cumsum(keep_list)]).astype(np.int32)
    scores = torch.cat(score_list)
    keep, drop = B.lazy_k_select(scores.cuda(), torch.tensor(cu_in).cuda(), torch.tensor(cu_keep).cuda())
    B.lazy_device_status()
    keep, drop = to_np(keep), to_np(drop)
    for s in range(len(score_list)):
        n = len(score_list[s])
        k_ref, d_ref = O.select_top(score_list[s].numpy(), keep_list[s], n - 1)
        got_k = keep[cu_keep[s]:cu_keep[s + 1]] - cu_in[s]
        d0 = cu_in[s] - cu_keep[s]
        got_d = drop[d0:d0 + n - keep_list[s]] - cu_in[s]
        assert np.array_equal(got_k, k_ref), (s, n, keep_list[s])
        assert np.array_equal(got_d, d_ref)


@pytest.mark.parametrize("kind", ["random", "uniform", "zeros", "duplicates", "lognormal"])
@pytest.mark.parametrize("n", [1, 2, 127, 128, 129, 1025, 3376, 4096, 65536])
def test_select_bit_exact(kind, n):
    s = synth.make_scores(n, kind, seed=n)
    for n_keep in sorted({1, max(1, (n * 3 + 9) // 10), max(1, (n * 7 + 9) // 10), n}):
        _select_case([s], [n_keep])


def test_select_per_sequence_batch():
    lens = [5, 1, 300, 2049, 64]
    scores = [synth.make_scores(n, k, seed=i) for i, (n, k) in
              enumerate(zip(lens, ["duplicates", "random", "zeros", "lognormal", "uniform"]))]
    _select_case(scores, [3, 1, 150, 615, 64])


# ------------------------------------------------------------------------------------------ gather
@pytest.mark.parametrize("dtype,d", [(torch.bfloat16, 4096), (torch.float32, 256)])
def test_gather_rows_is_an_exact_copy(dtype, d):
    src = _rand((500, d), 30, dtype)
    idx = torch.tensor(sorted(np.random.default_rng(1).choice(500, 301, replace=False)), dtype=torch.int32)
    out = B.lazy_k_gather_rows(src.cuda(), idx.cuda())
    B.lazy_device_status()
    assert torch.equal(out.cpu(), src[idx.long()])
    assert B.lazy_k_gather_rows(src.cuda(), idx[:0].cuda()).shape[0] == 0


def test_gather_rows_reports_a_bad_index_instead_of_reading_it():
    src = _rand((10, 64), 31, torch.bfloat16).cuda()
    idx = torch.tensor([0, 3, 10], dtype=torch.int32).cuda()      # 10 is out of range
    B.lazy_k_gather_rows(src, idx)
    with pytest.raises(B.LazyError) as e:
        B.lazy_device_status()
    assert e.value.status == -1
    B.lazy_device_status()                                          # cleared


# ----------------------------------------------------------------------------- bounded waits
@pytest.mark.parametrize("which,where", [(0, 15), (1, 14)])
def test_bounded_wait_runs_out_and_reports_timeout(which, where):
    """Every device-side wait of the tensor-core kernels is bounded.  A one-warp kernel waits, for at most
    one millisecond, on an mbarrier phase (which = 0) or on a split-wave arrival counter (which = 1) that
    nothing ever signals; no copy or MMA is in flight.  The wait must give up, LAZY_E_TIMEOUT with the
    waiting site's code must come back through the status word, and the device must serve the next call."""
    B.lazy_device_status()                                   # start from a clean status word
    B.lazy_k_wait_selftest(which, 1000)
    with pytest.raises(B.LazyError) as e:
        B.lazy_device_status()
    assert e.value.status == -5                              # LAZY_E_TIMEOUT
    assert B.lazy_status_detail()[0] == where
    B.lazy_device_status()                                   # cleared by the read
    x = torch.randn((64, 256)).to(torch.bfloat16).cuda()
    w = torch.randn((128, 256)).to(torch.bfloat16).cuda()
    got = B.lazy_k_gemm(x, w)                                # the device still answers, results still right
    B.lazy_device_status()
    ref = x.double().cpu().numpy() @ w.double().cpu().numpy().T
    assert rel_err(to_np(got), ref) < 1e-2


def test_select_kernel_writes_position_lists_and_handles_long_sequences():
    """The selection at sizes on both sides of its shared-memory key cache (8192 rows), clustered scores (all
    keys share their high bytes, the case the warp-combined histogram is for) included: bit-exact sets."""
    for n, kind in ((8192, "uniform"), (8193, "lognormal"), (20000, "duplicates"), (3376, "uniform")):
        s = synth.make_scores(n, kind, 77)
        if kind == "uniform":
            s = s + torch.arange(n, dtype=torch.float32) * 1e-12    # nearly equal, distinct in the low bits
        _select_case([s], [max(1, (n * 3) // 10)])


# ----------------------------------------------------------------------------- e4m3 projections
def test_quant_rows_e4m3_bit_exact():
    """Per-row e4m3 quantisation: the codes and scales the kernel decides equal the oracle's, bit for bit
    (both decide in float32: scale = max|x| / 448, code = nearest-even e4m3 of x / scale)."""
    g = torch.Generator().manual_seed(70)
    x = (torch.randn((37, 4096), generator=g) * torch.logspace(-3, 2, 37)[:, None]).to(torch.bfloat16)
    x[5] = 0
    x[6, :100] = 0
    q, sc = B.lazy_k_quant_rows_e4m3(x.cuda())
    B.lazy_device_status()
    codes, scale = O.quant_rows_e4m3(to_np(x))
    assert np.array_equal(to_np(sc), scale)
    got = q.view(torch.float8_e4m3fn).float().cpu().numpy()
    assert np.array_equal(got, codes)


def _fp8_operands(M, N, K, seed):
    a = _rand((M, K), seed, torch.bfloat16)
    w = _rand((N, K), seed + 1, torch.float32, std=0.02)
    ws = 2.0 ** np.ceil(np.log2(float(w.abs().max()) / 448.0))
    w8 = (w / ws).to(torch.float8_e4m3fn)
    a8, a_sc = B.lazy_k_quant_rows_e4m3(a.cuda())
    a_deq = a8.view(torch.float8_e4m3fn).float().cpu().numpy().astype(np.float64) * to_np(a_sc).astype(np.float64)[:, None]
    w_deq = w8.float().numpy().astype(np.float64) * ws
    return a8, a_sc, w8.view(torch.uint8).cuda(), float(ws), a_deq, w_deq


@pytest.mark.parametrize("M,N,K", [(5, 256, 128), (128, 256, 4096), (300, 520, 1040), (1013, 4096, 4096),
                                   (2364, 4096, 11008)])
def test_gemm_fp8_matches_the_product_of_the_dequantised_operands(M, N, K):
    """tcgen05 kind::f8f6f4 product of e4m3 codes with fp32 accumulation, scales applied on the way out: against
    the float64 product of the de-quantised operands (exact inputs on both sides; only the bf16 rounding of the
    output and the fp32 accumulation order differ).  Ragged rows / columns / K, several waves, a split last wave."""
    a8, a_sc, w8, ws, a_deq, w_deq = _fp8_operands(M, N, K, 80)
    ref = a_deq @ w_deq.T
    got = B.lazy_k_gemm_fp8(a8, a_sc, w8, ws)
    B.lazy_device_status()
    assert rel_err(to_np(got), ref) < BF16_STEP_TOL
    r = _rand((M, N), 83, torch.bfloat16)
    got = B.lazy_k_gemm_fp8(a8, a_sc, w8, ws, R=r.cuda())
    B.lazy_device_status()
    assert rel_err(to_np(got), ref + to_np(r)) < BF16_STEP_TOL


def test_gemm_fp8_swiglu():
    M, F, K = 700, 1408, 512
    a8, a_sc, g8, gs, a_deq, g_deq = _fp8_operands(M, F, K, 90)
    _, _, u8, us, _, u_deq = _fp8_operands(M, F, K, 94)
    a8b, a_scb, _, _, a_deqb, _ = _fp8_operands(M, F, K, 90)      # same activations (same seed)
    assert torch.equal(a8, a8b)
    gg = a_deq @ g_deq.T
    uu = a_deq @ u_deq.T
    ref = gg / (1.0 + np.exp(-gg)) * uu
    got = B.lazy_k_gemm_fp8(a8, a_sc, g8, gs, B8u=u8, w_scale_up=us)
    B.lazy_device_status()
    assert rel_err(to_np(got), ref) < BF16_STEP_TOL
