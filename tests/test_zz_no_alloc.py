"""The importance score for callers that may not allocate device memory.

Some users of the library run where device allocation is off limits: inside another application's
plugin interface that owns the memory pool, in a serving callback where a cudaMalloc would stall
the whole device, or late in a process that has already given its memory away.  For them
`lazy_k_score_static` keeps its scratch in a fixed array inside the library.  This test calls it
through the C ABI, twice in a row on different inputs (the array is shared and keeps whatever the
previous call left behind), and checks each result against the ordinary entry point, whose
scratch the caller provides, and against the CPU oracle's Eq. 1.  It also checks that oversized
requests are refused.

The file sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import numpy as np
import pytest
import torch

import lazyllm_oracle as O
from paper_2407_14057_b200 import binding as B
from paper_2407_14057_b200 import build

pytestmark = pytest.mark.gpu


def _case(seed, lengths, H, dh, dtype):
    g = torch.Generator().manual_seed(seed)
    n = sum(lengths)
    d = H * dh
    q = torch.randn((n, d), generator=g).to(dtype).cuda()
    k = torch.randn((n, d), generator=g).to(dtype).cuda()
    cu = torch.tensor(np.concatenate([[0], np.cumsum(lengths)]), dtype=torch.int32).cuda()
    return q, k, cu, n, d


def test_static_scratch_score_matches_caller_scratch_score_twice_in_a_row():
    build.build()
    B.lib()
    # second call is smaller than the first: stale logits of the first call stay in the array
    for seed, lengths, H, dh, dtype in [(1, [700, 1, 300], 4, 128, torch.bfloat16),
                                        (2, [130, 65], 4, 128, torch.bfloat16),
                                        (3, [90], 4, 64, torch.float32)]:
        q, k, cu, n, d = _case(seed, lengths, H, dh, dtype)
        want = B.lazy_k_score(q, d, k, d, cu, n, H, dh)
        out = torch.full((n,), -1.0, dtype=torch.float32, device="cuda")   # allocated by the caller
        got = B.lazy_k_score_static(q, d, k, d, cu, n, H, dh, out)
        B.lazy_device_status()
        assert torch.max(torch.abs(got - want)).item() < 1e-3            # the tolerance of the score tests
        assert torch.equal(got, want)                                      # same kernels: same bits
        assert abs(got[: lengths[0]].sum().item() - 1.0) < 1e-4
        # and against the definition itself (Eq. 1 written out on the CPU), sequence by sequence
        qn = q.float().cpu().numpy().reshape(n, H, dh)
        kn = k.float().cpu().numpy().reshape(n, H, dh)
        a = 0
        for ln in lengths:
            pos = np.arange(ln)
            _, s_ref = O.attend(qn[a:a + ln], kn[a:a + ln], np.zeros((ln, H, dh)), pos, pos, -1)
            assert np.max(np.abs(got[a:a + ln].cpu().numpy() - s_ref)) < 1e-3
            a += ln


def test_static_scratch_score_refuses_sizes_beyond_its_array():
    build.build()
    q, k, cu, n, d = _case(4, [64], 4, 128, torch.bfloat16)
    out = torch.empty(n, dtype=torch.float32, device="cuda")
    with pytest.raises(B.LazyError) as e:      # 32 heads x 8193 tokens > 262144 logits
        B._check("lazy_k_score_static", B.lib().lazy_k_score_static(
            B._stream(), B.LAZY_BF16, q.data_ptr(), d, k.data_ptr(), d, cu.data_ptr(), 1, 8193, 32, 128,
            out.data_ptr()))
    assert e.value.status == -3
    B.lazy_device_status()
