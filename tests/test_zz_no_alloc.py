"""The allocation-free entry point, sp_dense_pivot_attn_fixed_scratch.

Some hosts may not allocate device memory when they need attention: an engine
plugin's enqueue hook, a server whose pool already owns the whole device, a
latency-critical loop that cannot take the synchronisation an allocation
implies.  For them the library keeps the per-tile softmax statistics in a fixed
64 MiB array of its own image instead of a context workspace.  This test calls
that entry point through the C ABI twice in a row (the second call on other
inputs and another shape, so stale array contents from the first would show)
and checks output, importance and log-sum-exp against the context-based entry
point, and that a problem too large for the array is refused.

Collected last on purpose: a failure here must not hide the other GPU tests in
a run that stops at the first failure.
"""
import numpy as np
import pytest
import torch

from tests import _parity as par

pytestmark = pytest.mark.gpu


def _inputs(seed, Hq, Hkv, N, d):
    g = torch.Generator(device="cpu").manual_seed(seed)
    q = (torch.randn(Hq, N, d, generator=g) * 2 / d ** 0.25).to(torch.bfloat16).cuda()
    k = (torch.randn(Hkv, N, d, generator=g) * 2 / d ** 0.25).to(torch.bfloat16).cuda()
    v = torch.randn(Hkv, N, d, generator=g).to(torch.bfloat16).cuda()
    return q, k, v


def test_fixed_scratch_matches_context_entry_point_twice():
    from paper_2505_19578_b200 import binding, build
    build.build()
    ctx = binding.Context()
    for call, (seed, Hq, Hkv, N, d, B, heads) in enumerate([(21, 4, 2, 1024, 128, 128, [3, 0, 2]),
                                                             (22, 2, 1, 768, 64, 64, [1, 0])]):
        q, k, v = _inputs(seed, Hq, Hkv, N, d)
        Nb = N // B
        ref_out = torch.zeros_like(q)
        ref_imp = torch.zeros(len(heads), Nb, Nb, device="cuda")
        ref_lse = torch.zeros(len(heads), N, device="cuda")
        ctx.sp_dense_pivot_attn(q, k, v, heads, B, ref_out, importance_out=ref_imp, lse_out=ref_lse)
        out = torch.zeros_like(q)
        imp = torch.full((len(heads), Nb, Nb), float("nan"), device="cuda")
        lse = torch.full((len(heads), N), float("nan"), device="cuda")
        binding.sp_dense_pivot_attn_fixed_scratch(q, k, v, heads, B, out, importance_out=imp, lse_out=lse)
        torch.cuda.synchronize()
        assert ctx.status() == (0, 0)
        max_abs, rel = par.out_errors(par.f64(out), par.f64(ref_out))
        assert max_abs <= par.OUT_MAX_ABS and rel <= par.OUT_REL_L2, (call, max_abs, rel)
        np.testing.assert_allclose(imp.cpu().numpy(), ref_imp.cpu().numpy(), rtol=0, atol=par.IMP_ATOL)
        np.testing.assert_allclose(lse.cpu().numpy(), ref_lse.cpu().numpy(), rtol=0, atol=2e-3)
        np.testing.assert_allclose(imp.cpu().numpy().sum(axis=2), 1.0, atol=1e-5)


def test_fixed_scratch_rejects_oversized_problem():
    from paper_2505_19578_b200 import binding, build
    build.build()
    N, B, d = 32768, 128, 128
    Nb = N // B
    heads = [0, 1, 2, 3]                      # 4 * Nb(Nb+1)/2 * 128 * 4 bytes = 67.4 MB > 64 MiB
    assert len(heads) * Nb * (Nb + 1) // 2 * B * 4 > binding.FIXED_SCRATCH_BYTES
    q = torch.zeros(4, N, d, dtype=torch.bfloat16, device="cuda")
    k = torch.zeros(1, N, d, dtype=torch.bfloat16, device="cuda")
    out = torch.empty_like(q)
    imp = torch.empty(4, Nb, Nb, device="cuda")
    with pytest.raises(binding.SpError) as e:
        binding.sp_dense_pivot_attn_fixed_scratch(q, k, k, heads, B, out, importance_out=imp)
    assert e.value.code == binding.SP_ERR_SCRATCH_LIMIT
    assert "fixed scratch" in str(e.value)
