"""The allocation-free entry point, sp_dense_pivot_attn_fixed_scratch.

Some hosts may not allocate device memory when they need attention: an engine
plugin's enqueue hook, a server whose pool already owns the whole device, a
latency-critical loop that cannot take the synchronisation an allocation
implies.  For them the library keeps the per-tile softmax statistics in a fixed
64 MiB array of its own image instead of a context workspace.  This test calls
that entry point through the C ABI twice in a row (the second call on other
inputs and another shape, so stale array contents from the first would show)
and checks output, importance and log-sum-exp against the context-based entry
point and against the float64 oracle, that the device's free memory does not
move across a call, and that a problem too large for the array is refused.

Collected last on purpose: a failure here must not hide the other GPU tests in
a run that stops at the first failure.
"""
import numpy as np
import pytest
import torch

from oracle import shareprefill_oracle as orc
from tests import _parity as par

pytestmark = pytest.mark.gpu


def _inputs(seed, Hq, Hkv, N, d):
    g = torch.Generator(device="cpu").manual_seed(seed)
    q = (torch.randn(Hq, N, d, generator=g) * 2 / d ** 0.25).to(torch.bfloat16).cuda()
    k = (torch.randn(Hkv, N, d, generator=g) * 2 / d ** 0.25).to(torch.bfloat16).cuda()
    v = torch.randn(Hkv, N, d, generator=g).to(torch.bfloat16).cuda()
    return q, k, v


def test_fixed_scratch_matches_context_entry_point_and_oracle_twice():
    from paper_2505_19578_b200 import binding, build
    build.build()
    ctx = binding.Context()
    dev = torch.cuda.current_device()
    # first call: head_dim 128 / block 128 (the paired persistent kernel, 7 row-blocks: an odd tail pair);
    # second call: head_dim 64 / block 64 (the one-row-block kernel)
    for call, (seed, Hq, Hkv, N, d, B, heads) in enumerate([(21, 4, 2, 896, 128, 128, [3, 0, 2]),
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
        torch.cuda.synchronize()
        if call == 0:
            # the first call on a device resolves (and, with lazy loading, loads) the array: make it before measuring
            binding.sp_dense_pivot_attn_fixed_scratch(q, k, v, heads, B, out, importance_out=imp, lse_out=lse)
            torch.cuda.synchronize()
            out.zero_()
            imp.fill_(float("nan"))
            lse.fill_(float("nan"))
            torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        binding.sp_dense_pivot_attn_fixed_scratch(q, k, v, heads, B, out, importance_out=imp, lse_out=lse)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before, "the call changed the device's free memory"
        assert binding.fixed_scratch_status(dev) == (0, 0)
        assert ctx.status() == (0, 0)
        # against the context entry point
        max_abs, rel = par.out_errors(par.f64(out), par.f64(ref_out))
        assert max_abs <= par.OUT_MAX_ABS and rel <= par.OUT_REL_L2, (call, max_abs, rel)
        np.testing.assert_allclose(imp.cpu().numpy(), ref_imp.cpu().numpy(), rtol=0, atol=par.IMP_ATOL)
        np.testing.assert_allclose(lse.cpu().numpy(), ref_lse.cpu().numpy(), rtol=0, atol=2e-3)
        np.testing.assert_allclose(imp.cpu().numpy().sum(axis=2), 1.0, atol=1e-5)
        # against the float64 oracle
        Q, K, V = par.f64(q), par.f64(k), par.f64(v)
        got = par.f64(out)
        for t, h in enumerate(heads):
            imp_ref, o_ref = orc.importance_map(Q, K, V, h, B)
            par.assert_out_close(got[h], o_ref, f"call {call} head {h} vs oracle")
            np.testing.assert_allclose(imp[t].cpu().numpy(), imp_ref, rtol=0, atol=par.IMP_ATOL)


def test_fixed_scratch_rejects_oversized_problem():
    from paper_2505_19578_b200 import binding, build
    build.build()
    # head_dim 128 / block 128: min(SMs, heads * Nb / 2) regions of 2 * Nb * 128 * 4 bytes; 4 heads at 65536 tokens
    # give 1024 work items, so one region per SM: above 64 MiB from 129 SMs on
    N, B, d = 65536, 128, 128
    Nb = N // B
    heads = [0, 1, 2, 3]
    n_sm = torch.cuda.get_device_properties(0).multi_processor_count
    need = min(n_sm, len(heads) * ((Nb + 1) // 2)) * 2 * Nb * B * 4
    if need <= binding.FIXED_SCRATCH_BYTES:
        pytest.skip(f"a device with {n_sm} SMs fits this problem into the fixed array")
    q = torch.zeros(4, N, d, dtype=torch.bfloat16, device="cuda")
    k = torch.zeros(1, N, d, dtype=torch.bfloat16, device="cuda")
    out = torch.empty_like(q)
    imp = torch.empty(4, Nb, Nb, device="cuda")
    with pytest.raises(binding.SpError) as e:
        binding.sp_dense_pivot_attn_fixed_scratch(q, k, k, heads, B, out, importance_out=imp)
    assert e.value.code == binding.SP_ERR_SCRATCH_LIMIT
    assert "fixed scratch" in str(e.value)
    # the one-row-block kernel's rule (other shapes): heads * Nb (Nb + 1) / 2 * block * 4 bytes
    N2, B2, d2 = 32768, 64, 64
    Nb2 = N2 // B2
    assert 2 * Nb2 * (Nb2 + 1) // 2 * B2 * 4 > binding.FIXED_SCRATCH_BYTES
    q2 = torch.zeros(2, N2, d2, dtype=torch.bfloat16, device="cuda")
    out2 = torch.empty_like(q2)
    imp2 = torch.empty(2, Nb2, Nb2, device="cuda")
    with pytest.raises(binding.SpError) as e2:
        binding.sp_dense_pivot_attn_fixed_scratch(q2, q2, q2, [0, 1], B2, out2, importance_out=imp2)
    assert e2.value.code == binding.SP_ERR_SCRATCH_LIMIT
