"""The failure path of the device-side waits, exercised without any GPU fault: a one-warp kernel waits (bounded) on a
barrier nothing arrives at, the wait runs out, the status word is set, and until the host has read it every kernel of
the context does no work."""
import pytest
import torch

from paper_2505_19578_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def binding():
    from paper_2505_19578_b200 import binding as b, build
    build.build()
    return b


@pytest.mark.parametrize("name,seq", [("llama8b_32k", 1024), ("tiny", 512)])   # paired kernel / one-row-block kernel
def test_wait_runs_out_status_poisons_until_read(binding, name, seq):
    L = synth.make_layer(synth.scaled(synth.CONFIGS[name], seq), seed=11, device="cuda")
    cfg = L["cfg"]
    q, k, v = L["q"], L["k"], L["v"]
    heads = [0, cfg.n_q_heads - 1]
    Nb = cfg.seq // cfg.block

    fresh = binding.Context()
    want = torch.zeros_like(q)
    want_imp = torch.zeros(len(heads), Nb, Nb, device="cuda")
    fresh.sp_dense_pivot_attn(q, k, v, heads, cfg.block, want, importance_out=want_imp)
    torch.cuda.synchronize()
    assert fresh.status() == (0, 0)

    ctx = binding.Context()
    ctx.selftest_wait_timeout(200_000)                     # about 0.1 ms of SM cycles, then the wait gives up
    torch.cuda.synchronize()
    # not read yet: the next calls must leave their outputs alone
    out = torch.full_like(q, float("nan"))
    imp = torch.full((len(heads), Nb, Nb), -7.0, device="cuda")
    ctx.sp_dense_pivot_attn(q, k, v, heads, cfg.block, out, importance_out=imp)
    torch.cuda.synchronize()
    assert bool(torch.isnan(out).all())
    code, where = ctx.status()
    assert code == binding.SP_ERR_TIMEOUT and where == 99
    assert "wait" in binding.error_string(code).lower() or "time" in binding.error_string(code).lower()
    # read and cleared: the context works again and gives the same bits as a fresh one
    assert ctx.status() == (0, 0)
    ctx.sp_dense_pivot_attn(q, k, v, heads, cfg.block, out, importance_out=imp)
    torch.cuda.synchronize()
    assert ctx.status() == (0, 0)
    for h in heads:
        assert torch.equal(out[h].view(torch.int16), want[h].view(torch.int16))
    assert torch.equal(imp, want_imp)


def test_selftest_rejects_bad_limits(binding):
    ctx = binding.Context()
    for bad in (0, -5, 3_000_000_000):
        with pytest.raises(binding.SpError):
            ctx.selftest_wait_timeout(bad)
