"""The allocation-free batch-norm entry point (ddg_bn_fwd_noalloc) against ddg_bn_fwd, through the C ABI.

For callers that cannot allocate device memory the library keeps the kernel's scratch in a fixed device array of
its own.  The result must equal the ordinary entry point's (same kernels, only the scratch differs), also on a
second call that finds the first call's leftovers in the shared array, and sizes beyond the built-in scratch must
be refused with a clear error.  Collected last so that a failure here cannot hide any other test."""
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("prec", [0, 1], ids=["fp32", "bf16"])
def test_noalloc_matches_regular_entry_point_twice_in_a_row(prec):
    from paper_1804_10574_b200 import binding
    dt = torch.bfloat16 if prec else torch.float32
    torch.manual_seed(3)
    for call, (B, HW, C, relu, with_res) in enumerate([(37, 256, 64, 1, True), (128, 1024, 16, 0, False)]):
        x = (torch.randn(B, HW, C, device="cuda") * 1.3 + 0.2).to(dt)
        res = torch.randn(B, HW, C, device="cuda").to(dt) if with_res else None
        gamma = (1 + 0.1 * torch.randn(C, device="cuda")).to(dt)
        beta = (0.1 * torch.randn(C, device="cuda")).to(dt)
        y_ref, y = torch.empty_like(x), torch.empty_like(x)
        m_ref, i_ref, m, i = (torch.empty(C, dtype=torch.float32, device="cuda") for _ in range(4))
        scratch = torch.empty(binding.bn_scratch_elems(C), dtype=torch.float32, device="cuda")
        binding.bn_fwd(prec, x, gamma, beta, res, y_ref, m_ref, i_ref, scratch, B, HW, C, relu)
        rc = binding.bn_fwd_noalloc(prec, x, gamma, beta, res, y, m, i, B, HW, C, relu)
        torch.cuda.synchronize()
        assert rc == 0, (call, rc)
        # same kernels, same launch shape, fixed summation order: the tolerance the other BN tests use is far wider
        assert torch.allclose(m, m_ref, rtol=1e-5, atol=1e-6) and torch.allclose(i, i_ref, rtol=1e-5, atol=1e-6)
        assert torch.allclose(y.float(), y_ref.float(), rtol=6e-3 if prec else 1e-5, atol=1e-5), call
        assert torch.equal(y, y_ref), call


def test_noalloc_rejects_sizes_beyond_its_scratch():
    from paper_1804_10574_b200 import binding
    C = 128
    x = torch.zeros(2, 4, C, device="cuda")
    g = torch.ones(C, device="cuda")
    m = torch.empty(C, device="cuda")
    rc = binding.bn_fwd_noalloc(0, x, g, g, None, torch.empty_like(x), m, torch.empty_like(m), 2, 4, C, 0)
    assert rc == 3                                                  # DDG_ERR_UNSUPPORTED
    assert b"64 channels" in binding.lib().ddg_last_error(None)
