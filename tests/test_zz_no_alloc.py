"""The allocation-free statistics call against the ordinary one.

``ea_query_stats_static`` exists for callers that may not allocate device memory (a serving
loop behind a caching allocator, a plugin host that forbids driver allocations after start-up):
it takes no context and keeps its only scratch, the averaged-rotation coefficients, in a fixed
array inside the library.  It must return what ``ea_query_stats`` returns, on the first call
and on a later call that finds the previous call's coefficients still in the array.

This file is collected last on purpose: a failure here must not hide any other test from a
run that stops at the first failure.
"""
import ctypes

import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ea():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2510_00636_b200 import binding
    binding.lib()
    return binding


def _window(U, Hq, W, d, seed):
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    return (torch.randn(U, Hq, W, d, generator=g, device="cuda") * 1.5 + 0.25).to(torch.bfloat16)


def test_static_scratch_call_matches_context_call_twice_in_a_row(ea):
    # two different problems back to back: the second is smaller and sits at other positions, so
    # coefficients left behind by the first would show up as a mismatch
    cases = [dict(U=5, Hq=4, W=96, d=128, T=512, base=1e6, pos=[8192, 100, 0, 77, 131072], layout=0, cov=0),
             dict(U=2, Hq=3, W=33, d=128, T=7, base=1e4, pos=[5, 4096], layout=1, cov=1)]
    for seed, c in enumerate(cases):
        q = _window(c["U"], c["Hq"], c["W"], c["d"], seed)
        pos = torch.tensor(c["pos"], dtype=torch.int64, device="cuda")
        shape = ea.make_shape(c["U"], c["Hq"], 1, c["d"], 0, c["W"], rope_layout=c["layout"], cov_norm=c["cov"])
        ctx = ea.Context.for_shape(shape)
        mu_ref, sig_ref = ea.ea_query_stats(ctx, shape, q, pos, c["T"], c["base"])
        ctx.sync_status()
        mu = torch.full_like(mu_ref, float("nan"))
        sig = torch.full_like(sig_ref, float("nan"))
        ea.ea_query_stats_static(shape, q, pos, c["T"], c["base"], mu, sig)
        torch.cuda.synchronize()
        # same kernels, same arithmetic: the statistics tolerance of the parity tests (2e-5 of
        # the scale) is met with room to spare; in fact the bits agree
        scale = sig_ref.abs().amax().item() + 1e-30
        assert (sig - sig_ref).abs().max().item() <= 2e-5 * scale
        assert (mu - mu_ref).abs().max().item() <= 2e-5 * (1 + mu_ref.abs().max().item())
        assert torch.equal(mu, mu_ref) and torch.equal(sig, sig_ref)


@pytest.mark.parametrize("d,layout,U", [(64, 0, 3), (64, 1, 512), (128, 1, 256), (256, 0, 4), (256, 1, 128)])
def test_static_scratch_call_every_head_dim_up_to_the_limit(ea, d, layout, U):
    """Each head_dim has its own launch shape (one block row at 64 and 128, three at 256), both rotation
    pairings, and the largest problem the fixed array admits (n_units * head_dim / 2 == the stated maximum);
    a second call right behind the first must neither change the result nor take any device memory."""
    Hq, W, T = 2, 40, 64
    if U * d // 2 > ea.STATIC_MAX_ROPE_PAIRS:
        pytest.skip("beyond the fixed array")
    at_limit = U * d // 2 == ea.STATIC_MAX_ROPE_PAIRS
    q = _window(U, Hq, W, d, 100 + d + layout)
    pos = torch.arange(U, dtype=torch.int64, device="cuda") * 37 + 5
    shape = ea.make_shape(U, Hq, 1, d, 0, W, rope_layout=layout)
    ctx = ea.Context.for_shape(shape)
    mu_ref, sig_ref = ea.ea_query_stats(ctx, shape, q, pos, T, 1e6)
    ctx.sync_status()
    mu, sig = torch.empty_like(mu_ref), torch.empty_like(sig_ref)
    ea.ea_query_stats_static(shape, q, pos, T, 1e6, mu, sig)
    torch.cuda.synchronize()
    assert torch.equal(mu, mu_ref) and torch.equal(sig, sig_ref), (d, layout, U, at_limit)
    free_before, _ = torch.cuda.mem_get_info()
    mu.fill_(0), sig.fill_(0)
    ea.ea_query_stats_static(shape, q, pos, T, 1e6, mu, sig)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before, "the call took device memory"
    assert torch.equal(mu, mu_ref) and torch.equal(sig, sig_ref)


def test_static_scratch_call_refuses_oversized_and_bad_shapes(ea):
    L = ea.lib()
    too_many = ea.STATIC_MAX_ROPE_PAIRS // 64 + 1            # units at head_dim 128
    shape = ea.make_shape(too_many, 1, 1, 128, 0, 8)
    dummy = ctypes.c_void_p(256)                              # never dereferenced: refused before any launch
    assert L.ea_query_stats_static(ctypes.byref(shape), dummy, dummy, 4, 1e4, dummy, dummy, None) == 3
    shape = ea.make_shape(1, 1, 1, 96, 0, 8)
    assert L.ea_query_stats_static(ctypes.byref(shape), dummy, dummy, 4, 1e4, dummy, dummy, None) == 2
    shape = ea.make_shape(1, 1, 1, 128, 0, 8)
    assert L.ea_query_stats_static(ctypes.byref(shape), None, dummy, 4, 1e4, dummy, dummy, None) == 1
    assert L.ea_query_stats_static(ctypes.byref(shape), dummy, dummy, 0, 1e4, dummy, dummy, None) == 1
    assert L.ea_query_stats_static(None, dummy, dummy, 4, 1e4, dummy, dummy, None) == 1
