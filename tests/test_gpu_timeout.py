"""The device-timeout route: a bounded wait that runs out must reach the host as a status, once,
and leave the context usable.  The wait that runs out belongs to a one-thread self-test kernel
(a barrier nothing signals, no copy in flight); the production kernels are not touched."""
import pytest
import torch

from paper_2510_00636_b200 import inputs

pytestmark = pytest.mark.gpu

EA_ERR_DEVICE_TIMEOUT = 6


@pytest.fixture(scope="module")
def ea():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2510_00636_b200 import binding
    binding.lib()
    return binding


def test_wait_that_runs_out_is_reported_once_and_the_context_survives(ea):
    cfg = inputs.CONFIGS[1]
    q, k, v, pos = inputs.generate_layer(cfg, device="cuda")
    shape = ea.make_shape(cfg.n_units, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.n_keys, cfg.window)
    ctx = ea.Context.for_shape(shape)
    mu, sig = ea.ea_query_stats(ctx, shape, q, pos.cuda(), cfg.n_future, cfg.rope_base)
    before = ea.ea_score(ctx, shape, k, v, mu, sig, cfg.eps)
    ctx.sync_status()                                   # healthy so far

    ctx.selftest_wait_timeout(200)
    with pytest.raises(ea.EAError) as e:
        ctx.sync_status()
    assert e.value.status == EA_ERR_DEVICE_TIMEOUT
    ctx.sync_status()                                   # reported once, then cleared

    # the status word's clearing did not disturb anything: same context, same bits
    after = ea.ea_score(ctx, shape, k, v, mu, sig, cfg.eps)
    ctx.sync_status()
    assert torch.equal(before, after)

    # a second timeout is reported again; work enqueued behind it on the same stream still runs
    ctx.selftest_wait_timeout(50)
    again = ea.ea_score(ctx, shape, k, v, mu, sig, cfg.eps)
    with pytest.raises(ea.EAError) as e:
        ctx.sync_status()
    assert e.value.status == EA_ERR_DEVICE_TIMEOUT
    assert torch.equal(before, again)
    ctx.sync_status()


def test_selftest_limit_is_validated(ea):
    ctx = ea.Context(0, 0)
    for bad in (0, -5, 1001):
        with pytest.raises(ea.EAError) as e:
            ctx.selftest_wait_timeout(bad)
        assert e.value.status == 1
    ctx.sync_status()
