"""In-place compaction and CUDA-graph capture of a compression event (the decoding set-up)."""
import numpy as np
import pytest
import torch

from paper_2510_00636_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ea():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2510_00636_b200 import binding
    binding.lib()          # raises if libea.so is missing: there is no fallback to hide behind
    return binding


@pytest.mark.parametrize("n,n_kept,d", [(1, 1, 64), (7, 3, 64), (129, 129, 128), (1000, 1, 128), (4608, 4096, 128),
                                        (5000, 0, 64), (3001, 1500, 256), (70001, 35000, 64)])
def test_inplace_compaction_exact(ea, oracle, n, n_kept, d):
    torch.manual_seed(n)
    U, Hkv = 2, 3
    sc = torch.rand(U, Hkv, n, device="cuda")
    sc[0, 0] = (sc[0, 0] * 4).floor() / 4               # many ties at the cut
    sc[0, 1] = torch.arange(n, 0, -1, device="cuda")    # the first n_kept rows stay where they are
    sc[1, 0] = torch.arange(n, device="cuda")           # the last n_kept rows move to the front
    k = torch.randn(U, Hkv, n, d, device="cuda").to(torch.bfloat16)
    v = torch.randn(U, Hkv, n, d, device="cuda").to(torch.bfloat16)
    k0, v0 = inputs.bits(k), inputs.bits(v)
    shape = ea.make_shape(U, Hkv, Hkv, d, n, 1)
    ctx = ea.Context.for_shape(shape)
    idx = ea.ea_select_compact_inplace(ctx, shape, sc, n_kept, k, v)
    ctx.sync_status()
    want = oracle.select(sc.cpu().numpy().astype(np.float64), n_kept)
    assert np.array_equal(idx.cpu().numpy(), want)
    k1, v1 = inputs.bits(k), inputs.bits(v)
    assert np.array_equal(k1[:, :, :n_kept], oracle.gather(k0, want))
    assert np.array_equal(v1[:, :, :n_kept], oracle.gather(v0, want))
    assert np.array_equal(k1[:, :, n_kept:], k0[:, :, n_kept:])      # the tail is left alone
    assert np.array_equal(v1[:, :, n_kept:], v0[:, :, n_kept:])


def test_inplace_rejects_overlapping_buffers(ea):
    shape = ea.make_shape(1, 1, 1, 64, 16, 1)
    ctx = ea.Context.for_shape(shape)
    kv = torch.zeros(1, 1, 16, 64, device="cuda", dtype=torch.bfloat16)
    with pytest.raises(ea.EAError) as e:
        ea.ea_select_compact_inplace(ctx, shape, torch.rand(1, 1, 16, device="cuda"), 4, kv, kv)
    assert e.value.status == 1


def test_compression_event_replays_as_a_cuda_graph(ea, oracle):
    """ea_query_stats + ea_score + ea_select_compact_inplace captured once and replayed on new data of
    the same shape: every output is bitwise the one of the eager calls, and matches the oracle's
    selection on the GPU's own scores."""
    cfg = inputs.CONFIGS[0].tempered(2.0)
    shape = ea.make_shape(cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.n_keys, cfg.window)
    ctx = ea.Context.for_shape(shape)
    dev = torch.device("cuda")
    data = [inputs.generate_layer(cfg, layer=layer, device=dev) for layer in range(3)]
    q, k, v = (torch.empty_like(t) for t in data[0][:3])
    pos = torch.empty_like(data[0][3], device=dev)
    mu = torch.empty((cfg.batch, cfg.n_q_heads, cfg.head_dim), device=dev)
    sigma = torch.empty((cfg.batch, cfg.n_q_heads, cfg.head_dim, cfg.head_dim), device=dev)
    scores = torch.empty((cfg.batch, cfg.n_kv_heads, cfg.n_keys), device=dev)
    idx = torch.empty((cfg.batch, cfg.n_kv_heads, cfg.n_kept), dtype=torch.int32, device=dev)

    def event():
        ea.ea_query_stats(ctx, shape, q, pos, cfg.n_future, cfg.rope_base, mu, sigma)
        ea.ea_score(ctx, shape, k, v, mu, sigma, cfg.eps, scores)
        ea.ea_select_compact_inplace(ctx, shape, scores, cfg.n_kept, k, v, idx)

    def load(layer):
        for dst, src in zip((q, k, v), data[layer][:3]):
            dst.copy_(src)
        pos.copy_(data[layer][3] + 100 * layer)

    eager = []
    for layer in range(3):
        load(layer)
        event()
        ctx.sync_status()
        eager.append([t.clone() for t in (scores, idx, k, v)])

    load(0)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        event()                                           # warm-up outside the capture
    torch.cuda.current_stream().wait_stream(side)
    graph = torch.cuda.CUDAGraph()
    load(0)
    # A Context that the garbage collector happens to destroy while the capture is open would call
    # cudaFree, which invalidates a capture: collect what earlier tests left behind first.
    import gc
    gc.collect()
    with torch.cuda.graph(graph):
        event()
    for layer in (1, 2, 0):
        load(layer)
        graph.replay()
        torch.cuda.synchronize()
        for got, want in zip((scores, idx, k, v), eager[layer]):
            assert torch.equal(got, want)
        own = oracle.select(scores.cpu().numpy().astype(np.float64), cfg.n_kept)
        assert np.array_equal(idx.cpu().numpy(), own)
    ctx.sync_status()
