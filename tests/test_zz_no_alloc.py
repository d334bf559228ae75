"""The allocation-free Top-k entry point against the context-based one.

`deco_topk_compress_static` serves callers that cannot allocate device memory when they need
a compressed update (stream capture in progress, a host program that owns the memory pool, a
loop that cannot take cudaMalloc's synchronisation): its working memory is a fixed device
array inside the library.  This file is collected last on purpose, so that a run that stops
at the first failure has already run every other test; it also passes on its own in a fresh
process.  Two calls in a row check that nothing of the first call's scratch contents leaks
into the second."""
import gc

import numpy as np
import pytest
import torch

from paper_2507_17346_b200 import binding as B

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    from paper_2507_17346_b200 import build
    build.build()
    B.load()


def _reference_message(a, k):
    """Messages of the existing entry point for a single worker with e = 0 and gamma = 1,
    so that the compressed vector is `a` itself."""
    d = a.numel()
    ctx = B.deco_init(d, 1, k / d, 0, 1.0, select_mode=B.DECO_SELECT_EXACT_PASSES)
    try:
        assert B.deco_get_k(ctx) == k
        B.deco_ef_compress(ctx, a.view(1, d))
        buf = B.deco_get_buffers(ctx)
        out = B.view_i32(buf["msg"], (1, buf["k_cap"], 2))[0, :k].clone()
        assert B.deco_get_stats(ctx)["device_status"] == 0
        return out
    finally:
        B.deco_destroy(ctx)


def _oracle_message(a, k):
    """The same message from the CPU oracle's definition of Top-k (full sort)."""
    from oracle import dd_ef_sgd as O
    host = a.cpu().numpy()
    sel = O.topk_select(host, k)
    return sel, host[sel]


def _free_bytes():
    """Free device memory as the driver sees it (any allocator: torch's, cudaMalloc inside the
    library, anything else in the process)."""
    torch.cuda.synchronize()
    return torch.cuda.mem_get_info()[0]


def test_static_entry_point_matches_context_path_twice_in_a_row():
    torch.cuda.set_device(0)
    g = torch.Generator(device="cuda")
    g.manual_seed(20250717)
    cases = []
    d1, k1 = 1_000_003, 10_000                                  # ragged tail, 123 tiles
    cases.append((torch.randn(d1, generator=g, device="cuda"), k1))
    d2, k2 = 300_001, 4_321                                     # fewer tiles, heavy ties
    coarse = torch.randint(-8, 9, (d2,), generator=g, device="cuda").float() / 8.0
    cases.append((coarse, k2))
    want = [_reference_message(a, k) for a, k in cases]
    outs = [torch.full((k, 2), -1, dtype=torch.int32, device="cuda") for _, k in cases]
    # the first call on a device looks up the scratch array's address: take it out of the way
    warm = torch.zeros((8, 2), dtype=torch.int32, device="cuda")
    B.deco_topk_compress_static(cases[0][0], 64, 8, warm)
    # Tensors left over from earlier tests may be released by Python's collector at any moment,
    # which lowers the counter: collect them first, and accept only "no growth" afterwards.
    gc.collect()
    before_torch = torch.cuda.memory_allocated()
    before_free = _free_bytes()
    for (a, k), out in zip(cases, outs):                         # two calls back to back
        B.deco_topk_compress_static(a, a.numel(), k, out)
    after_free = _free_bytes()
    assert torch.cuda.memory_allocated() <= before_torch         # nothing through torch
    assert after_free >= before_free                             # nothing through the driver
    for (a, k), out, ref in zip(cases, outs, want):
        # integer indices and copied values: the tolerance of the parity tests is bit-exact
        assert torch.equal(out, ref)
        idx = out[:, 0].cpu().numpy().view(np.uint32).astype(np.int64)
        assert np.all(np.diff(idx) > 0) and idx[-1] < a.numel()
        sel, vals = _oracle_message(a, k)                         # and the oracle says the same
        assert np.array_equal(out[:, 0].cpu().numpy().view(np.uint32), sel)
        assert np.array_equal(out[:, 1].cpu().numpy().view(np.uint32), vals.view(np.uint32))


@pytest.mark.parametrize("d,k", [(1, 1), (5000, 5000), (8193, 1), (8192, 8192), (70_001, 35_000)])
def test_static_entry_point_edge_shapes(d, k):
    """Shorter than one tile, k = d, k = 1, a vector that ends one entry into a new tile."""
    g = torch.Generator(device="cuda")
    g.manual_seed(d * 31 + k)
    a = torch.randn(d, generator=g, device="cuda")
    a[:: 7] = 0.5                                                # some ties
    out = torch.full((k, 2), -1, dtype=torch.int32, device="cuda")
    B.deco_topk_compress_static(a, d, k, out)
    torch.cuda.synchronize()
    assert torch.equal(out, _reference_message(a, k))
    sel, vals = _oracle_message(a, k)
    assert np.array_equal(out[:, 0].cpu().numpy().view(np.uint32), sel)
    assert np.array_equal(out[:, 1].cpu().numpy().view(np.uint32), vals.view(np.uint32))


def test_static_entry_point_at_its_size_limit():
    """The longest vector the fixed scratch serves (2048 tiles), and one entry more."""
    d, k = B.DECO_STATIC_MAX_D, 16_778
    g = torch.Generator(device="cuda")
    g.manual_seed(99)
    a = torch.randn(d + 1, generator=g, device="cuda")
    out = torch.full((k, 2), -1, dtype=torch.int32, device="cuda")
    B.deco_topk_compress_static(a, d, k, out)
    torch.cuda.synchronize()
    assert torch.equal(out, _reference_message(a[:d].contiguous(), k))
    sel, vals = _oracle_message(a[:d], k)
    assert np.array_equal(out[:, 0].cpu().numpy().view(np.uint32), sel)
    assert np.array_equal(out[:, 1].cpu().numpy().view(np.uint32), vals.view(np.uint32))
    with pytest.raises(B.DecoError) as e:                        # a real buffer, one entry too long
        B.deco_topk_compress_static(a, d + 1, k, out)
    assert e.value.status == B.DECO_ERR_CAPACITY


def test_static_entry_point_rejects_bad_sizes():
    a = torch.zeros(16, device="cuda")
    out = torch.zeros((16, 2), dtype=torch.int32, device="cuda")
    for d, k in ((16, 0), (16, 17), (0, 1)):
        with pytest.raises(B.DecoError) as e:
            B.deco_topk_compress_static(a, d, k, out)
        assert e.value.status == B.DECO_ERR_INVALID_ARG
    with pytest.raises(B.DecoError) as e:                        # beyond the fixed scratch
        B.deco_topk_compress_static(a, B.DECO_STATIC_MAX_D + 1, 1, out)
    assert e.value.status == B.DECO_ERR_CAPACITY
