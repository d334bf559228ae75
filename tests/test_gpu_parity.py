"""GPU parity: libdeco (through the C-ABI) against the CPU oracle, element by element, on the
same seeded inputs.  Sizes span several tiles of 8192 entries plus ragged tails."""
import numpy as np
import pytest
import torch

from paper_2507_17346_b200 import binding as B
from paper_2507_17346_b200 import workloads as W
from tests.parity import run_layered_parity, run_parity

pytestmark = pytest.mark.gpu

MODES = [B.DECO_SELECT_EXACT_PASSES, B.DECO_SELECT_AUTO]


@pytest.fixture(scope="module", autouse=True)
def _lib():
    from paper_2507_17346_b200 import build
    build.build()
    B.load()


def _values(kind, n, d, step, dtype):
    g = torch.Generator(device="cuda")
    g.manual_seed(1000 * step + d + 7 * n)
    if kind == "normal":
        x = torch.randn((n, d), generator=g, device="cuda")
    elif kind == "all_equal":
        x = torch.full((n, d), -1.5, device="cuda")
    elif kind == "all_zero":
        x = torch.zeros((n, d), device="cuda")
    elif kind == "two_valued":
        x = torch.where(torch.rand((n, d), generator=g, device="cuda") < 0.3, 2.0, -0.25)
    elif kind == "signed_zero":
        r = torch.rand((n, d), generator=g, device="cuda")
        x = torch.where(r < 0.4, 0.0, torch.where(r < 0.8, -0.0, 1.0))
    elif kind == "coarse":                                  # few distinct magnitudes
        x = torch.randint(-8, 9, (n, d), generator=g, device="cuda").float() / 8.0
    else:
        raise KeyError(kind)
    return x.to(dtype).contiguous()


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("kind", ["normal", "all_equal", "all_zero", "two_valued",
                                  "signed_zero", "coarse"])
def test_tiny_and_ragged_shapes(kind, mode):
    for d, n, delta in [(1, 1, 1.0), (3, 2, 0.5), (31, 3, 0.1), (4097, 2, 0.01),
                        (8192, 1, 0.3), (8193, 3, 0.02), (20001, 2, 1.0), (24576, 2, 1e-9)]:
        for dtype, name in ((torch.float32, "f32"), (torch.bfloat16, "bf16")):
            run_parity(d, n, delta, 1, 0.1, lambda t: _values(kind, n, d, t, dtype), steps=3,
                       grad_dtype=name, select_mode=mode)


@pytest.mark.parametrize("mode", MODES)
def test_flat_1m_all_steps(mode):
    wl = W.make_workload("flat_1m")
    run_parity(wl.d, wl.n, wl.delta, wl.tau, wl.lr, lambda t: W.gradients(wl, t, "cuda"),
               steps=wl.steps, grad_dtype=wl.grad_dtype, select_mode=mode)


@pytest.mark.parametrize("mode", MODES)
@pytest.mark.parametrize("name,scale,steps", [("resnet18", 0.25, 8), ("gpt2_small", 0.08, 12),
                                              ("decoder_1b", 0.03, 7)])
def test_scaled_workloads(name, scale, steps, mode):
    """The shaped workloads at reduced width, each for more than tau iterations (so that stale
    updates are applied and the cache wraps), every buffer compared with the oracle."""
    wl = W.make_workload(name, scale)
    assert steps > wl.tau + 2
    run_parity(wl.d, wl.n, wl.delta, wl.tau, wl.lr, lambda t: W.gradients(wl, t, "cuda"),
               steps=steps, grad_dtype=wl.grad_dtype, select_mode=mode)


def test_resnet18_full_size():
    """Configuration 2 as stated: full size, all 50 iterations, every buffer every iteration."""
    wl = W.make_workload("resnet18")
    assert wl.d == 11_689_512 and len(wl.tensors) == 62 and wl.steps == 50 and wl.tau == 4
    run_parity(wl.d, wl.n, wl.delta, wl.tau, wl.lr, lambda t: W.gradients(wl, t, "cuda"),
               steps=wl.steps, grad_dtype=wl.grad_dtype)


@pytest.mark.parametrize("mode", MODES)
def test_policy_changes_at_run_time(mode):
    d, n = 300_000, 4
    plan = {3: (0.05, 1), 6: (0.001, 4), 9: (0.1, 0), 12: (0.0001, 2)}
    wl = W.make_workload("sweep_100m", 0.003)
    assert wl.d == d
    run_parity(d, n, 0.01, 2, 0.1, lambda t: W.gradients(wl, t, "cuda"), steps=16,
               policy_plan=plan, tau_max=4, delta_max=0.1, select_mode=mode)


@pytest.mark.parametrize("mode", MODES)
def test_degradation_to_dsgd_and_stepsize_at_server(mode):
    d, n = 50_000, 4
    wl = W.make_workload("sweep_100m", 0.0005)
    assert wl.d == d
    run_parity(d, n, 1.0, 0, 0.1, lambda t: W.gradients(wl, t, "cuda"), steps=4,
               select_mode=mode)                                    # delta = 1, tau = 0: D-SGD
    run_parity(d, n, 1.0, 3, 0.1, lambda t: W.gradients(wl, t, "cuda"), steps=6,
               select_mode=mode)                                    # delayed aggregation only
    run_parity(d, n, 0.02, 2, 0.25, lambda t: W.gradients(wl, t, "cuda"), steps=6,
               lr_at_server=True, select_mode=mode)


def test_streaming_route_is_taken_and_falls_back_on_degenerate_inputs():
    """With the default selection mode, ordinary inputs go through the sampled single-pass
    route; inputs whose tie class is far larger than the staging area (all equal, all zero,
    two-valued) must be handed to the multi-pass route inside the same call."""
    d, n = 300_000, 3
    run_parity(d, n, 0.01, 1, 0.1, lambda t: _values("normal", n, d, t, torch.float32),
               steps=4, expect_exact=False)
    for kind in ("all_equal", "all_zero"):
        run_parity(d, n, 0.01, 1, 0.1, lambda t: _values(kind, n, d, t, torch.float32),
                   steps=3, expect_exact=True)
    # two-valued: the tie class overflows the staging area at step 0 only
    st = run_parity(d, n, 0.01, 1, 0.1, lambda t: _values("two_valued", n, d, t, torch.float32),
                    steps=3)
    assert st["exact_pass_workers"] >= n
    # mixed: worker 0 degenerate, the others ordinary -> per-worker decision
    def mixed(t):
        g = _values("normal", n, d, t, torch.float32)
        g[0] = 0.5
        return g
    ctx_stats = run_parity(d, n, 0.01, 1, 0.1, mixed, steps=3)
    assert 0 < ctx_stats["exact_pass_workers"] < 3 * n


def test_adaptive_policy_run():
    """DeCo-SGD (Algorithm 2): every E iterations the host re-selects (tau, delta) with DeCo
    (Algorithm 3) from a synthetic bandwidth/latency trace; the library's decision must equal
    the oracle's, and the iterations stay in parity across the changes."""
    from oracle import deco_policy as P
    wl = W.make_workload("sweep_100m", 0.004)
    d, n, steps, E = wl.d, wl.n, 60, 10
    V_g, T_comp, tau_max, delta_max = 32.0 * 1e8, 0.05, 16, 0.2
    lat, bw = W.network_trace(wl.seed, steps)
    plan = {}
    for t in range(E, steps, E):                      # decided after iteration t-1
        a_bar, b = float(np.mean(bw[t - E:t])), float(lat[t - 1])
        tau, delta = B.deco_policy_select(V_g, a_bar, b, T_comp, tau_max, False)
        otau, odelta = P.deco_select(V_g, a_bar, b, T_comp)
        if otau > tau_max:
            otau, odelta = tau_max, P.delta_star(tau_max, V_g, a_bar, b, T_comp)
        assert (tau, delta) == (otau, pytest.approx(odelta, rel=1e-12))
        delta = min(delta_max, max(delta, 1.0 / d))
        plan[t] = (delta, tau)
    assert len({v for v in plan.values()}) >= 3          # the trace does move the decision
    run_parity(d, n, 0.01, 2, 0.1, lambda t: W.gradients(wl, t, "cuda"), steps=steps,
               policy_plan=plan, tau_max=tau_max, delta_max=delta_max, check_every=3)


@pytest.mark.parametrize("mode", MODES)
def test_many_workers_and_odd_length(mode):
    """More workers than the aggregation keeps in registers at once, rows that are not
    16-byte aligned, a vector that ends in the middle of a tile."""
    d, n = 50_001, 20
    for dtype, name in ((torch.float32, "f32"), (torch.bfloat16, "bf16")):
        run_parity(d, n, 0.02, 2, 0.1, lambda t: _values("normal", n, d, t, dtype), steps=5,
                   grad_dtype=name, select_mode=mode)
    run_parity(d, n, 0.5, 1, 0.1, lambda t: _values("coarse", n, d, t, torch.float32), steps=3,
               select_mode=mode)


@pytest.mark.parametrize("n", [3, 8, 20])
def test_sparse_messages_take_every_aggregation_path(n):
    """A few entries per tile: the aggregation merges a tile in one warp, in one go (at most 32
    entries), window by window (at most 32 per quarter of the tile), or hands it to the whole
    CTA (a hot tile).  Workers share most of their large entries, so sums of 2..n terms, in
    worker order, are the rule."""
    d, delta = 200_003, 0.002

    def grads(t):
        g = torch.Generator(device="cuda")
        g.manual_seed(77 + t)
        base = torch.randn((1, d), generator=g, device="cuda")
        x = base * (1.0 + 0.2 * torch.randn((n, d), generator=g, device="cuda"))
        x[:, 3 * 8192:4 * 8192] *= 50.0                      # hot tile: hundreds of entries
        x[:, 10 * 8192:10 * 8192 + 2048] *= 4.0              # one crowded quarter
        x[:, 17 * 8192:19 * 8192] *= 2.0                     # 30..100 entries per tile
        return x.contiguous()

    st = run_parity(d, n, delta, 1, 0.1, grads, steps=4)
    assert st["device_status"] == 0


@pytest.mark.parametrize("seed", [11, 12, 13, 14])
def test_seeded_random_configurations(seed):
    """Shapes, worker counts, densities, staleness, dtypes and value structure drawn from a seeded
    generator: every draw must match the oracle bit for bit like the hand-picked cases."""
    rng = np.random.default_rng(seed)
    for _ in range(8):
        d = int(rng.choice([rng.integers(1, 3000), rng.integers(3000, 70_000),
                            rng.integers(70_000, 400_000)]))
        n = int(rng.integers(1, 25))
        delta = float(min(1.0, 10.0 ** rng.uniform(-4, 0.1)))
        tau = int(rng.integers(0, 4))
        dtype, name = ((torch.float32, "f32"), (torch.bfloat16, "bf16"))[int(rng.integers(0, 2))]
        kind = str(rng.choice(["normal", "coarse", "hot", "shared"]))
        hot_lo = int(rng.integers(0, d))
        hot_hi = min(d, hot_lo + int(rng.integers(1, 20_000)))
        case_seed = int(rng.integers(0, 1 << 30))
        delta2 = float(min(1.0, 10.0 ** rng.uniform(-4, 0.1)))

        def grads(t):
            g = torch.Generator(device="cuda")
            g.manual_seed(case_seed + t)
            if kind == "coarse":
                x = torch.randint(-8, 9, (n, d), generator=g, device="cuda").float() / 8.0
            else:
                x = torch.randn((n, d), generator=g, device="cuda")
            if kind == "shared":                                  # workers agree on the large entries
                x = x[:1] * (1.0 + 0.1 * x)
            if kind in ("hot", "shared"):
                x[:, hot_lo:hot_hi] *= 30.0
            return x.to(dtype).contiguous()

        dmax = max(delta, delta2)
        run_parity(d, n, delta, tau, 0.1, grads, steps=4, grad_dtype=name,
                   policy_plan={2: (delta2, int(rng.integers(0, 4)))}, tau_max=3, delta_max=dmax)


def test_per_layer_topk_variant():
    """Top-k per tensor instead of over the flat vector: tiny tensors (k_l = 1), tensors that
    start at odd offsets (gradient rows of a layer are then not 16-byte aligned), a loud layer,
    a policy change; fp32 and bf16 gradients."""
    wl = W.make_workload("resnet18", 0.125)                  # 62 tensors, ResNet-18 structure
    offsets = [0]
    for t in wl.tensors:
        offsets.append(offsets[-1] + int(t.numel))
    assert offsets[-1] == wl.d
    run_layered_parity(offsets, 3, 0.01, 2, 0.1, lambda t: W.gradients(wl, t, "cuda")[:3].contiguous(),
                       steps=4, policy_plan={2: (0.03, 1)}, tau_max=2, delta_max=0.03)
    odd = [0, 1, 4, 1001, 1002, 30_003, 100_000, 100_007]
    for dtype, name in ((torch.float32, "f32"), (torch.bfloat16, "bf16")):
        def grads(t):
            g = torch.Generator(device="cuda")
            g.manual_seed(900 + t)
            x = torch.randn((4, odd[-1]), generator=g, device="cuda")
            x[:, 4:1001] *= 40.0
            return x.to(dtype).contiguous()
        run_layered_parity(odd, 4, 0.02, 1, 0.1, grads, steps=4, grad_dtype=name)
    # the multi-pass selection keeps the route that steps every layer's context on its own
    run_layered_parity(offsets, 3, 0.01, 1, 0.1, lambda t: W.gradients(wl, t, "cuda")[:3].contiguous(),
                       steps=3, select_mode=B.DECO_SELECT_EXACT_PASSES)


@pytest.mark.parametrize("kind", ["normal", "coarse", "all_equal", "signed_zero"])
def test_per_layer_topk_short_layers_batch(kind):
    """Layers of at most 8192 entries are stepped as one batch (a CTA per layer and worker, a
    CTA per layer on the server side): lengths 1, 31, 8191, 8192 next to one of 8193 that takes
    the ordinary route, heavy ties (few distinct magnitudes, all equal, signed zeros), delta
    up to 1, and a staleness that goes 3 -> 0 -> 2 so that one update drains several cached
    aggregates and another applies its own iteration's."""
    lengths = [1, 31, 8191, 8192, 8193, 2, 4097, 640]
    offsets = [0]
    for ln in lengths:
        offsets.append(offsets[-1] + ln)
    n = 5
    for dtype, name in ((torch.float32, "f32"), (torch.bfloat16, "bf16")):
        run_layered_parity(offsets, n, 0.05, 3, 0.1,
                           lambda t: _values(kind, n, offsets[-1], t, dtype), steps=9,
                           grad_dtype=name, policy_plan={4: (1.0, 0), 6: (0.3, 2)},
                           tau_max=3, delta_max=1.0)


def test_per_layer_thousands_of_layers():
    """4400 layers just above one tile (8200 entries each) with one worker: the kernels on the
    staged pairs share a CTA budget out over the layers, and with more layers than the budget
    every layer still gets its one CTA (two for emit) - the map from CTA to layer has to hold
    them all.  Two layers of 300 K entries take the long end of the shares."""
    lengths = [8200] * 2200 + [300_000] + [8200] * 2200 + [300_001]
    offsets = [0]
    for ln in lengths:
        offsets.append(offsets[-1] + ln)
    n = 1
    run_layered_parity(offsets, n, 0.01, 1, 0.1,
                       lambda t: _values("normal", n, offsets[-1], t, torch.float32), steps=3,
                       grad_dtype="f32", tau_max=1, delta_max=0.01)


def test_per_layer_bound_carried_over_between_iterations():
    """After a few iterations under one policy the per-layer path takes its speculative bound
    from the previous iterations' exact thresholds instead of a sample.  Stationary gradients:
    no row may need the multi-pass route once the bound is carried (iterations 4 to 13).  Then a
    collapse and a jump of the gradient scale, which a carried bound cannot foresee: the count of
    staged candidates must catch both and the rows take the multi-pass route, still bit for bit."""
    lengths = [9000, 50_000, 200_003, 8193, 31, 120_000]
    offsets = [0]
    for ln in lengths:
        offsets.append(offsets[-1] + ln)
    d, n = offsets[-1], 3

    def steady(t, dtype=torch.float32):
        return _values("normal", n, d, t, dtype)

    for dtype, name in ((torch.float32, "f32"), (torch.bfloat16, "bf16")):
        assert run_layered_parity(offsets, n, 0.01, 2, 0.1, lambda t: steady(t, dtype), steps=14,
                                  grad_dtype=name) == 0

    def jumpy(t):
        scale = 1.0 if t < 7 else (1e-3 if t < 10 else 300.0)
        return (steady(t) * scale).contiguous()

    assert run_layered_parity(offsets, n, 0.01, 1, 0.1, jumpy, steps=13) > 0
    run_layered_parity(offsets, n, 0.02, 1, 0.1, lambda t: _values("coarse", n, d, t, torch.float32), steps=9)


def test_per_layer_random_k_equals_one_context_per_layer():
    """Random-k per layer (layer l draws from the stream seeded seed + l) keeps the route that
    steps every layer's context on its own; it must give what separate ordinary contexts give
    on the layers' slices (those are checked against the oracle elsewhere)."""
    lengths = [5000, 8192, 30_001, 70_000]
    offsets = [0]
    for ln in lengths:
        offsets.append(offsets[-1] + ln)
    d, n, seed = offsets[-1], 3, 4242
    lay = B.deco_layered_init(d, n, offsets, 0.02, 1, 0.1, compressor=B.DECO_COMPRESSOR_RANDK, seed=seed)
    flat = [B.deco_init(ln, n, 0.02, 1, 0.1, compressor=B.DECO_COMPRESSOR_RANDK, seed=seed + l)
            for l, ln in enumerate(lengths)]
    try:
        info = B.deco_layered_info(lay)
        for t in range(4):
            g = _values("normal", n, d, t, torch.float32)
            B.deco_layered_step(lay, g)
            for l, ln in enumerate(lengths):
                B.deco_step(flat[l], g[:, offsets[l]:offsets[l + 1]].contiguous())
            B.deco_layered_join(lay)
            torch.cuda.synchronize()
            for l, ln in enumerate(lengths):
                sub, off, _ = B.deco_layered_layer(lay, l)
                ba, bb = B.deco_get_buffers(sub), B.deco_get_buffers(flat[l])
                k = B.deco_get_k(sub)
                assert k == B.deco_get_k(flat[l])
                assert torch.equal(B.view_i32(ba["msg"], (n, ba["k_cap"], 2))[:, :k],
                                   B.view_i32(bb["msg"], (n, bb["k_cap"], 2))[:, :k]), (t, l)
                assert torch.equal(B.view_i32(ba["e"], (n, ba["e_stride"])),
                                   B.view_i32(bb["e"], (n, bb["e_stride"]))), (t, l)
                assert torch.equal(B.view_i32(info["params"], (d,))[off:off + ln],
                                   B.view_i32(bb["params"], (ln,))), (t, l)
    finally:
        B.deco_layered_destroy(lay)
        for c in flat:
            B.deco_destroy(c)


@pytest.mark.parametrize("seed", [31, 32])
def test_per_layer_seeded_random_partitions(seed):
    """Layer lengths (1 … 200 K, on both sides of the 8192-entry limit of the batched route),
    worker counts, densities, staleness, dtypes and value structure drawn from a seeded
    generator, with a policy change in the middle: bit for bit against the oracle."""
    rng = np.random.default_rng(seed)
    for _ in range(6):
        nl = int(rng.integers(1, 25))
        lens = [int(rng.choice([rng.integers(1, 200), rng.integers(200, 8193),
                                rng.integers(8193, 200_000)])) for _ in range(nl)]
        offsets = [0]
        for ln in lens:
            offsets.append(offsets[-1] + ln)
        d, n = offsets[-1], int(rng.integers(1, 12))
        delta = float(min(1.0, 10.0 ** rng.uniform(-3.5, 0.1)))
        delta2 = float(min(1.0, 10.0 ** rng.uniform(-3.5, 0.1)))
        tau, tau2 = int(rng.integers(0, 4)), int(rng.integers(0, 4))
        dtype, name = ((torch.float32, "f32"), (torch.bfloat16, "bf16"))[int(rng.integers(0, 2))]
        kind = str(rng.choice(["normal", "coarse", "all_equal", "two_valued"]))
        run_layered_parity(offsets, n, delta, tau, 0.1, lambda t: _values(kind, n, d, t, dtype),
                           steps=5, grad_dtype=name, policy_plan={2: (delta2, tau2)}, tau_max=3,
                           delta_max=max(delta, delta2))


@pytest.mark.parametrize("compressor,delta,delta2", [("topk", 0.004, 0.02), ("randk", 0.004, 0.02),
                                                     ("topk", 0.06, 0.01)])
def test_worker_sharded_contexts_equal_the_single_job(compressor, delta, delta2):
    """Five workers split 2 + 3 over two contexts on one GPU.  Each compresses its own workers;
    the rows of the exchange buffer are then copied across (what the all-gather does
    between GPUs), and both replicas aggregate and update.  Local messages and residuals, the
    aggregate and both parameter replicas must equal the oracle's single five-worker job."""
    from oracle import dd_ef_sgd as O
    from tests.parity import bits, read_aggregate, read_e, read_messages, read_params
    d, n, tau, lr = 70_004, 5, 1, 0.1
    split = [(0, 2), (2, 3)]
    comp = B.DECO_COMPRESSOR_RANDK if compressor == "randk" else B.DECO_COMPRESSOR_TOPK
    ctxs = [B.deco_init(d, cnt, delta, tau, lr, n_total=n, worker_base=base, compressor=comp,
                        seed=99, tau_max=2, delta_max=max(delta, delta2)) for base, cnt in split]
    orc = O.DDEFSGD(d, n, delta, tau, lr, compressor=compressor, seed=99)
    try:
        with pytest.raises(B.DecoError):
            B.deco_step(ctxs[0], torch.zeros((2, d), device="cuda"))
        for t in range(6):
            if t == 3:                                   # the rows change length (and the aggregate its layout)
                for c in ctxs:
                    B.deco_set_policy(c, delta2, 2)
                orc.set_policy(delta2, 2)
            g = _values("normal", n, d, t, torch.float32)
            ref = orc.step(W.to_numpy_bits(g))
            views = []
            for c, (base, cnt) in zip(ctxs, split):
                B.deco_ef_compress(c, g[base:base + cnt])
                rows, x = B.exchange_view(c)
                # one contiguous range of k (not k_cap) pairs and a directory per worker
                assert x["row_words"] == (2 * ref["k"] + (d + 8191) // 8192 + 1 + 1) // 2 * 2
                assert rows.is_contiguous() and rows.shape == (n, x["row_words"])
                views.append(rows)
            for me, (base, cnt) in enumerate(split):               # the exchange, by copies
                for other in range(len(split)):
                    if other != me:
                        views[other][base:base + cnt].copy_(views[me][base:base + cnt])
            touched = np.unique(np.concatenate([s for s, _ in ref["msgs"]]))
            for c, (base, cnt) in zip(ctxs, split):
                idx, val = read_messages(c, cnt, ref["k"])
                for i in range(cnt):
                    assert np.array_equal(idx[i], ref["msgs"][base + i][0]), (t, base + i)
                    assert np.array_equal(bits(val[i]), bits(ref["msgs"][base + i][1]))
                assert np.array_equal(bits(read_e(c, cnt, d)), bits(orc.e[base:base + cnt]))
                B.deco_aggregate_stale(c)
                aidx, aval = read_aggregate(c, t, 0, d, touched)
                assert np.array_equal(aidx, touched), t
                assert np.array_equal(bits(aval), bits(ref["S"][touched])), t
                B.deco_apply_update(c)
                assert np.array_equal(bits(read_params(c, d)), bits(orc.x)), t
        for c in ctxs:
            st = B.deco_get_stats(c)
            assert st["device_status"] == 0 and st["step"] == 6
    finally:
        for c in ctxs:
            B.deco_destroy(c)


def test_sharded_step_through_nccl_with_one_rank():
    """The binding's sharded step (compress, all-gather of the exchange buffers through
    torch.distributed / NCCL, aggregate, update) with a world of one rank gives the bits of
    the plain three calls."""
    import torch.distributed as dist
    from tests.parity import bits, read_params
    d, n = 120_000, 4
    dist.init_process_group("nccl", init_method="tcp://127.0.0.1:29541", rank=0, world_size=1,
                            device_id=torch.device("cuda", 0))
    a = B.deco_init(d, n, 0.01, 2, 0.1, n_total=n, delta_max=0.05)
    b = B.deco_init(d, n, 0.01, 2, 0.1, delta_max=0.05)
    try:
        with pytest.raises(B.DecoError):                  # no exchange buffer without n_total
            B.deco_get_exchange(b)
        for t in range(5):
            if t == 3:                                     # the rows get longer
                B.deco_set_policy(a, 0.05, 1)
                B.deco_set_policy(b, 0.05, 1)
            g = _values("normal", n, d, t, torch.float32)
            B.deco_step_sharded(a, g)
            B.deco_ef_compress(b, g)
            B.deco_aggregate_stale(b)
            B.deco_apply_update(b)
            torch.cuda.synchronize()
            assert np.array_equal(bits(read_params(a, d)), bits(read_params(b, d))), t
    finally:
        B.deco_destroy(a)
        B.deco_destroy(b)
        dist.destroy_process_group()


@pytest.mark.parametrize("mode", MODES)
def test_random_k_sparsifier(mode):
    """Random-k in place of Top-k: the same Philox priorities on both sides give the same index
    sets; everything downstream (residual, aggregate, update) is shared with Top-k."""
    seed = 0x5EED0123456789AB
    for d, n, delta, dtype, name in [(4097, 2, 0.01, torch.float32, "f32"),
                                     (20001, 3, 0.3, torch.bfloat16, "bf16"),
                                     (300_000, 4, 0.01, torch.float32, "f32"),
                                     (300_000, 2, 0.0005, torch.float32, "f32"),
                                     (50_000, 2, 1.0, torch.float32, "f32")]:
        run_parity(d, n, delta, 2, 0.1, lambda t: _values("normal", n, d, t, dtype), steps=5,
                   grad_dtype=name, select_mode=mode, compressor="randk", seed=seed)
    wl = W.make_workload("resnet18", 0.25)
    st = run_parity(wl.d, wl.n, wl.delta, wl.tau, wl.lr, lambda t: W.gradients(wl, t, "cuda"),
                    steps=6, select_mode=mode, compressor="randk", seed=7)
    if mode == B.DECO_SELECT_AUTO:
        assert st["exact_pass_workers"] == 0          # the sampled bound holds for uniform priorities


def test_call_order_and_capacity_errors():
    d, n = 10_000, 2
    ctx = B.deco_init(d, n, 0.01, 1, 0.1, tau_max=2, delta_max=0.05)
    try:
        g = torch.randn((n, d), device="cuda")
        with pytest.raises(B.DecoError) as e:
            B.deco_aggregate_stale(ctx)
        assert e.value.status == B.DECO_ERR_STATE
        with pytest.raises(B.DecoError) as e:
            B.deco_apply_update(ctx)
        assert e.value.status == B.DECO_ERR_STATE
        B.deco_ef_compress(ctx, g)
        with pytest.raises(B.DecoError) as e:
            B.deco_ef_compress(ctx, g)
        assert e.value.status == B.DECO_ERR_STATE
        with pytest.raises(B.DecoError) as e:
            B.deco_set_policy(ctx, 0.02, 1)
        assert e.value.status == B.DECO_ERR_STATE
        B.deco_aggregate_stale(ctx)
        B.deco_apply_update(ctx)
        for delta, tau in ((0.06, 1), (0.01, 3)):
            with pytest.raises(B.DecoError) as e:
                B.deco_set_policy(ctx, delta, tau)
            assert e.value.status == B.DECO_ERR_CAPACITY
        assert B.deco_get_k(ctx) == 100                              # unchanged
        B.deco_set_policy(ctx, 0.05, 2)
        assert B.deco_get_k(ctx) == 500
        with pytest.raises(B.DecoError) as e:
            B.deco_ef_compress(ctx, g[:, 1:])                        # misaligned base pointer
        assert e.value.status == B.DECO_ERR_INVALID_ARG
        assert B.deco_get_stats(ctx)["step"] == 1
    finally:
        B.deco_destroy(ctx)


def test_two_runs_give_the_same_bits():
    wl = W.make_workload("resnet18", 0.25)
    outs = []
    for _ in range(2):
        ctx = B.deco_init(wl.d, wl.n, wl.delta, wl.tau, wl.lr)
        try:
            for t in range(6):
                B.deco_step(ctx, W.gradients(wl, t, "cuda"))
            buf = B.deco_get_buffers(ctx)
            outs.append((B.view_i32(buf["e"], (wl.n, buf["e_stride"])).clone(),
                         B.view_i32(buf["params"], (wl.d,)).clone(),
                         B.view_i32(buf["msg"], (wl.n, buf["k_cap"], 2)).clone()))
            assert B.deco_get_stats(ctx)["device_status"] == 0
        finally:
            B.deco_destroy(ctx)
    for a, b in zip(*outs):
        assert torch.equal(a, b)


def test_fused_step_equals_the_three_calls():
    """deco_step runs the stale update on an internal stream next to the worker side and leaves
    its aggregation running there; the result must be the bits of compress -> aggregate ->
    apply issued one after the other, also across changes of tau (including tau = 0, where
    nothing may overlap) and when the two forms are mixed on one context."""
    wl = W.make_workload("resnet18", 0.25)
    kw = dict(tau_max=3, delta_max=0.02)
    a = B.deco_init(wl.d, wl.n, wl.delta, 2, wl.lr, **kw)
    b = B.deco_init(wl.d, wl.n, wl.delta, 2, wl.lr, **kw)
    side = torch.cuda.Stream()
    try:
        plan = {3: (0.02, 0), 5: (0.005, 3), 8: (0.01, 1)}
        for t in range(14):
            if t in plan:
                B.deco_set_policy(a, *plan[t])
                B.deco_set_policy(b, *plan[t])
            g = W.gradients(wl, t, "cuda")
            torch.cuda.synchronize()
            with torch.cuda.stream(side):                       # a non-default caller stream
                if t % 4 == 3:                                  # the three calls right behind a
                    B.deco_ef_compress(a, g)                    # fused step: they have to order
                    B.deco_aggregate_stale(a)                   # themselves after its aggregation
                    B.deco_apply_update(a)
                else:
                    B.deco_step(a, g)
            B.deco_ef_compress(b, g)
            B.deco_aggregate_stale(b)
            B.deco_apply_update(b)
            torch.cuda.synchronize()
            ba, bb = B.deco_get_buffers(a), B.deco_get_buffers(b)
            assert torch.equal(B.view_i32(ba["params"], (wl.d,)), B.view_i32(bb["params"], (wl.d,))), t
            assert torch.equal(B.view_i32(ba["e"], (wl.n, ba["e_stride"])),
                               B.view_i32(bb["e"], (wl.n, bb["e_stride"]))), t
        sa, sb = B.deco_get_stats(a), B.deco_get_stats(b)
        assert sa["step"] == sb["step"] == 14 and sa["cached_aggregates"] == sb["cached_aggregates"]
        assert sa["device_status"] == 0 and sb["device_status"] == 0
    finally:
        B.deco_destroy(a)
        B.deco_destroy(b)


@pytest.mark.parametrize("tau", [1, 2])
def test_fused_step_with_a_long_aggregation(tau):
    """Dense messages (delta = 0.05 of 4 M entries): the aggregation left behind by one fused
    step is still running when the next step's worker side starts, so the orderings between
    the internal streams (emit after the previous aggregation, update after the aggregate it
    consumes) carry real waits.  Bits must equal the strictly sequential three calls."""
    d, n = 4_000_000, 4
    a = B.deco_init(d, n, 0.05, tau, 0.1)
    b = B.deco_init(d, n, 0.05, tau, 0.1)
    try:
        pool = [_values("normal", n, d, t, torch.float32) for t in range(3)]
        for t in range(12):
            B.deco_step(a, pool[t % 3])                          # back to back, no host sync
        for t in range(12):
            B.deco_ef_compress(b, pool[t % 3])
            B.deco_aggregate_stale(b)
            B.deco_apply_update(b)
        B.deco_join(a)
        torch.cuda.synchronize()
        ba, bb = B.deco_get_buffers(a), B.deco_get_buffers(b)
        assert torch.equal(B.view_i32(ba["params"], (d,)), B.view_i32(bb["params"], (d,)))
        assert torch.equal(B.view_i32(ba["e"], (n, ba["e_stride"])), B.view_i32(bb["e"], (n, bb["e_stride"])))
        for s_ in range(12 - tau, 12):                           # the aggregates still cached
            va = B.view_i32(B.deco_get_aggregate_vector(a, s_), (d,))   # dense messages: vector layout
            vb = B.view_i32(B.deco_get_aggregate_vector(b, s_), (d,))
            assert torch.equal(va, vb)
        assert B.deco_get_stats(a)["device_status"] == 0
    finally:
        B.deco_destroy(a)
        B.deco_destroy(b)


@pytest.mark.parametrize("d,n,delta", [(6_000_000, 8, 0.05), (16_000_000, 16, 0.0065)])
def test_fused_step_with_the_server_side_behind_the_pass(d, n, delta):
    """With many staged pairs in all (n (2 k + 65536) above 4 Mi) the selection is a row of
    ordinary launches, and deco_step then books the aggregation of an iteration and launches it
    only behind the streaming pass of the next call, together with the update.  The first
    shape keeps the aggregate as a vector, the second as pairs.  Bits must equal the strictly
    sequential three calls: back to back without a host sync, across policy changes (which
    have to launch a booked aggregation first, tau = 1 and tau = 0 included), with the three
    calls mixed in, with a read of the cache in between, and through export / import while an
    aggregation is booked."""
    k = int(B.deco_k_from_delta(delta, d))
    assert n * (2 * k + 65536) > (4 << 20)
    kw = dict(tau_max=3, delta_max=delta)
    a = B.deco_init(d, n, delta, 2, 0.1, **kw)
    b = B.deco_init(d, n, delta, 2, 0.1, **kw)
    c = B.deco_init(d, n, delta, 2, 0.1, **kw)
    try:
        pool = [_values("normal", n, d, t, torch.float32) for t in range(3)]
        plan = {4: (delta, 1), 7: (delta * 0.9, 3), 10: (delta, 0), 12: (delta * 0.8, 2)}
        steps = 16
        for t in range(steps):
            if t in plan:
                B.deco_set_policy(a, *plan[t])
            if t % 5 == 3:
                B.deco_ef_compress(a, pool[t % 3])
                B.deco_aggregate_stale(a)
                B.deco_apply_update(a)
            else:
                B.deco_step(a, pool[t % 3])
            if t == 8:
                B.deco_get_aggregate_vector(a, 8) if 8 * n * B.deco_get_k(a) >= d else B.deco_get_aggregate(a, 8)
            if t == 11:                                          # resume in another context
                B.deco_import_state(c, B.deco_export_state(a))
        for t in range(12, steps):
            if t in plan:
                B.deco_set_policy(c, *plan[t])
            B.deco_step(c, pool[t % 3])
        for t in range(steps):
            if t in plan:
                B.deco_set_policy(b, *plan[t])
            B.deco_ef_compress(b, pool[t % 3])
            B.deco_aggregate_stale(b)
            B.deco_apply_update(b)
        B.deco_join(a)
        B.deco_join(c)
        torch.cuda.synchronize()
        bb = B.deco_get_buffers(b)
        kk = B.deco_get_k(b)
        for other in (a, c):
            bo = B.deco_get_buffers(other)
            assert torch.equal(B.view_i32(bo["params"], (d,)), B.view_i32(bb["params"], (d,)))
            assert torch.equal(B.view_i32(bo["e"], (n, bo["e_stride"])), B.view_i32(bb["e"], (n, bb["e_stride"])))
            assert torch.equal(B.view_i32(bo["msg"], (n, bo["k_cap"], 2))[:, :kk],
                               B.view_i32(bb["msg"], (n, bb["k_cap"], 2))[:, :kk])
            so, sb = B.deco_get_stats(other), B.deco_get_stats(b)
            assert so["step"] == sb["step"] == steps and so["cached_aggregates"] == sb["cached_aggregates"]
            assert so["device_status"] == 0
            for s_ in range(steps - 2, steps):                   # the aggregates still cached (tau = 2)
                if 8 * n * kk >= d:
                    assert torch.equal(B.view_i32(B.deco_get_aggregate_vector(other, s_), (d,)),
                                       B.view_i32(B.deco_get_aggregate_vector(b, s_), (d,)))
                else:
                    (pa, na), (pb, nb) = B.deco_get_aggregate(other, s_), B.deco_get_aggregate(b, s_)
                    assert na == nb
                    assert torch.equal(B.view_i32(pa, (na, 2)), B.view_i32(pb, (nb, 2)))
    finally:
        B.deco_destroy(a)
        B.deco_destroy(b)
        B.deco_destroy(c)


@pytest.mark.parametrize("seed", range(700, 712))
def test_fused_step_random_call_mixes(seed):
    """deco_step against the strictly sequential three calls on seeded random shapes (up to
    4 * 10^7 entries, 1 to 16 workers, both gradient types), policies that change at random
    iterations (tau down to 0), and random mixes of calls between the steps: the three calls,
    a join, a read of the statistics, and an export / import into a fresh context.  Parameters,
    residuals, messages and the number of cached aggregates must agree bit for bit."""
    rng = np.random.default_rng(seed)
    n = int(rng.integers(1, 17))
    d = int(rng.choice([rng.integers(200_000, 2_000_000), rng.integers(2_000_000, 12_000_000),
                        rng.integers(12_000_000, 40_000_000)]))
    d = min(d, 150_000_000 // n)
    delta_max = float(min(1.0, 10.0 ** rng.uniform(-3, -0.7)))
    tau_max = int(rng.integers(1, 5))
    dtype = (torch.float32, torch.bfloat16)[int(rng.integers(0, 2))]

    def policy():
        return float(delta_max * 10.0 ** rng.uniform(-1.0, 0)), int(rng.integers(0, tau_max + 1))

    first = policy()
    steps = int(rng.integers(8, 16))
    plan = {int(s_): policy() for s_ in rng.choice(np.arange(1, steps), size=int(rng.integers(0, 4)), replace=False)}
    acts = [str(rng.choice(["step", "step", "step", "three", "step_join", "step_stats"])) for _ in range(steps)]
    swap_at = int(rng.integers(2, steps - 1)) if rng.integers(0, 2) else -1
    pool = [_values("normal", n, d, seed + t, dtype) for t in range(3)]
    kw = dict(grad_dtype=B.DECO_F32 if dtype == torch.float32 else B.DECO_BF16, tau_max=tau_max,
              delta_max=delta_max)
    a = B.deco_init(d, n, first[0], first[1], 0.1, **kw)
    b = B.deco_init(d, n, first[0], first[1], 0.1, **kw)
    try:
        for t in range(steps):
            if t in plan:
                B.deco_set_policy(a, *plan[t])
                B.deco_set_policy(b, *plan[t])
            g = pool[t % 3]
            if acts[t] == "three":
                B.deco_ef_compress(a, g)
                B.deco_aggregate_stale(a)
                B.deco_apply_update(a)
            else:
                B.deco_step(a, g)
                if acts[t] == "step_join":
                    B.deco_join(a)
                if acts[t] == "step_stats":
                    B.deco_get_stats(a)
            B.deco_ef_compress(b, g)
            B.deco_aggregate_stale(b)
            B.deco_apply_update(b)
            if t == swap_at:                                     # carry on in a fresh context
                blob = B.deco_export_state(a)
                B.deco_destroy(a)
                a = B.deco_init(d, n, first[0], first[1], 0.1, **kw)
                B.deco_import_state(a, blob)
        B.deco_join(a)
        torch.cuda.synchronize()
        ba, bb = B.deco_get_buffers(a), B.deco_get_buffers(b)
        k = B.deco_get_k(b)
        assert torch.equal(B.view_i32(ba["params"], (d,)), B.view_i32(bb["params"], (d,)))
        assert torch.equal(B.view_i32(ba["e"], (n, ba["e_stride"])), B.view_i32(bb["e"], (n, bb["e_stride"])))
        assert torch.equal(B.view_i32(ba["msg"], (n, ba["k_cap"], 2))[:, :k],
                           B.view_i32(bb["msg"], (n, bb["k_cap"], 2))[:, :k])
        sa, sb = B.deco_get_stats(a), B.deco_get_stats(b)
        assert sa["step"] == sb["step"] == steps and sa["cached_aggregates"] == sb["cached_aggregates"]
        assert sa["device_status"] == 0 and sb["device_status"] == 0
    finally:
        B.deco_destroy(a)
        B.deco_destroy(b)
        del pool
        torch.cuda.empty_cache()


def test_checkpoint_and_resume_give_the_same_bits():
    wl = W.make_workload("gpt2_small", 0.08)
    kw = dict(grad_dtype=B.DECO_BF16, tau_max=4, delta_max=0.01)
    a = B.deco_init(wl.d, wl.n, wl.delta, 3, wl.lr, **kw)
    b = B.deco_init(wl.d, wl.n, wl.delta, 3, wl.lr, **kw)
    try:
        for t in range(5):
            if t == 3:
                B.deco_set_policy(a, 0.004, 2)
            B.deco_step(a, W.gradients(wl, t, "cuda"))
        blob = B.deco_export_state(a)
        assert len(blob) == B.deco_state_bytes(a)
        B.deco_import_state(b, blob)
        assert B.deco_get_stats(b)["step"] == 5 and B.deco_get_k(b) == B.deco_get_k(a)
        assert B.deco_get_stats(b)["cached_aggregates"] == B.deco_get_stats(a)["cached_aggregates"]
        for t in range(5, 10):
            g = W.gradients(wl, t, "cuda")
            B.deco_step(a, g)
            B.deco_step(b, g)
        torch.cuda.synchronize()
        ba, bb = B.deco_get_buffers(a), B.deco_get_buffers(b)
        k = B.deco_get_k(a)
        for name, shape in (("e", (wl.n, ba["e_stride"])), ("params", (wl.d,))):
            assert torch.equal(B.view_i32(ba[name], shape), B.view_i32(bb[name], shape)), name
        assert torch.equal(B.view_i32(ba["msg"], (wl.n, ba["k_cap"], 2))[:, :k],
                           B.view_i32(bb["msg"], (wl.n, bb["k_cap"], 2))[:, :k])
        # a blob from another shape is refused
        c = B.deco_init(wl.d + 8, wl.n, wl.delta, 3, wl.lr, **kw)
        try:
            with pytest.raises(B.DecoError) as e:
                B.deco_import_state(c, blob)
            assert e.value.status == B.DECO_ERR_INVALID_ARG
        finally:
            B.deco_destroy(c)
    finally:
        B.deco_destroy(a)
        B.deco_destroy(b)


@pytest.mark.parametrize("mode", MODES)
def test_dense_messages_keep_the_aggregate_as_a_vector(mode):
    """When the n messages hold at least d / 8 entries in all the cached aggregate is the plain
    vector S[d] (same worker-order sums; +0 where nothing was sent) and the update sweeps it.
    The density crosses that limit in both directions at run time, with a cache of several
    slots, odd lengths and both gradient types; every buffer against the oracle."""
    d, n = 150_003, 4
    plan = {2: (0.02, 3), 4: (0.3, 1), 7: (0.07, 2), 9: (0.01, 0)}
    for dtype, name in ((torch.float32, "f32"), (torch.bfloat16, "bf16")):
        run_parity(d, n, 0.1, 2, 0.1, lambda t: _values("normal", n, d, t, dtype), steps=12,
                   grad_dtype=name, policy_plan=plan, tau_max=3, delta_max=0.3, select_mode=mode)
    run_parity(8193, 9, 0.05, 1, 0.1, lambda t: _values("coarse", 9, 8193, t, torch.float32), steps=4,
               select_mode=mode)


def test_checkpoint_with_vector_aggregates():
    """Cached aggregates in both layouts travel through export / import."""
    d, n = 120_001, 4
    kw = dict(tau_max=3, delta_max=0.2)
    a = B.deco_init(d, n, 0.1, 3, 0.1, **kw)
    b = B.deco_init(d, n, 0.1, 3, 0.1, **kw)
    try:
        for t in range(6):
            if t == 4:
                B.deco_set_policy(a, 0.01, 3)            # the last two aggregates are pairs
            B.deco_step(a, _values("normal", n, d, t, torch.float32))
        B.deco_get_aggregate_vector(a, 3)
        B.deco_get_aggregate(a, 5)
        with pytest.raises(B.DecoError):
            B.deco_get_aggregate(a, 3)
        blob = B.deco_export_state(a)
        assert len(blob) == B.deco_state_bytes(a)
        B.deco_import_state(b, blob)
        for t in range(6, 11):
            g = _values("normal", n, d, t, torch.float32)
            B.deco_step(a, g)
            B.deco_step(b, g)
        torch.cuda.synchronize()
        ba, bb = B.deco_get_buffers(a), B.deco_get_buffers(b)
        for name, shape in (("e", (n, ba["e_stride"])), ("params", (d,))):
            assert torch.equal(B.view_i32(ba[name], shape), B.view_i32(bb[name], shape)), name
        assert B.deco_get_stats(a)["device_status"] == 0 and B.deco_get_stats(b)["device_status"] == 0
    finally:
        B.deco_destroy(a)
        B.deco_destroy(b)


def test_host_buffer_step_matches_device_step():
    wl = W.make_workload("resnet18", 0.25)
    k = B.deco_k_from_delta(wl.delta, wl.d)
    a = B.deco_init(wl.d, wl.n, wl.delta, wl.tau, wl.lr)
    b = B.deco_init(wl.d, wl.n, wl.delta, wl.tau, wl.lr)
    try:
        msg_host = torch.empty((wl.n, k, 2), dtype=torch.int32).pin_memory()
        x_host = torch.empty(wl.d, dtype=torch.float32).pin_memory()
        for t in range(6):
            g = W.gradients(wl, t, "cuda")
            g_host = g.cpu().pin_memory()
            B.deco_step(a, g)
            B.deco_step_host(b, g_host, msg_host, x_host)
            torch.cuda.synchronize()
            buf = B.deco_get_buffers(a)
            want_msg = B.view_i32(buf["msg"], (wl.n, buf["k_cap"], 2))[:, :k].cpu()
            want_x = B.view_f32(buf["params"], (wl.d,)).cpu()
            assert torch.equal(msg_host, want_msg)
            assert torch.equal(x_host.view(torch.int32), want_x.view(torch.int32))
    finally:
        B.deco_destroy(a)
        B.deco_destroy(b)


def test_host_buffer_steps_back_to_back():
    """deco_step_host copies the gradients on a stream of the library's own into one of two device
    buffers: calls made back to back, without a host sync in between, must each see their own
    gradients (a buffer is not refilled before the step that read it is through) and give the
    bits of the device-buffer steps, message by message."""
    wl = W.make_workload("resnet18", 0.25)
    k = B.deco_k_from_delta(wl.delta, wl.d)
    steps = 7
    a = B.deco_init(wl.d, wl.n, wl.delta, wl.tau, wl.lr)
    b = B.deco_init(wl.d, wl.n, wl.delta, wl.tau, wl.lr)
    try:
        grads = [W.gradients(wl, t, "cuda") for t in range(steps)]
        hosts = [g.cpu().pin_memory() for g in grads]
        msgs = [torch.empty((wl.n, k, 2), dtype=torch.int32).pin_memory() for _ in range(steps)]
        xs = [torch.empty(wl.d, dtype=torch.float32).pin_memory() for _ in range(steps)]
        torch.cuda.synchronize()
        for t in range(steps):
            B.deco_step_host(b, hosts[t], msgs[t], xs[t] if t % 2 == 0 else None)
        B.deco_join(b)
        torch.cuda.synchronize()
        buf = B.deco_get_buffers(a)
        for t in range(steps):
            B.deco_step(a, grads[t])
            torch.cuda.synchronize()
            assert torch.equal(msgs[t], B.view_i32(buf["msg"], (wl.n, buf["k_cap"], 2))[:, :k].cpu()), t
            if t % 2 == 0:
                assert torch.equal(xs[t].view(torch.int32),
                                   B.view_i32(buf["params"], (wl.d,)).cpu()), t
        bb = B.deco_get_buffers(b)
        assert torch.equal(B.view_i32(bb["e"], (wl.n, bb["e_stride"])), B.view_i32(buf["e"], (wl.n, buf["e_stride"])))
        assert B.deco_get_stats(b)["device_status"] == 0
    finally:
        B.deco_destroy(a)
        B.deco_destroy(b)

