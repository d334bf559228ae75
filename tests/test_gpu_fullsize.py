"""Full-size parity in the launch configuration the benchmark times: the three workloads with
d >= 100 M.  The oracle cannot sort 10^9 entries in seconds, so the unique Top-k set is pinned
by properties that hold at any size (count, strict index order, threshold domination, tie cut
by index — together they admit exactly one set), and every arithmetic result is compared with
the oracle's own functions on sampled positions, bit for bit."""
import numpy as np
import pytest
import torch

from oracle import dd_ef_sgd as O
from paper_2507_17346_b200 import binding as B
from paper_2507_17346_b200 import workloads as W

pytestmark = pytest.mark.gpu

ABS = 0x7FFFFFFF
SAMPLES = 200_000


@pytest.fixture(scope="module", autouse=True)
def _lib():
    from paper_2507_17346_b200 import build
    build.build()
    B.load()


def _keys(t):
    return t.view(torch.int32) & ABS


def _host_bits(g_row, idx):
    """Gradient entries at idx as the oracle wants them (float32 or bfloat16 bit patterns)."""
    v = g_row[idx].cpu()
    if v.dtype == torch.bfloat16:
        return v.view(torch.int16).numpy().view(np.uint16)
    return v.numpy()


def _check_step(ctx, wl, g, e_prev, k, lr, rng, samples=SAMPLES):
    n, d = wl.n, wl.d
    buf = B.deco_get_buffers(ctx)
    e_new = B.view_f32(buf["e"], (n, buf["e_stride"]))
    msg = B.view_i32(buf["msg"], (n, buf["k_cap"], 2))
    thr, n_greater, _ = B.deco_get_select_info(ctx, n)
    for i in range(n):
        idx = msg[i, :k, 0].long()
        val = msg[i, :k, 1].contiguous().view(torch.float32)
        # --- the message is a valid, and the only valid, Top-k set
        assert int(idx.min()) >= 0 and int(idx.max()) < d
        assert bool((idx[1:] > idx[:-1]).all())
        row = e_new[i, :d]
        assert bool((row[idx].view(torch.int32) == 0).all())          # +0 where sent
        kv = _keys(val)
        t_key = int(kv.min())
        assert t_key == thr[i]
        assert int((kv > t_key).sum()) == n_greater[i]
        rest_max = int(_keys(row).max())
        assert t_key >= rest_max
        if t_key == rest_max and t_key != 0:
            left = torch.nonzero(_keys(row) == t_key).flatten()       # ties not taken
            taken = idx[kv == t_key]
            assert int(taken.max()) < int(left.min())
        # --- arithmetic on sampled positions, through the oracle's accumulate
        pos = torch.from_numpy(rng.integers(0, d, samples)).cuda()
        pos = torch.cat([pos, idx[:: max(1, k // 50_000)]])
        a = O.accumulate(np.float32(lr), _host_bits(g[i], pos),
                         e_prev[i, :d][pos].cpu().numpy())
        sent = torch.zeros(d, dtype=torch.bool, device="cuda")
        sent[idx] = True
        is_sent = sent[pos].cpu().numpy()
        got_e = row[pos].cpu().numpy()
        want_e = np.where(is_sent, np.float32(0.0), a)
        assert np.array_equal(got_e.view(np.uint32), want_e.view(np.uint32))
        # message values are a verbatim
        where = torch.searchsorted(idx, pos[is_sent])
        got_v = val[where].cpu().numpy()
        assert np.array_equal(got_v.view(np.uint32), a[is_sent].view(np.uint32))
        del sent


def _dense_from_messages(msg, n, k, d):
    """Worker-order fp32 sum from +0 with torch index_put (one worker at a time)."""
    S = torch.zeros(d, dtype=torch.float32, device="cuda")
    for i in range(n):
        idx = msg[i, :k, 0].long()
        S[idx] = S[idx] + msg[i, :k, 1].contiguous().view(torch.float32)
    return S


@pytest.mark.parametrize("name", ["gpt2_small", "sweep_100m", "decoder_1b"])
def test_full_size_workload(name):
    wl = W.make_workload(name)
    n, d = wl.n, wl.d
    tau = 1                                   # apply from the second step on (ring logic is
    steps = 3                                 # covered at small sizes); delta and the rest as configured
    rng = np.random.default_rng(wl.seed)
    ctx = B.deco_init(d, n, wl.delta, tau, wl.lr,
                      grad_dtype=B.DECO_F32 if wl.grad_dtype == "f32" else B.DECO_BF16)
    try:
        k = B.deco_get_k(ctx)
        assert k == O.k_from_delta(wl.delta, d)
        buf = B.deco_get_buffers(ctx)
        e_view = B.view_f32(buf["e"], (n, buf["e_stride"]))
        x_view = B.view_f32(buf["params"], (d,))
        msg = B.view_i32(buf["msg"], (n, buf["k_cap"], 2))
        S_prev = None
        g = None
        for t in range(steps):
            g = W.gradients(wl, t, "cuda", out=g)
            e_prev = e_view.clone()
            x_prev = x_view.clone()
            B.deco_ef_compress(ctx, g)
            _check_step(ctx, wl, g, e_prev, k, wl.lr, rng)
            del e_prev
            B.deco_aggregate_stale(ctx)
            # aggregate: every touched index once, with the worker-order fp32 sum
            S = _dense_from_messages(msg, n, k, d)
            addr, positions = B.deco_get_aggregate(ctx, t)
            slot = B.view_i32(addr, (positions, 2))
            keep = slot[:, 0] != -1
            sidx = slot[keep, 0].long()
            sval = slot[keep, 1].contiguous().view(torch.float32)
            touched = torch.zeros(d, dtype=torch.bool, device="cuda")
            for i in range(n):
                touched[msg[i, :k, 0].long()] = True
            assert int(sidx.numel()) == int(touched.sum())
            assert bool((sidx[1:] > sidx[:-1]).all()) and bool(touched[sidx].all())
            assert bool((sval.view(torch.int32) == S[sidx].view(torch.int32)).all())
            del touched
            # the same through the oracle's aggregate, on a sample of the touched indices
            pick = sidx[torch.from_numpy(rng.integers(0, sidx.numel(), 100_000)).cuda()].unique()
            small = []
            for i in range(n):
                idx_i = msg[i, :k, 0].long()
                m = torch.isin(idx_i, pick)
                small.append((torch.searchsorted(pick, idx_i[m]).cpu().numpy().astype(np.uint32),
                              msg[i, :k, 1][m].contiguous().view(torch.float32).cpu().numpy()))
            S_orc, _ = O.aggregate(small, int(pick.numel()))
            got = sval[torch.searchsorted(sidx, pick)].cpu().numpy()
            assert np.array_equal(got.view(np.uint32), S_orc.view(np.uint32))
            B.deco_apply_update(ctx)
            if t >= tau:
                # x_new = fma(-1/n, S_{t-tau}, x_old) through the oracle on sampled positions
                pos = torch.from_numpy(rng.integers(0, d, SAMPLES)).cuda()
                pos = torch.cat([pos, torch.nonzero(S_prev).flatten()[::97][:SAMPLES]])
                xs = x_prev[pos].cpu().numpy().copy()
                O.apply_update(xs, S_prev[pos].cpu().numpy().copy(), np.float32(1.0) / np.float32(n))
                got = x_view[pos].cpu().numpy()
                assert np.array_equal(got.view(np.uint32), xs.view(np.uint32))
                untouched = (S_prev == 0)
                assert bool((x_view.view(torch.int32)[untouched] ==
                             x_prev.view(torch.int32)[untouched]).all())
                del untouched
            else:
                assert bool((x_view == 0).all())
            S_prev = S
            del x_prev
        st = B.deco_get_stats(ctx)
        assert st["device_status"] == 0 and st["exact_pass_workers"] == 0
    finally:
        B.deco_destroy(ctx)
        torch.cuda.empty_cache()


class _Layer:
    """What _check_step reads of a workload, for one layer of the per-layer variant."""
    def __init__(self, n, d):
        self.n, self.d = n, d


def test_full_size_per_layer_variant():
    """GPT-2-small shape, Top-k per tensor (148 layers: 50 through the table-driven kernels, 98
    through the batch kernels for short layers), two iterations with tau = 1.  On a spread of
    layers — the two embeddings, every seventh tensor, the last one — each layer's message is
    pinned as the unique Top-k set of that layer by the properties above, the arithmetic is
    compared with the oracle on sampled positions, and the update of iteration 1 with the
    worker-order sum of iteration 0's messages."""
    wl = W.make_workload("gpt2_small")
    n = wl.n
    offsets = [0]
    for t in wl.tensors:
        offsets.append(offsets[-1] + int(t.numel))
    rng = np.random.default_rng(wl.seed + 1)
    ctx = B.deco_layered_init(wl.d, n, offsets, wl.delta, 1, wl.lr, grad_dtype=B.DECO_BF16)
    try:
        info = B.deco_layered_info(ctx)
        nl = info["n_layers"]
        chosen = sorted(set([0, 1, nl - 1] + list(range(2, nl, 7))))
        x_all = B.view_f32(info["params"], (wl.d,))
        S_prev = {}
        g = None
        for t in range(2):
            g = W.gradients(wl, t, "cuda", out=g)
            subs, e_prev, x_prev = {}, {}, {}
            for l in chosen:
                sub, off, ln = B.deco_layered_layer(ctx, l)
                buf = B.deco_get_buffers(sub)
                subs[l] = (sub, off, ln, buf)
                e_prev[l] = B.view_f32(buf["e"], (n, buf["e_stride"])).clone()
                x_prev[l] = x_all[off:off + ln].clone()
            B.deco_layered_step(ctx, g)
            B.deco_layered_join(ctx)
            torch.cuda.synchronize()
            for l in chosen:
                sub, off, ln, buf = subs[l]
                k_l = B.deco_get_k(sub)
                assert k_l == O.k_from_delta(wl.delta, ln)
                _check_step(sub, _Layer(n, ln), g[:, off:off + ln], e_prev[l], k_l, wl.lr, rng,
                            samples=min(SAMPLES, 4 * ln))
                msg = B.view_i32(buf["msg"], (n, buf["k_cap"], 2))
                S = _dense_from_messages(msg, n, k_l, ln)
                x_new = x_all[off:off + ln]
                if t == 0:
                    assert bool((x_new == 0).all())
                else:
                    want = x_prev[l].cpu().numpy().copy()
                    O.apply_update(want, S_prev[l].cpu().numpy().copy(), np.float32(1.0) / np.float32(n))
                    assert np.array_equal(x_new.cpu().numpy().view(np.uint32), want.view(np.uint32)), l
                S_prev[l] = S
            del e_prev, x_prev
        for l in range(nl):
            st = B.deco_get_stats(B.deco_layered_layer(ctx, l)[0])
            assert st["device_status"] == 0 and st["step"] == 2
    finally:
        B.deco_layered_destroy(ctx)
        torch.cuda.empty_cache()
