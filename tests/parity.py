"""Shared driver of the GPU parity tests: runs libdeco (through the C-ABI binding) and the
CPU oracle side by side on the same seeded gradients and compares every output.

Acceptance (written here once, used by every parity test):
  * selected indices per worker: identical arrays (both sides store them ascending);
  * message values and the residual e: identical bit patterns;
  * aggregated values and parameters: identical bit patterns are expected because both sides
    sum in worker order; the stated bar is |a-b| <= rtol*max(|a|,|b|) + rtol*A with
    rtol = 1e-6 (fp32 gradients) or 1e-2 (bf16 gradients) against the float64 shadow, where
    A is the magnitude of the summed terms (per-entry sum of |term|; guards cancellation).
"""
import numpy as np
import torch

from oracle import dd_ef_sgd as O
from paper_2507_17346_b200 import binding as B
from paper_2507_17346_b200 import workloads as W


def read_messages(ctx, n, k, device=0):
    buf = B.deco_get_buffers(ctx)
    raw = B.view_i32(buf["msg"], (n, buf["k_cap"], 2), device)[:, :k, :].cpu().numpy()
    idx = raw[:, :, 0].view(np.uint32)
    val = np.ascontiguousarray(raw[:, :, 1]).view(np.float32)
    return idx, val


def read_e(ctx, n, d, device=0):
    buf = B.deco_get_buffers(ctx)
    full = B.view_f32(buf["e"], (n, buf["e_stride"]), device)
    pad = full[:, d:]
    assert pad.numel() == 0 or bool((pad == 0).all()), "padding of e must stay zero"
    return full[:, :d].cpu().numpy()


def read_params(ctx, d, device=0):
    buf = B.deco_get_buffers(ctx)
    return B.view_f32(buf["params"], (d,), device).cpu().numpy()


def read_aggregate(ctx, step, device=0, d=None, touched=None):
    """The cached aggregate as (indices ascending, values).  The library keeps it as pairs or,
    for dense messages, as the plain vector S[d]; the vector must be +0 outside `touched`, and
    is returned restricted to `touched`."""
    try:
        addr, positions = B.deco_get_aggregate(ctx, step)
    except B.DecoError as err:
        if err.status != B.DECO_ERR_STATE or d is None:
            raise
        S = B.view_f32(B.deco_get_aggregate_vector(ctx, step), (d,), device).cpu().numpy()
        rest = np.ones(d, dtype=bool)
        rest[touched] = False
        assert not np.any(S.view(np.uint32)[rest]), "dense aggregate: +0 where nothing was sent"
        return touched.astype(np.uint32), S[touched]
    raw = B.view_i32(addr, (positions, 2), device).cpu().numpy()
    idx = raw[:, 0].view(np.uint32)
    val = np.ascontiguousarray(raw[:, 1]).view(np.float32)
    keep = idx != np.uint32(B.DECO_NO_INDEX)
    return idx[keep], val[keep]


def bits(a):
    return np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)


def close(a, b64, scale_terms, rtol):
    a = a.astype(np.float64)
    return np.all(np.abs(a - b64) <= rtol * np.maximum(np.abs(a), np.abs(b64)) + rtol * scale_terms)


def run_parity(d, n, delta, tau, lr, grad_fn, steps, grad_dtype="f32", select_mode=None,
               policy_plan=None, lr_at_server=False, tau_max=0, delta_max=0.0, device=0,
               check_every=1, expect_exact=None, compressor="topk", seed=0):
    """grad_fn(step) -> torch CUDA tensor [n, d] (float32 or bfloat16).

    policy_plan: {step: (delta, tau)} applied before that step on both sides."""
    rtol = 1e-6 if grad_dtype == "f32" else 1e-2
    mode = B.DECO_SELECT_AUTO if select_mode is None else select_mode
    ctx = B.deco_init(d, n, delta, tau, lr,
                      grad_dtype=B.DECO_F32 if grad_dtype == "f32" else B.DECO_BF16,
                      tau_max=tau_max, delta_max=delta_max, lr_at_server=lr_at_server,
                      device=device, select_mode=mode,
                      compressor=B.DECO_COMPRESSOR_RANDK if compressor == "randk"
                      else B.DECO_COMPRESSOR_TOPK, seed=seed)
    try:
        orc = O.DDEFSGD(d, n, delta, tau, lr, lr_in_compress=not lr_at_server,
                        compressor=compressor, seed=seed)
        assert B.deco_get_k(ctx) == orc.k
        abs_S, mass = {}, np.zeros(d)
        scale = float(np.float32(1.0 if not lr_at_server else lr) / np.float32(n))
        for t in range(steps):
            if policy_plan and t in policy_plan:
                B.deco_set_policy(ctx, *policy_plan[t])
                orc.set_policy(*policy_plan[t])
                assert B.deco_get_k(ctx) == orc.k
            g = grad_fn(t)
            assert g.is_cuda and g.shape == (n, d)
            ref = orc.step(W.to_numpy_bits(g))
            k = ref["k"]
            B.deco_ef_compress(ctx, g)
            check = (t % check_every == 0) or t == steps - 1
            if check:
                idx, val = read_messages(ctx, n, k, device)
                for i, (sel, vals) in enumerate(ref["msgs"]):
                    assert np.array_equal(idx[i], sel), "step %d worker %d: index set" % (t, i)
                    assert np.array_equal(bits(val[i]), bits(vals)), \
                        "step %d worker %d: message values" % (t, i)
                e = read_e(ctx, n, d, device)
                assert np.array_equal(bits(e), bits(orc.e)), "step %d: residual" % t
                if expect_exact is not None:
                    _, _, ex = B.deco_get_select_info(ctx, n)
                    assert all(bool(x) == expect_exact for x in ex), (t, ex)
            B.deco_aggregate_stale(ctx)
            terms = np.zeros(d)                                # per-entry sum of |term|
            for s, v in ref["msgs"]:
                terms[s] += np.abs(v.astype(np.float64))
            if check:
                touched = np.unique(np.concatenate([s for s, _ in ref["msgs"]]))
                aidx, aval = read_aggregate(ctx, t, device, d, touched)
                assert np.array_equal(aidx, touched), "step %d: aggregate index set" % t
                terms = np.zeros(d)
                for s, v in ref["msgs"]:
                    terms[s] += np.abs(v.astype(np.float64))
                assert close(aval, ref["S64"][touched], terms[touched], rtol), \
                    "step %d: aggregate vs float64" % t
                assert np.array_equal(bits(aval), bits(ref["S"][touched])), \
                    "step %d: aggregate not the worker-order fp32 sum" % t
            B.deco_apply_update(ctx)
            abs_S[t] = terms
            for s_applied in ref["applied"]:
                mass += scale * abs_S.pop(s_applied)          # magnitude of the summed terms
            if check:
                x = read_params(ctx, d, device)
                assert close(x, orc.x64, mass, rtol), "step %d: parameters vs float64" % t
                assert np.array_equal(bits(x), bits(orc.x)), "step %d: parameters" % t
        st = B.deco_get_stats(ctx)
        assert st["device_status"] == 0 and st["step"] == steps
        assert st["cached_aggregates"] == len(orc.in_flight())
        return st
    finally:
        B.deco_destroy(ctx)


def run_layered_parity(layer_offsets, n, delta, tau, lr, grad_fn, steps, grad_dtype="f32",
                       policy_plan=None, tau_max=0, delta_max=0.0, device=0, select_mode=None):
    """Per-layer Top-k: the layered context (one library context per layer, stepped together)
    against the oracle's per-layer variant, which keeps one flat state and only selects per
    range.  Messages, residuals, aggregates and parameters must agree bit for bit."""
    d = int(layer_offsets[-1])
    ctx = B.deco_layered_init(d, n, layer_offsets, delta, tau, lr,
                              grad_dtype=B.DECO_F32 if grad_dtype == "f32" else B.DECO_BF16,
                              tau_max=tau_max, delta_max=delta_max, device=device,
                              select_mode=B.DECO_SELECT_AUTO if select_mode is None else select_mode)
    try:
        orc = O.DDEFSGD(d, n, delta, tau, lr, layer_offsets=layer_offsets)
        info = B.deco_layered_info(ctx)
        assert info["n_layers"] == len(layer_offsets) - 1 and info["k_total"] == orc.k
        layers = [B.deco_layered_layer(ctx, l) for l in range(info["n_layers"])]
        tau_now = tau
        for t in range(steps):
            if policy_plan and t in policy_plan:
                B.deco_layered_set_policy(ctx, *policy_plan[t])
                orc.set_policy(*policy_plan[t])
                tau_now = policy_plan[t][1]
                assert B.deco_layered_info(ctx)["k_total"] == orc.k
            g = grad_fn(t)
            ref = orc.step(W.to_numpy_bits(g))
            B.deco_layered_step(ctx, g)
            torch.cuda.synchronize()
            idx_parts = [[] for _ in range(n)]
            val_parts = [[] for _ in range(n)]
            agg_idx, agg_val = [], []
            for sub, off, ln in layers:
                k_l = B.deco_get_k(sub)
                idx, val = read_messages(sub, n, k_l, device)
                for i in range(n):
                    idx_parts[i].append(idx[i].astype(np.uint64) + off)
                    val_parts[i].append(val[i])
                e = read_e(sub, n, ln, device)
                assert np.array_equal(bits(e), bits(orc.e[:, off:off + ln])), \
                    "step %d layer at %d: residual" % (t, off)
                if tau_now > 0:        # with tau = 0 the aggregate is consumed inside the step
                    aidx, aval = read_aggregate(sub, t, device)
                    agg_idx.append(aidx.astype(np.uint64) + off)
                    agg_val.append(aval)
            for i, (sel, vals) in enumerate(ref["msgs"]):
                assert np.array_equal(np.concatenate(idx_parts[i]), sel.astype(np.uint64)), \
                    "step %d worker %d: index set" % (t, i)
                assert np.array_equal(bits(np.concatenate(val_parts[i])), bits(vals)), \
                    "step %d worker %d: message values" % (t, i)
            if tau_now > 0:
                touched = np.unique(np.concatenate([s for s, _ in ref["msgs"]]))
                assert np.array_equal(np.concatenate(agg_idx), touched.astype(np.uint64)), \
                    "step %d: aggregate index set" % t
                assert np.array_equal(bits(np.concatenate(agg_val)), bits(ref["S"][touched])), \
                    "step %d: aggregate" % t
            x = B.view_f32(info["params"], (d,), device).cpu().numpy()
            assert np.array_equal(bits(x), bits(orc.x)), "step %d: parameters" % t
        multipass = 0
        for sub, _, _ in layers:
            st = B.deco_get_stats(sub)
            assert st["device_status"] == 0 and st["step"] == steps
            multipass += st["exact_pass_workers"]
        assert B.deco_layered_info(ctx)["step"] == steps
        return multipass
    finally:
        B.deco_layered_destroy(ctx)
