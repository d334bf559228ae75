"""Seeded synthetic inputs: gradient tensors shaped like the paper's workloads, and the
network trace that feeds the DeCo policy.

This module is plumbing shared by the tests, the benchmark and the CPU oracle's callers.  It
contains none of the method's arithmetic (no error feedback, no Top-k, no aggregation, no
policy): it only draws random numbers with a stated shape, scale and structure.  The paper's
own gradients came from CIFAR-10 / ImageNet / Wikitext training runs, which need datasets and
trained weights; the recipes below stand in for them.

Every draw is a pure function of (workload seed, step, worker): the generator is re-seeded
per (step, worker), so any step can be regenerated on its own.  CPU and CUDA generators give
different streams; callers generate once on one device and copy.
"""
from dataclasses import dataclass, field
from typing import List, Tuple

import numpy as np
import torch


@dataclass
class TensorSpec:
    name: str
    shape: Tuple[int, ...]
    layer: int = -1                     # layer index (for per-layer scales), -1 = none

    @property
    def numel(self):
        n = 1
        for s in self.shape:
            n *= s
        return n

    @property
    def fan_in(self):
        n = 1
        for s in self.shape[1:]:
            n *= s
        return n


@dataclass
class Workload:
    name: str
    n: int                               # workers
    delta: float                         # compression ratio
    tau: int                             # staleness
    lr: float
    steps: int
    grad_dtype: str                      # "f32" or "bf16"
    dist: str                            # "normal" | "student_t" | "normal_outlier_rows" | "normal_layer_scale"
    tensors: List[TensorSpec] = field(default_factory=list)
    sigma: float = 1.0
    seed: int = 0xDEC0

    @property
    def d(self):
        return sum(t.numel for t in self.tensors)


# ----------------------------------------------------------------------------- shapes

def flat_shape(d):
    return [TensorSpec("flat", (int(d),))]


def resnet18_shapes(width=64, classes=1000):
    """The 62 parameter tensors of a ResNet-18 (conv / batch-norm / fc), in module order."""
    w = width
    out = [TensorSpec("conv1.weight", (w, 3, 7, 7)),
           TensorSpec("bn1.weight", (w,)), TensorSpec("bn1.bias", (w,))]
    cin = w
    for stage, cout in enumerate([w, 2 * w, 4 * w, 8 * w]):
        for blk in range(2):
            p = "layer%d.%d." % (stage + 1, blk)
            out += [TensorSpec(p + "conv1.weight", (cout, cin, 3, 3)),
                    TensorSpec(p + "bn1.weight", (cout,)), TensorSpec(p + "bn1.bias", (cout,)),
                    TensorSpec(p + "conv2.weight", (cout, cout, 3, 3)),
                    TensorSpec(p + "bn2.weight", (cout,)), TensorSpec(p + "bn2.bias", (cout,))]
            if blk == 0 and cin != cout:
                out += [TensorSpec(p + "downsample.0.weight", (cout, cin, 1, 1)),
                        TensorSpec(p + "downsample.1.weight", (cout,)),
                        TensorSpec(p + "downsample.1.bias", (cout,))]
            cin = cout
    out += [TensorSpec("fc.weight", (classes, 8 * w)), TensorSpec("fc.bias", (classes,))]
    return out


def gpt2_shapes(n_layer=12, d_model=768, vocab=50257, n_ctx=1024):
    """GPT-2 parameter tensors with the output head tied to the token embedding."""
    m = d_model
    out = [TensorSpec("wte", (vocab, m)), TensorSpec("wpe", (n_ctx, m))]
    for l in range(n_layer):
        p = "h.%d." % l
        out += [TensorSpec(p + "ln_1.weight", (m,), l), TensorSpec(p + "ln_1.bias", (m,), l),
                TensorSpec(p + "attn.c_attn.weight", (3 * m, m), l),
                TensorSpec(p + "attn.c_attn.bias", (3 * m,), l),
                TensorSpec(p + "attn.c_proj.weight", (m, m), l),
                TensorSpec(p + "attn.c_proj.bias", (m,), l),
                TensorSpec(p + "ln_2.weight", (m,), l), TensorSpec(p + "ln_2.bias", (m,), l),
                TensorSpec(p + "mlp.c_fc.weight", (4 * m, m), l),
                TensorSpec(p + "mlp.c_fc.bias", (4 * m,), l),
                TensorSpec(p + "mlp.c_proj.weight", (m, 4 * m), l),
                TensorSpec(p + "mlp.c_proj.bias", (m,), l)]
    out += [TensorSpec("ln_f.weight", (m,)), TensorSpec("ln_f.bias", (m,))]
    return out


def decoder_shapes(n_layer=22, d_model=2048, d_ffn=5632, vocab=32000, d_kv=256):
    """Decoder with grouped-query attention, gated FFN, two norms per layer, untied
    input/output embeddings and a final norm (22/2048/5632/32000/256 gives 1.1 B)."""
    m = d_model
    out = [TensorSpec("embed", (vocab, m))]
    for l in range(n_layer):
        p = "layers.%d." % l
        out += [TensorSpec(p + "attn_norm", (m,), l),
                TensorSpec(p + "q_proj", (m, m), l), TensorSpec(p + "k_proj", (d_kv, m), l),
                TensorSpec(p + "v_proj", (d_kv, m), l), TensorSpec(p + "o_proj", (m, m), l),
                TensorSpec(p + "ffn_norm", (m,), l),
                TensorSpec(p + "gate_proj", (d_ffn, m), l),
                TensorSpec(p + "up_proj", (d_ffn, m), l),
                TensorSpec(p + "down_proj", (m, d_ffn), l)]
    out += [TensorSpec("final_norm", (m,)), TensorSpec("lm_head", (vocab, m))]
    return out


# -------------------------------------------------------------------------- workloads

def make_workload(name, scale=1.0):
    """The five benchmark configurations; scale < 1 shrinks widths for CPU-sized tests
    while keeping the tensor structure, dtype, distribution, delta and tau."""
    s = float(scale)

    def sc(v, mult=8):
        return max(mult, int(round(v * s / mult)) * mult)

    if name == "flat_1m":
        return Workload(name, n=4, delta=0.01, tau=2, lr=0.1, steps=20, grad_dtype="f32",
                        dist="normal", tensors=flat_shape(sc(1 << 20)), seed=0xDEC1)
    if name == "resnet18":
        return Workload(name, n=8, delta=0.01, tau=4, lr=0.1, steps=50, grad_dtype="f32",
                        dist="student_t", seed=0xDEC2,
                        tensors=resnet18_shapes(sc(64), classes=sc(1000)))
    if name == "gpt2_small":
        return Workload(name, n=8, delta=0.001, tau=8, lr=0.1, steps=20, grad_dtype="bf16",
                        dist="normal_outlier_rows", sigma=0.02, seed=0xDEC3,
                        tensors=gpt2_shapes(12 if s == 1.0 else max(2, int(12 * s)), sc(768),
                                            50257 if s == 1.0 else sc(50257),
                                            sc(1024)))
    if name == "sweep_100m":
        return Workload(name, n=4, delta=0.01, tau=2, lr=0.1, steps=200, grad_dtype="f32",
                        dist="normal", tensors=flat_shape(sc(100_000_000)), seed=0xDEC4)
    if name == "decoder_1b":
        return Workload(name, n=4, delta=0.001, tau=4, lr=0.1, steps=10, grad_dtype="bf16",
                        dist="normal_layer_scale", sigma=0.01, seed=0xDEC5,
                        tensors=decoder_shapes(22 if s == 1.0 else max(2, int(22 * s)),
                                               sc(2048), sc(5632), sc(32000), sc(256)))
    raise KeyError(name)


WORKLOADS = ["flat_1m", "resnet18", "gpt2_small", "sweep_100m", "decoder_1b"]


# -------------------------------------------------------------------------- gradients

def _gen(device, seed):
    g = torch.Generator(device=device)
    g.manual_seed(int(seed) & 0x7FFFFFFFFFFFFFFF)
    return g


def _mix(*vals):
    """64-bit mix of integers (splitmix-style) for per-(step, worker) seeds."""
    h = 0x9E3779B97F4A7C15
    for v in vals:
        h ^= (int(v) + 0x9E3779B97F4A7C15 + ((h << 6) & 0xFFFFFFFFFFFFFFFF) + (h >> 2))
        h &= 0xFFFFFFFFFFFFFFFF
        h = (h ^ (h >> 30)) * 0xBF58476D1CE4E5B9 & 0xFFFFFFFFFFFFFFFF
        h = (h ^ (h >> 27)) * 0x94D049BB133111EB & 0xFFFFFFFFFFFFFFFF
        h ^= h >> 31
    return h


def outlier_rows(wl, spec_index, device="cpu"):
    """Rows (2-D tensors) or entries (1-D) that carry the x50 outlier scale: 1 % of them,
    fixed for the workload (the same for every step and worker)."""
    spec = wl.tensors[spec_index]
    rows = spec.shape[0] if len(spec.shape) > 1 else spec.numel
    g = _gen("cpu", _mix(wl.seed, 0x0071, spec_index))
    return (torch.rand(rows, generator=g) < 0.01).to(device)


def layer_scales(wl):
    """Per-tensor multiplier for 'normal_layer_scale': 10^U[-1,1], one draw per layer index
    (shared by the layer's tensors); tensors outside any layer get their own draw."""
    rs = np.random.RandomState(wl.seed & 0x7FFFFFFF)
    n_layers = 1 + max([t.layer for t in wl.tensors] + [-1])
    per_layer = 10.0 ** rs.uniform(-1.0, 1.0, size=n_layers)
    out = []
    for t in wl.tensors:
        out.append(float(per_layer[t.layer]) if t.layer >= 0
                   else float(10.0 ** rs.uniform(-1.0, 1.0)))
    return out


_CHUNK = 1 << 26


def _randn(numel, gen, device):
    return torch.randn(numel, generator=gen, device=device, dtype=torch.float32)


def gradients(wl, step, device="cpu", out=None):
    """Gradients of all n workers for one step: tensor [n, d], float32 or bfloat16."""
    dtype = torch.float32 if wl.grad_dtype == "f32" else torch.bfloat16
    d = wl.d
    if out is None:
        out = torch.empty((wl.n, d), dtype=dtype, device=device)
    assert out.shape == (wl.n, d) and out.dtype == dtype
    scales = layer_scales(wl) if wl.dist == "normal_layer_scale" else None
    masks = None
    if wl.dist == "normal_outlier_rows":
        masks = [outlier_rows(wl, ti, device) for ti in range(len(wl.tensors))]
    for i in range(wl.n):
        gen = _gen(device, _mix(wl.seed, step, i))
        off = 0
        for ti, spec in enumerate(wl.tensors):
            numel = spec.numel
            for c0 in range(0, numel, _CHUNK):
                c1 = min(numel, c0 + _CHUNK)
                m = c1 - c0
                z = _randn(m, gen, device)
                if wl.dist == "student_t":
                    # Student-t, nu = 3: z / sqrt(chi2_3 / 3), scaled by 1/sqrt(fan_in)
                    w = _randn(3 * m, gen, device).view(3, m)
                    z = z / torch.sqrt((w * w).sum(0) / 3.0)
                    z = z * (1.0 / float(spec.fan_in) ** 0.5)
                elif wl.dist == "normal_outlier_rows":
                    z = z * wl.sigma
                    cols = spec.fan_in if len(spec.shape) > 1 else 1
                    # chunk boundaries may cut a row; expand the row mask over the chunk
                    idx = torch.arange(c0, c1, device=device) // cols
                    z = torch.where(masks[ti][idx], z * 50.0, z)
                elif wl.dist == "normal_layer_scale":
                    z = z * (wl.sigma * scales[ti])
                else:
                    z = z * wl.sigma
                out[i, off + c0: off + c1] = z.to(dtype)
            off += numel
    return out


def entry_scales(wl, device="cpu"):
    """Per-entry multiplier [d] float32 that turns unit draws into the workload's values:
    1/sqrt(fan_in) of the entry's tensor (Student-t recipe), sigma times the layer's scale,
    sigma times 50 on the outlier rows, or sigma."""
    parts = []
    scales = layer_scales(wl) if wl.dist == "normal_layer_scale" else None
    for ti, spec in enumerate(wl.tensors):
        if wl.dist == "student_t":
            parts.append(torch.full((spec.numel,), 1.0 / float(spec.fan_in) ** 0.5))
        elif wl.dist == "normal_layer_scale":
            parts.append(torch.full((spec.numel,), wl.sigma * scales[ti]))
        elif wl.dist == "normal_outlier_rows":
            cols = spec.fan_in if len(spec.shape) > 1 else 1
            rows = outlier_rows(wl, ti).repeat_interleave(cols)
            parts.append(torch.where(rows, 50.0 * wl.sigma, wl.sigma).to(torch.float32))
        else:
            parts.append(torch.full((spec.numel,), float(wl.sigma)))
    return torch.cat(parts).to(torch.float32).to(device)


def gradients_batched(wl, step, scales, out=None):
    """The workload's distribution drawn for all workers at once (a handful of device launches
    per step instead of several per tensor and worker): unit draws [n, d] times `scales` =
    entry_scales(wl, device).  Another stream than gradients(), the same recipe."""
    device = scales.device
    gen = _gen(device, _mix(wl.seed, step, 0x6261))
    z = torch.randn((wl.n, wl.d), generator=gen, device=device, dtype=torch.float32)
    if wl.dist == "student_t":
        w = torch.randn((3, wl.n, wl.d), generator=gen, device=device, dtype=torch.float32)
        z = z / torch.sqrt((w * w).sum(0) / 3.0)
    z = z * scales
    dtype = torch.float32 if wl.grad_dtype == "f32" else torch.bfloat16
    if out is None:
        return z.to(dtype)
    out.copy_(z)
    return out


def to_numpy_bits(g):
    """Host copy for the oracle: float32 array, or uint16 bit patterns for bfloat16."""
    g = g.detach().cpu().contiguous()
    if g.dtype == torch.bfloat16:
        return g.view(torch.int16).numpy().view(np.uint16)
    return g.numpy()


# ------------------------------------------------------------------------------ trace

def network_trace(seed, steps, seg_len=(10, 40), latency_s=(0.020, 0.200),
                  bandwidth_bps=(0.1e9, 10e9)):
    """Piecewise-constant (latency, bandwidth) per step: segment lengths U{10..40} steps,
    latency U[20, 200] ms, bandwidth log-uniform in [0.1, 10] Gbps."""
    rs = np.random.RandomState(int(seed) & 0x7FFFFFFF)
    lat = np.empty(steps)
    bw = np.empty(steps)
    t = 0
    while t < steps:
        L = int(rs.randint(seg_len[0], seg_len[1] + 1))
        b = rs.uniform(*latency_s)
        a = float(np.exp(rs.uniform(np.log(bandwidth_bps[0]), np.log(bandwidth_bps[1]))))
        lat[t:t + L] = b
        bw[t:t + L] = a
        t += L
    return lat, bw
