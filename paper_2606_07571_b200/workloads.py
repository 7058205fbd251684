"""Seeded synthetic workloads shaped like the paper's serving scenarios.

This module only *draws inputs* (lengths, prefix assignment, tensors, a
stand-in depth table, a page order).  It holds none of the method's
arithmetic and is the one module both the tests' oracle side and the CUDA side
take their inputs from, so both see the same bytes.

The paper evaluates on public benchmarks with a system prompt as the shared
prefix (shared-prefix ratio 76-95 %, a 22 % low-ratio variant, output lengths
256/512, 32 layers).  Those datasets are not used here; the workloads below
reproduce their shapes only.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np
import torch


def standin_depth_table(num_layers: int) -> np.ndarray:
    """Stand-in for the profiled lookup table T (ratio bin -> shallow depth).

    The paper prints no table values (its ratio->depth curve is a figure), so
    this is an input recipe, not a reproduction: non-decreasing in the ratio,
    at least 1 for any shared prefix, about half the layers at ratio 0.85
    (the paper's average workload) and all layers at ratio 1.
    """
    L = int(num_layers)
    t = np.empty(101, dtype=np.int32)
    t[0] = min(1, L)
    for idx in range(1, 101):
        t[idx] = min(L, max(1, (L * idx ** 4) // (100 ** 4)))
    return t


def shuffled_page_order(num_pages: int, seed: int) -> np.ndarray:
    """A seeded permutation of the page indices (scattered physical pages)."""
    return np.random.default_rng(seed).permutation(num_pages).astype(np.int32)


@dataclass
class Workload:
    name: str
    num_layers: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    dtype: torch.dtype
    page_size: int
    prefix_lens: list            # m_g per distinct prefix
    req_prefix: list             # prefix index of each request (grouped: non-decreasing)
    suffix_lens: list            # n_i per request
    softmax_scale: float
    value_std: float = 1.0       # std of Q, K, V entries
    seed: int = 0
    shuffle_pages: bool = False
    note: str = ""
    # derived
    full_lens: list = field(default_factory=list)       # N_i = m + n
    full_row_off: list = field(default_factory=list)    # first row of request i in the full buffers
    suffix_row_off: list = field(default_factory=list)  # first suffix row of request i

    def __post_init__(self):
        off = 0
        self.full_lens, self.full_row_off, self.suffix_row_off = [], [], []
        for g, n in zip(self.req_prefix, self.suffix_lens):
            m = self.prefix_lens[g]
            self.full_row_off.append(off)
            self.suffix_row_off.append(off + m)
            self.full_lens.append(m + n)
            off += m + n
        self.total_rows = off

    @property
    def num_requests(self):
        return len(self.suffix_lens)

    @property
    def suffix_tokens(self):
        return int(sum(self.suffix_lens))

    def pages_needed(self):
        return sum((m + self.page_size - 1) // self.page_size for m in self.prefix_lens)

    def req_prefix_len(self):
        return [self.prefix_lens[g] for g in self.req_prefix]

    def attend_flops(self):
        """Algorithmic FLOPs of one shallow layer with every request reusing."""
        return 4 * self.head_dim * self.num_q_heads * sum(
            n * (self.prefix_lens[g] + n) for g, n in zip(self.req_prefix, self.suffix_lens))

    def attend_bytes(self):
        """Algorithmic bytes of one `attend` launch: every group's cached K and V once, every
        request's suffix Q, K, V read and output written once."""
        e = 2 if self.dtype == torch.bfloat16 else 4
        groups = sorted(set(self.req_prefix))
        b = sum(2 * self.prefix_lens[g] * self.num_kv_heads * self.head_dim * e for g in groups)
        b += sum(2 * n * (self.num_q_heads + self.num_kv_heads) * self.head_dim * e for n in self.suffix_lens)
        return b

    def full_flops(self):
        """Algorithmic FLOPs of one deep layer with every request recomputing."""
        return 4 * self.head_dim * self.num_q_heads * sum(N * N for N in self.full_lens)


def _normal(shape, gen, dtype, device, std):
    x = torch.randn(shape, generator=gen, device=device, dtype=torch.float32)
    if std != 1.0:
        x = x * std
    return x.to(dtype)


def draw_full_qkv(w: Workload, device="cpu"):
    """Q [rows, Hq, D], K, V [rows, Hkv, D] for every request's full input
    (prefix rows then suffix rows), one set reused by every layer."""
    gen = torch.Generator(device=device)
    gen.manual_seed(w.seed)
    q = _normal((w.total_rows, w.num_q_heads, w.head_dim), gen, w.dtype, device, w.value_std)
    k = _normal((w.total_rows, w.num_kv_heads, w.head_dim), gen, w.dtype, device, w.value_std)
    v = _normal((w.total_rows, w.num_kv_heads, w.head_dim), gen, w.dtype, device, w.value_std)
    return q, k, v


def draw_prefix_kv(w: Workload, g: int, device="cpu", layers=None):
    """Cached K, V [L, m_g, Hkv, D] of prefix g, drawn independently per layer
    (seed depends on the prefix only, so any subset of layers can be redrawn)."""
    L = w.num_layers
    m = w.prefix_lens[g]
    ks, vs = [], []
    for l in (range(L) if layers is None else layers):
        gen = torch.Generator(device=device)
        gen.manual_seed(w.seed * 1000003 + 7919 * (g + 1) + 104729 * (l + 1))
        ks.append(_normal((m, w.num_kv_heads, w.head_dim), gen, w.dtype, device, w.value_std))
        vs.append(_normal((m, w.num_kv_heads, w.head_dim), gen, w.dtype, device, w.value_std))
    return torch.stack(ks), torch.stack(vs)


def draw_hidden_and_weights(m, d_model, num_kv_heads, head_dim, seed, dtype=torch.bfloat16, device="cpu"):
    """Inputs of the K/V projection of one layer: hidden states h [m, d_model] ~ N(0, 1) (the scale
    of a normalised residual stream) and weights w_k, w_v [Hkv * D, d_model] ~ N(0, 1 / d_model), so
    that the projected K/V have unit variance like the drawn ones."""
    gen = torch.Generator(device=device)
    gen.manual_seed(seed * 1000003 + 15485863)
    h = _normal((m, d_model), gen, dtype, device, 1.0)
    out = num_kv_heads * head_dim
    w_k = _normal((out, d_model), gen, dtype, device, d_model ** -0.5)
    w_v = _normal((out, d_model), gen, dtype, device, d_model ** -0.5)
    return h, w_k, w_v


def prefix_key(w: Workload, g: int) -> int:
    """A 64-bit identifier standing in for the hash of the prefix's token ids."""
    return (0x9E3779B97F4A7C15 * (g + 1) + w.seed) & 0xFFFFFFFFFFFFFFFF


def to_f64(t: torch.Tensor) -> np.ndarray:
    """Exact widening of a tensor's values to float64 on the host."""
    return t.detach().to("cpu").to(torch.float64).numpy()


# ---------------------------------------------------------------------------
# The five configurations and the small-suffix bandwidth shapes.
# ---------------------------------------------------------------------------

def config1():
    return Workload("config1-tiny-fp32", 1, 4, 4, 64, torch.float32, 16,
                    [64], [0] * 4, [32] * 4, softmax_scale=1.0 / 8.0, value_std=1.0 / 8.0,
                    note="tiny op: 1 prefix of 64 tokens, 4 requests x 32 suffix tokens")


def config2():
    return Workload("config2-llada-layer", 1, 32, 32, 128, torch.bfloat16, 16,
                    [1024], [0] * 16, [256] * 16, softmax_scale=128 ** -0.5,
                    note="LLaDA-8B-shaped layer: prefix 1024, 16 requests x 256 suffix tokens")


def config3():
    rng = np.random.default_rng(0)
    n = rng.integers(64, 513, size=64).tolist()
    return Workload("config3-llada-stack", 32, 32, 32, 128, torch.bfloat16, 16,
                    [2048], [0] * 64, n, softmax_scale=128 ** -0.5,
                    note="32-layer stack: one 2048-token prefix, 64 requests, suffix U[64,512]")


def config4():
    rng = np.random.default_rng(0)
    m = rng.integers(512, 4097, size=8).tolist()
    p = np.arange(1, 9, dtype=np.float64) ** -1.1
    p /= p.sum()
    assign = np.sort(rng.choice(8, size=256, p=p)).tolist()
    n = rng.integers(32, 1025, size=256).tolist()
    return Workload("config4-serving-mix", 32, 32, 32, 128, torch.bfloat16, 16,
                    m, assign, n, softmax_scale=128 ** -0.5, shuffle_pages=True,
                    note="8 prefixes U[512,4096], 256 requests Zipf(1.1), suffix U[32,1024]")


def config5():
    return Workload("config5-dream-gqa", 28, 28, 4, 128, torch.bfloat16, 16,
                    [16384], [0] * 32, [1024] * 32, softmax_scale=128 ** -0.5,
                    note="Dream-7B-shaped GQA 28/4: prefix 16384, 32 requests x 1024")


def small_suffix(name):
    """Bandwidth-bound supplementary shapes (few query rows per cached tile)."""
    table = {
        "b1": (32, 32, 32, [4096], [32]),
        "b2": (32, 32, 32, [16384], [32]),
        "b3": (32, 32, 32, [16384], [32] * 4),
        "b4": (28, 28, 4, [16384], [16]),
    }
    L, hq, hkv, m, n = table[name]
    return Workload("small-suffix-" + name, L, hq, hkv, 128, torch.bfloat16, 16,
                    m, [0] * len(n), n, softmax_scale=128 ** -0.5,
                    note="small-suffix shape %s: prefix %d, %d request(s) x %d" % (name, m[0], len(n), n[0]))


def scaled_down(w: Workload, num_layers=None, max_requests=None, prefix_div=1, suffix_div=1,
                name=None):
    """A smaller workload with the same structure (for element-by-element
    parity at sizes the oracle finishes in seconds)."""
    L = w.num_layers if num_layers is None else num_layers
    R = w.num_requests if max_requests is None else min(max_requests, w.num_requests)
    # keep one request out of every (num_requests // R) so every group survives where possible
    idx = np.linspace(0, w.num_requests - 1, R).round().astype(int).tolist()
    groups = sorted(set(w.req_prefix[i] for i in idx))
    remap = {g: j for j, g in enumerate(groups)}
    m = [max(1, w.prefix_lens[g] // prefix_div) for g in groups]
    return Workload(name or (w.name + "-small"), L, w.num_q_heads, w.num_kv_heads, w.head_dim,
                    w.dtype, w.page_size, m, [remap[w.req_prefix[i]] for i in idx],
                    [max(1, w.suffix_lens[i] // suffix_div) for i in idx],
                    softmax_scale=w.softmax_scale, value_std=w.value_std, seed=w.seed,
                    shuffle_pages=w.shuffle_pages, note=w.note + " (scaled down)")


def config5_small():
    """Four of config 5's 32 requests (same prefix, same lengths): a case small enough for a full
    profiler capture; DRAM traffic per launch scales with the number of requests."""
    w = config5()
    return Workload("config5-dream-gqa-4req", w.num_layers, w.num_q_heads, w.num_kv_heads, w.head_dim, w.dtype, 16,
                    w.prefix_lens, [0] * 4, [1024] * 4, softmax_scale=w.softmax_scale,
                    note="config 5 with 4 of its 32 requests (profiling case)")


CONFIGS = {
    "config1": config1, "config2": config2, "config3": config3,
    "config4": config4, "config5": config5, "config5s": config5_small,
    "b1": lambda: small_suffix("b1"), "b2": lambda: small_suffix("b2"),
    "b3": lambda: small_suffix("b3"), "b4": lambda: small_suffix("b4"),
}
