"""Seeded synthetic inputs and workload shapes for the Union-of-Experts hot path.

This module only *describes problems* and *draws random numbers*.  It holds none of the
method's arithmetic (no gate, no selection, no expert math): both the CPU oracle's tests
and the CUDA path's tests/bench take their inputs from here, so the two sides see the same
bits without sharing any code of the method itself.

Random numbers come from a counter-based generator written from its published definition:
SplitMix64 (Steele, Lea, Flood 2014: golden-gamma counter, two xor-shift-multiply rounds)
feeding the Box-Muller transform in float64.  Element e of stream s under a seed is a pure
function of (seed, s, e), so arrays can be produced in chunks, in any order.

Workloads: the shapes follow the paper's three experiment families (causal language
modelling, long-sequence classification, ViT image tokens; Section IV) plus a small fp32
check and a large scale case.  They stand in for the paper's datasets, none of which is
used: x ~ N(0,1) iid, weights ~ N(0, w_std), router ~ N(0, 0.02), upstream grad ~ N(0,1).
"""
from __future__ import annotations

import dataclasses
from dataclasses import dataclass

import numpy as np

_MASK = np.uint64(0xFFFFFFFFFFFFFFFF)
_GAMMA = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)


def _splitmix64(z: np.ndarray) -> np.ndarray:
    """SplitMix64 output function applied to an array of 64-bit states (wrapping arithmetic)."""
    with np.errstate(over="ignore"):
        z = (z ^ (z >> np.uint64(30))) * _M1
        z = (z ^ (z >> np.uint64(27))) * _M2
        z = z ^ (z >> np.uint64(31))
    return z


def _stream_base(seed: int, stream: int) -> np.uint64:
    s = _splitmix64(np.array([(seed * 0x9E3779B97F4A7C15 + 0x1234567) & 0xFFFFFFFFFFFFFFFF], dtype=np.uint64))
    t = _splitmix64(s ^ np.uint64((stream * 0xD1342543DE82EF95 + 1) & 0xFFFFFFFFFFFFFFFF))
    return t[0]


def uniform_bits(seed: int, stream: int, start: int, count: int) -> np.ndarray:
    """64 random bits for elements [start, start+count) of a stream."""
    base = _stream_base(seed, stream)
    with np.errstate(over="ignore"):
        ctr = (np.arange(start, start + count, dtype=np.uint64) + np.uint64(1)) * _GAMMA + base
    return _splitmix64(ctr)


def normal(seed: int, stream: int, shape, std: float = 1.0, chunk: int = 1 << 22) -> np.ndarray:
    """float64 array of N(0, std^2) draws; element e uses counters 2e and 2e+1 (Box-Muller)."""
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.float64)
    inv = 1.0 / 9007199254740992.0  # 2^-53
    for s in range(0, n, chunk):
        cnt = min(chunk, n - s)
        bits = uniform_bits(seed, stream, 2 * s, 2 * cnt)
        u1 = ((bits[0::2] >> np.uint64(11)).astype(np.float64) + 1.0) * inv  # (0, 1]
        u2 = (bits[1::2] >> np.uint64(11)).astype(np.float64) * inv          # [0, 1)
        out[s:s + cnt] = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
    if std != 1.0:
        out *= std
    return out.reshape(shape)


def integers(seed: int, stream: int, count: int, high: int) -> np.ndarray:
    """`count` integers in [0, high) (modulo reduction of 64 random bits; bias < 2^-40 for small high)."""
    return (uniform_bits(seed, stream, 0, count) % np.uint64(high)).astype(np.int64)


# ----------------------------------------------------------------------------------------------
# storage formats: the values both sides compute on are the *rounded* ones
# ----------------------------------------------------------------------------------------------

def round_f32(a: np.ndarray) -> np.ndarray:
    return np.asarray(a, dtype=np.float64).astype(np.float32)


def f32_to_bf16_bits(a32: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (round to nearest, ties to even); returns the uint16 patterns."""
    u = np.ascontiguousarray(a32, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = u + np.uint32(0x7FFF) + lsb
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


@dataclass
class Stored:
    """One input array in its storage format: `f64` holds exactly the stored values."""
    f64: np.ndarray            # what the oracle reads
    raw: np.ndarray            # float32 array (dtype f32) or uint16 bf16 bit patterns (dtype bf16)
    dtype: str                 # "f32" | "bf16"


def store(a: np.ndarray, dtype: str) -> Stored:
    if dtype == "f32":
        r = round_f32(a)
        return Stored(r.astype(np.float64), r, "f32")
    if dtype == "bf16":
        bits = f32_to_bf16_bits(np.asarray(a, dtype=np.float64).astype(np.float32))
        return Stored(bf16_bits_to_f64(bits), bits, "bf16")
    raise ValueError(dtype)


# ----------------------------------------------------------------------------------------------
# workloads
# ----------------------------------------------------------------------------------------------

@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    L: int              # padded length = m * l_p
    L_valid: int        # tokens that are real (the rest are zero pad rows)
    d: int
    n: int              # experts (both blocks use the same count in every workload here)
    k: int              # experts per sample
    m: int              # patches per sample
    c: int              # patches per expert
    d_ff: int           # MLP hidden width, split over n experts (0 = no UoME block)
    H: int              # attention heads (0 = no SMHA block)
    d_h: int
    dtype: str          # "f32" | "bf16"
    act: str            # "gelu_erf" | "gelu_tanh" | "silu" | "identity"
    causal: bool
    w_std: float
    seed: int
    backward: bool = False
    stands_in_for: str = ""

    @property
    def l_p(self) -> int:
        return self.L // self.m

    @property
    def l_a(self) -> int:
        return self.c * self.l_p

    @property
    def d_e(self) -> int:
        return self.d_ff // self.n if self.d_ff else 0

    @property
    def d_g(self) -> int:
        return (self.H // self.n) * self.d_h if self.H else 0

    @property
    def R(self) -> int:
        return self.B * self.k * self.l_a

    def replace(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


WORKLOADS = {
    "cfg1_small_f32": Workload("cfg1_small_f32", B=2, L=256, L_valid=256, d=256, n=4, k=2, m=8, c=4,
                               d_ff=1024, H=0, d_h=0, dtype="f32", act="gelu_erf", causal=False,
                               w_std=0.02, seed=0, stands_in_for="unit-scale check"),
    "cfg2_lm": Workload("cfg2_lm", B=16, L=512, L_valid=512, d=512, n=8, k=4, m=16, c=8,
                        d_ff=2048, H=8, d_h=64, dtype="bf16", act="silu", causal=True,
                        w_std=0.02, seed=1, stands_in_for="causal language modelling block"),
    "cfg3_long": Workload("cfg3_long", B=8, L=4096, L_valid=4096, d=256, n=4, k=2, m=64, c=16,
                          d_ff=1024, H=4, d_h=64, dtype="bf16", act="silu", causal=False,
                          w_std=0.02, seed=2, stands_in_for="long-sequence classification block"),
    "cfg4_vit": Workload("cfg4_vit", B=256, L=224, L_valid=197, d=384, n=6, k=3, m=14, c=7,
                         d_ff=1536, H=6, d_h=64, dtype="bf16", act="silu", causal=False,
                         w_std=0.02, seed=3, stands_in_for="ViT image-token block (196 + cls, padded to 224)"),
    "cfg5_scale": Workload("cfg5_scale", B=8, L=4096, L_valid=4096, d=4096, n=16, k=4, m=32, c=16,
                           d_ff=16384, H=0, d_h=0, dtype="bf16", act="silu", causal=False,
                           w_std=0.01, seed=4, backward=True, stands_in_for="large language-model MLP block"),
}

# stream ids (fixed so every consumer draws the same arrays)
S_X, S_WR_MLP, S_W1, S_W2, S_WR_ATT, S_WQ, S_WK, S_WV, S_WO, S_DY, S_SKEW = range(11)


def make_x(w: Workload, skew_beta: float = 0.0, W_r: np.ndarray | None = None) -> Stored:
    """x[B, L, d] ~ N(0,1); rows t >= L_valid are zero.

    With skew_beta > 0 every valid row of sample b is shifted along the direction of one router
    column (drawn per sample with Zipf(1) weights over experts), which raises that expert's logit
    by skew_beta: a deliberately imbalanced expert load.
    """
    x = normal(w.seed, S_X, (w.B, w.L, w.d))
    if skew_beta > 0.0:
        assert W_r is not None
        p = 1.0 / np.arange(1, w.n + 1)
        cdf = np.cumsum(p / p.sum())
        u = (uniform_bits(w.seed, S_SKEW, 0, w.B) >> np.uint64(11)).astype(np.float64) / 9007199254740992.0
        z = np.minimum(np.searchsorted(cdf, u), w.n - 1)
        for b in range(w.B):
            col = W_r[:, z[b]]
            x[b] += skew_beta * col / float(col @ col)
    if w.L_valid < w.L:
        x[:, w.L_valid:, :] = 0.0
    return store(x, w.dtype)


def make_router(w: Workload, block: str = "mlp") -> Stored:
    return store(normal(w.seed, S_WR_MLP if block == "mlp" else S_WR_ATT, (w.d, w.n), 0.02), w.dtype)


def make_mlp_weights(w: Workload):
    """A^I as [n, d, d_e] (column slices of the first layer), A^O as [n, d_e, d] (row slices of the second)."""
    W1 = store(normal(w.seed, S_W1, (w.n, w.d, w.d_e), w.w_std), w.dtype)
    W2 = store(normal(w.seed, S_W2, (w.n, w.d_e, w.d), w.w_std), w.dtype)
    return W1, W2


def make_attn_weights(w: Workload):
    """W^q, W^k, W^v as [n, d, d_g]; W^o as [n, d_g, d]."""
    Wq = store(normal(w.seed, S_WQ, (w.n, w.d, w.d_g), w.w_std), w.dtype)
    Wk = store(normal(w.seed, S_WK, (w.n, w.d, w.d_g), w.w_std), w.dtype)
    Wv = store(normal(w.seed, S_WV, (w.n, w.d, w.d_g), w.w_std), w.dtype)
    Wo = store(normal(w.seed, S_WO, (w.n, w.d_g, w.d), w.w_std), w.dtype)
    return Wq, Wk, Wv, Wo


def make_dy(w: Workload) -> Stored:
    dy = normal(w.seed, S_DY, (w.B, w.L, w.d))
    if w.L_valid < w.L:
        dy[:, w.L_valid:, :] = 0.0
    return store(dy, w.dtype)


def tiny(name: str = "tiny", **kw) -> Workload:
    """A small workload for exhaustive checks; override any field."""
    base = dict(name=name, B=3, L=24, L_valid=24, d=16, n=4, k=2, m=6, c=3, d_ff=32, H=4, d_h=4,
                dtype="f32", act="silu", causal=False, w_std=0.3, seed=11)
    base.update(kw)
    return Workload(**base)
