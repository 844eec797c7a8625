"""Plain float64 restatement of the SignMuon optimizer step.

TEST INFRASTRUCTURE ONLY: a slow, obviously-correct CPU implementation used to
check the CUDA path.  It follows the paper's algorithms step by step, in the
paper's order, with numpy matmul as the only library primitive.  No blocking,
fusion or reordering.  It shares no code with the CUDA path and imports nothing
from it.

Notation (the paper uses M for both the momentum and the worker count; here
`num_workers` is the worker count and `mom` the momentum buffer):

    Alg. 1  single-worker SignMuon          Alg. 2  distributed, int8 SUM all-reduce
    Alg. 3  distributed, 1-bit all-gather   Alg. 4  PolarNS (scale = fro or spectral)
    Alg. 5  PowerIter (spectral-norm estimate; the sampled start vector is an input)
    Alg. 6  bare Newton-Schulz loop          Eq. 1   majority vote
    Eq. 2   normalised update S/sqrt(mn)     App. B  packed 1-bit representation

Pins (tests/test_oracle_pins.py): SVD closed form of the K-step map, the
polar-factor error bound of the Newton-Schulz theorem, literal-vs-short-side
equality, brute-force vote counting, int8-sum vs popcount vote, the packed size
s1 = ceil(d/8) and the 32x ratio, the ResNet-50 worked example of App. B, and
the closed form of the momentum recursion; the Muon comparison step against the SVD form of its
direction and the exact polar factor in the converged band; for PowerIter: rank-one matrices
(exact after one round), the diagonal closed form, the sigma_max lower bound and
its limit against numpy's SVD, P = 0.  The end-to-end multi-step weight
trajectory has no printed example in the paper: beyond the per-stage pins it is
"parity unpinned".
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np

__all__ = [
    "OracleConfig", "ParamSpec", "OracleState",
    "momentum_update", "frobenius_norm", "power_iter", "newton_schulz", "polar_ns",
    "polar_ns_short_side", "sign_pm1", "encode_bits", "decode_bits",
    "pack_bits", "unpack_bits", "bytes_to_words", "words_to_bytes",
    "majority_vote_sum", "majority_vote_popcount", "local_polar",
    "apply_update", "payload_bytes", "round_to_bf16", "init_state", "step",
    "step_param", "StepTrace", "muon_step_param",
]


# --------------------------------------------------------------------------- #
# configuration / state containers (no arithmetic)
# --------------------------------------------------------------------------- #
@dataclass
class ParamSpec:
    rows: int
    cols: int
    kind: str = "matrix"          # "matrix": Newton-Schulz path; "plain": plain sign update
    weight_dtype: str = "f32"     # "f32" or "bf16" (storage type of W)


@dataclass
class OracleConfig:
    num_workers: int
    momentum: float = 0.9          # beta (Alg. 1 input)
    lr: float = 1e-3               # eta
    ns_steps: int = 5              # K
    local_polar: bool = False      # optional polar(S_bar) step (Sec. 3, "Sign-Muon update")
    weight_decay: float = 0.0      # lambda
    eps: float = 1e-12             # epsilon of Alg. 4
    update_scale: int = 0          # 0: W -= eta*S (Alg. 2); 1: W -= eta*S/sqrt(rc) (Eq. 2)
    ns_scale: str = "fro"          # Alg. 4 scale: "fro" or "spectral" (the workers' PolarNS; the local polar
                                   # step keeps "fro": ||S_bar||_F = sqrt(rc) needs no sampled vector)
    power_iters: int = 2           # P of Alg. 5 (the paper's experiments fix 2)


@dataclass
class OracleState:
    mom: List[np.ndarray] = field(default_factory=list)   # per param: [num_workers, rows, cols] float64


@dataclass
class StepTrace:
    """Intermediate results of one parameter's step, kept for staged parity tests."""
    mom: np.ndarray                       # [M, r, c] momentum after the update
    polar: Optional[np.ndarray]           # [M, r, c] U = PolarNS(mom) (matrix params) or mom (plain)
    bits: np.ndarray                      # [M, d] uint8 0/1, encode_bits(U)
    vote_bits: np.ndarray                 # [d] uint8 0/1
    direction: np.ndarray                 # [r, c] float64 D
    new_weight: np.ndarray                # [r, c] float64 W - eta D


# --------------------------------------------------------------------------- #
# Alg. 1 / Alg. 2: weight decay and momentum
# --------------------------------------------------------------------------- #
def momentum_update(mom, grad, weight, beta, weight_decay):
    """G~ = G + lambda W ;  Mom <- beta Mom + (1 - beta) G~   (Alg. 2, per worker)."""
    mom = np.asarray(mom, dtype=np.float64)
    grad = np.asarray(grad, dtype=np.float64)
    weight = np.asarray(weight, dtype=np.float64)
    g_tilde = grad + weight_decay * weight
    return beta * mom + (1.0 - beta) * g_tilde


# --------------------------------------------------------------------------- #
# Alg. 4 (PolarNS, scale = fro) and Alg. 6 (bare loop)
# --------------------------------------------------------------------------- #
def frobenius_norm(x):
    x = np.asarray(x, dtype=np.float64)
    return math.sqrt(float(np.sum(x * x)))


def power_iter(x, num_rounds, eps, v0):
    """Alg. 5: estimate of ||X||_op by `num_rounds` rounds of power iteration on X^T X.

    v0 is the "sampled" start vector of length c (an input here, so that runs are reproducible):
        v <- v0 / (||v0|| + eps)
        repeat P times:  u <- X v,  u <- u / (||u|| + eps);  v <- X^T u,  v <- v / (||v|| + eps)
        return ||X v||
    """
    x = np.asarray(x, dtype=np.float64)
    v = np.asarray(v0, dtype=np.float64).reshape(-1)
    v = v / (math.sqrt(float(np.sum(v * v))) + eps)
    for _ in range(num_rounds):
        u = x @ v
        u = u / (math.sqrt(float(np.sum(u * u))) + eps)
        v = x.T @ u
        v = v / (math.sqrt(float(np.sum(v * v))) + eps)
    w = x @ v
    return math.sqrt(float(np.sum(w * w)))


def newton_schulz(y0, num_iters):
    """Alg. 6: Y_{k+1} = 1/2 Y_k (3 I - Y_k^T Y_k), K times, I the c x c identity."""
    y = np.array(y0, dtype=np.float64, copy=True)
    c = y.shape[1]
    eye = np.eye(c, dtype=np.float64)
    for _ in range(num_iters):
        y = 0.5 * (y @ (3.0 * eye - y.T @ y))
    return y


def polar_ns(x, num_iters, eps=1e-12, sigma=None):
    """Alg. 4: sigma = ||X||_F (scale = fro; the default) or the caller's PowerIter estimate (scale =
    spectral, passed as `sigma`); Y = X / max(sigma, eps); K Newton-Schulz steps."""
    x = np.asarray(x, dtype=np.float64)
    if sigma is None:
        sigma = frobenius_norm(x)
    y = x / max(sigma, eps)
    return newton_schulz(y, num_iters)


def polar_ns_short_side(x, num_iters, eps=1e-12, sigma=None):
    """Same map as polar_ns, with the Gram matrix taken on the shorter side.

    For r < c,  Y (3 I_c - Y^T Y) = (3 I_r - Y Y^T) Y, so the iteration may use the
    r x r Gram matrix.  Only a cheaper route for large wide matrices; its equality
    with the literal form is itself a test.
    """
    x = np.asarray(x, dtype=np.float64)
    r, c = x.shape
    if r >= c:
        return polar_ns(x, num_iters, eps, sigma)
    if sigma is None:
        sigma = frobenius_norm(x)
    y = x / max(sigma, eps)
    eye = np.eye(r, dtype=np.float64)
    for _ in range(num_iters):
        y = 0.5 * ((3.0 * eye - y @ y.T) @ y)
    return y


# --------------------------------------------------------------------------- #
# sign, 1-bit encoding and packing (Alg. 3 note; App. B "Packed 1-bit representation")
# --------------------------------------------------------------------------- #
def sign_pm1(u):
    """Entrywise sign with the algorithmic convention  x >= 0 -> +1,  x < 0 -> -1.

    -0.0 compares >= 0 and maps to +1; NaN fails the comparison and maps to -1.
    """
    u = np.asarray(u)
    return np.where(u >= 0, np.int8(1), np.int8(-1)).astype(np.int8)


def encode_bits(u):
    """Encoding of Alg. 3:  >= 0 -> 1,  < 0 -> 0."""
    return (np.asarray(u) >= 0).astype(np.uint8)


def decode_bits(bits):
    """Decoding of Alg. 3:  0 -> -1,  1 -> +1."""
    return (2 * np.asarray(bits, dtype=np.int8) - 1).astype(np.int8)


def payload_bytes(d, bits_per_entry=1):
    """s = ceil(b d / 8) bytes (Sec. 4 "Distributed Communication Complexity"; App. B s_1)."""
    return (bits_per_entry * d + 7) // 8


def pack_bits(bits):
    """Flat 0/1 array -> byte array of ceil(d/8) bytes, 8 signs per byte.

    Entry i goes to bit (i mod 8) of byte (i div 8), least-significant bit first;
    the unused high bits of the last byte are 0.
    """
    bits = np.asarray(bits, dtype=np.uint8).reshape(-1)
    d = bits.size
    out = np.zeros(payload_bytes(d), dtype=np.uint8)
    for k in range(8):
        chunk = bits[k::8]
        out[: chunk.size] |= (chunk << k).astype(np.uint8)
    return out


def unpack_bits(packed, d):
    packed = np.asarray(packed, dtype=np.uint8).reshape(-1)
    idx = np.arange(d)
    return ((packed[idx >> 3] >> (idx & 7).astype(np.uint8)) & 1).astype(np.uint8)


def bytes_to_words(packed):
    """Little-endian view of the byte payload as uint32 words (zero-padded to 4 bytes)."""
    packed = np.asarray(packed, dtype=np.uint8).reshape(-1)
    pad = (-packed.size) % 4
    if pad:
        packed = np.concatenate([packed, np.zeros(pad, dtype=np.uint8)])
    return packed.view("<u4").copy()


def words_to_bytes(words, d):
    words = np.ascontiguousarray(np.asarray(words, dtype="<u4"))
    return words.view(np.uint8)[: payload_bytes(d)].copy()


# --------------------------------------------------------------------------- #
# majority vote: Eq. 1 / Alg. 2 (integer sum) and App. B (2c - M from bits)
# --------------------------------------------------------------------------- #
def majority_vote_sum(signs):
    """Alg. 2: sum_signs = sum_m S^(m) in integers; S_bar = sign(sum_signs), ties -> +1."""
    signs = np.asarray(signs, dtype=np.int64)          # [M, ...], entries +-1
    total = signs.sum(axis=0)
    return np.where(total >= 0, np.int8(1), np.int8(-1)).astype(np.int8)


def majority_vote_popcount(packed_per_worker, d):
    """App. B: c_i = sum_m b_i^(m); signed sum = 2 c_i - M; S_bar_i = sign(2 c_i - M), ties -> +1.

    Input: one packed byte array per worker.  Output: vote as 0/1 bits (1 <-> +1).
    """
    num_workers = len(packed_per_worker)
    count = np.zeros(d, dtype=np.int64)
    for buf in packed_per_worker:
        count += unpack_bits(buf, d)
    return ((2 * count - num_workers) >= 0).astype(np.uint8)


# --------------------------------------------------------------------------- #
# optional local polar step and the weight update
# --------------------------------------------------------------------------- #
def local_polar(vote_pm1, num_iters, eps=1e-12, short_side=False):
    """D = PolarNS(S_bar; K, eps, fro): the polar step applied locally to the shared vote."""
    fn = polar_ns_short_side if short_side else polar_ns
    return fn(np.asarray(vote_pm1, dtype=np.float64), num_iters, eps)


def apply_update(weight, direction, lr):
    """W <- W - eta D (Alg. 1/2/3 last line), in float64."""
    return np.asarray(weight, dtype=np.float64) - lr * np.asarray(direction, dtype=np.float64)


def round_to_bf16(x):
    """Round float64 values to the nearest bfloat16 (ties to even); result held in float32.

    Goes through float32 and repairs the double rounding: when the float32 value sits
    exactly on a bfloat16 tie, the direction is taken from the float64 value.
    """
    x = np.asarray(x, dtype=np.float64)
    f32 = x.astype(np.float32)
    bits = f32.view(np.uint32).astype(np.uint64)
    low = bits & 0xFFFF
    base = bits & ~np.uint64(0xFFFF)
    up = base + np.uint64(0x10000)
    mag64 = np.abs(x)
    mag32 = np.abs(f32.astype(np.float64))
    tie = low == 0x8000
    lsb_odd = ((bits >> np.uint64(16)) & np.uint64(1)) == 1
    round_up = np.where(tie, np.where(mag64 > mag32, True, np.where(mag64 < mag32, False, lsb_odd)),
                        low > 0x8000)
    out = np.where(round_up, up, base).astype(np.uint32)
    res = out.view(np.float32).reshape(x.shape)
    # NaN / inf pass through
    special = ~np.isfinite(f32)
    return np.where(special, f32, res).astype(np.float32)


# --------------------------------------------------------------------------- #
# one full step
# --------------------------------------------------------------------------- #
def init_state(params: Sequence[ParamSpec], cfg: OracleConfig) -> OracleState:
    """Mom_0^(m) = 0 for every worker (Alg. 2 initialisation)."""
    return OracleState(mom=[np.zeros((cfg.num_workers, p.rows, p.cols), dtype=np.float64) for p in params])


def step_param(spec: ParamSpec, cfg: OracleConfig, mom, weight, grads, lr=None,
               short_side=False, vote_bits_override=None, power_start=None) -> StepTrace:
    """One SignMuon step for one parameter block.

    mom    [M, r, c] float64 momentum of every worker (input state)
    weight [r, c]    current weights (any float dtype; widened to float64)
    grads  [M, r, c] one gradient per worker
    vote_bits_override: if given (flat 0/1 array of d entries), stages after the vote
        use these bits instead of the oracle's own (staged parity: feed the oracle the
        vote another implementation produced).
    power_start: [M, c] start vectors of PowerIter (needed when cfg.ns_scale == "spectral").
    """
    lr = cfg.lr if lr is None else lr
    M = cfg.num_workers
    r, c = spec.rows, spec.cols
    d = r * c
    weight64 = np.asarray(weight, dtype=np.float64).reshape(r, c)
    grads = np.asarray(grads, dtype=np.float64).reshape(M, r, c)
    ns = polar_ns_short_side if short_side else polar_ns

    new_mom = np.empty((M, r, c), dtype=np.float64)
    polar = np.empty((M, r, c), dtype=np.float64)
    bits = np.empty((M, d), dtype=np.uint8)
    packed = []
    for m in range(M):                                     # "each worker m independently"
        new_mom[m] = momentum_update(mom[m], grads[m], weight64, cfg.momentum, cfg.weight_decay)
        if spec.kind == "matrix":
            sigma = None
            if cfg.ns_scale == "spectral":
                sigma = power_iter(new_mom[m], cfg.power_iters, cfg.eps, np.asarray(power_start)[m])
            polar[m] = ns(new_mom[m], cfg.ns_steps, cfg.eps, sigma)   # U = PolarNS(Mom)
        else:
            polar[m] = new_mom[m]                              # vector-like params: sign of the momentum
        bits[m] = encode_bits(polar[m]).reshape(-1)            # S = sign(U), encoded
        packed.append(pack_bits(bits[m]))                      # B = PackBits(S)

    vote_bits = majority_vote_popcount(packed, d)              # all-gather + local vote
    if vote_bits_override is not None:
        vote_bits = np.asarray(vote_bits_override, dtype=np.uint8).reshape(-1)[:d]
    vote_pm1 = decode_bits(vote_bits).reshape(r, c).astype(np.float64)

    if spec.kind == "matrix" and cfg.local_polar:
        direction = local_polar(vote_pm1, cfg.ns_steps, cfg.eps, short_side=short_side)
    elif cfg.update_scale == 1:
        direction = vote_pm1 / math.sqrt(r * c)                # Eq. 2
    else:
        direction = vote_pm1                                   # Alg. 2 as printed
    new_weight = apply_update(weight64, direction, lr)
    return StepTrace(mom=new_mom, polar=polar, bits=bits, vote_bits=vote_bits,
                     direction=direction, new_weight=new_weight)


def muon_step_param(spec: ParamSpec, cfg: OracleConfig, mom, weight, grads, lr=None, short_side=False):
    """Full-precision Muon, the comparison optimizer of Sec. 5.1: Alg. 1 without the sign line.

    Data-parallel form with float gradient averaging (the float32 all-reduce that App. B compares against):
        G = mean_m G^(m);  G~ = G + lambda W;  Mom <- beta Mom + (1 - beta) G~      (one momentum, [r, c])
        U = PolarNS(Mom; K, eps, fro);  W <- W - eta U
    Returns (new momentum, U, new weight), all float64.  Plain ("vector-like") parameters have no polar factor:
    they keep the sign update of step_param and are not handled here.
    """
    if spec.kind != "matrix":
        raise ValueError("muon_step_param handles matrix parameters only")
    lr = cfg.lr if lr is None else lr
    r, c = spec.rows, spec.cols
    weight64 = np.asarray(weight, dtype=np.float64).reshape(r, c)
    grads = np.asarray(grads, dtype=np.float64).reshape(cfg.num_workers, r, c)
    g_mean = grads.sum(axis=0) / cfg.num_workers
    new_mom = momentum_update(np.asarray(mom, dtype=np.float64).reshape(r, c), g_mean, weight64, cfg.momentum,
                              cfg.weight_decay)
    ns = polar_ns_short_side if short_side else polar_ns
    u = ns(new_mom, cfg.ns_steps, cfg.eps)
    return new_mom, u, apply_update(weight64, u, lr)


def step(params: Sequence[ParamSpec], cfg: OracleConfig, state: OracleState, weights, grads,
         lr=None, short_side=False, power_starts=None):
    """One optimizer step over all parameter blocks.

    weights: list of [r, c] arrays; grads: list of [M, r, c] arrays.  Returns
    (new_weights_float64, traces) and updates state.mom in place.
    """
    new_weights, traces = [], []
    for p, spec in enumerate(params):
        tr = step_param(spec, cfg, state.mom[p], weights[p], grads[p], lr=lr, short_side=short_side,
                        power_start=None if power_starts is None else power_starts[p])
        state.mom[p] = tr.mom
        new_weights.append(tr.new_weight)
        traces.append(tr)
    return new_weights, traces
