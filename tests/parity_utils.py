"""Staged GPU-vs-oracle comparison of one SignMuon step (used by the -m gpu tests and the smoke check).

Every stage feeds the oracle what the GPU produced at the previous stage, so each tolerance
covers one stage only:
  momentum     fp32 recursion vs float64:                     max |diff| <= 2e-6 max|Mom|
  norm         1/max(sigma, eps) vs float64:                  relative 1e-5 (sigma = Frobenius norm, or the
               power-iteration estimate of Alg. 5 from the same start vectors: relative 2e-5)
  polar (NS)   bf16 tensor-core iteration vs float64 Alg. 4:  relative Frobenius error <= 2e-2
  sign bits    >= 99.9 % equal, every mismatch where |oracle U| < 1e-3 RMS(U) (both scales)
  pack / vote / vote->update: bit-exact given the GPU's own bits
  update       fp32 weights: 1e-6 relative to max(|W|, |W'|, eta |D|); bf16 weights: the neighbouring bf16 only where the exact
               value is within 1e-6 relative of a rounding tie; local polar: direction within 2e-2
               relative Frobenius error of the oracle's PolarNS of the GPU's vote
"""
from __future__ import annotations

import math
from typing import List, Optional, Sequence

import numpy as np
import torch

import oracle as O
from paper_2605_16311_b200 import binding as B
from paper_2605_16311_b200 import workloads as wlmod


def make_optimizer(wl, flags=B.FLAG_KEEP_POLAR, **kw) -> B.SignMuon:
    kw.setdefault("ns_scale", wl.extra.get("ns_scale", "fro"))
    kw.setdefault("power_iters", wl.extra.get("power_iters", 2))
    return B.SignMuon(wl.params, wl.num_workers, momentum=wl.momentum, lr=wl.lr, ns_steps=wl.ns_steps,
                      local_polar=wl.local_polar, flags=flags, **kw)


def _np64(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


def check_param_step(opt: B.SignMuon, wl, p_idx: int, w_before: torch.Tensor, w_after: torch.Tensor,
                     grads: torch.Tensor, mom_before: Optional[np.ndarray], lr: float, weight_decay: float = 0.0,
                     check_polar: bool = True, report: Optional[dict] = None, power_start=None, power_iters: int = 2,
                     ns_workers: Optional[Sequence[int]] = None, have_polar: bool = True):
    """Checks every stage of parameter p_idx for the step just run. Returns the oracle momentum
    (float64, [M, r, c]) evolved from `mom_before` (None = zeros).  `ns_workers` restricts the Newton-Schulz
    comparison (the costly part of the oracle) to those workers; every other stage covers all workers.
    `have_polar` = False: the context was created without FLAG_KEEP_POLAR (the configuration a caller and the
    benchmark run), so Y_K of a parameter whose sign bits are packed in the last epilogue is never stored: its
    value comparison is skipped, the sign-bit comparison with the oracle stays."""
    p = wl.params[p_idx]
    M, r, c, d = wl.num_workers, p.rows, p.cols, p.rows * p.cols
    K = wl.ns_steps
    g64 = _np64(grads).reshape(M, r, c)
    w0 = _np64(w_before).reshape(r, c)
    if mom_before is None:
        mom_before = np.zeros((M, r, c))
    rep = report if report is not None else {}

    # ---- momentum
    mom_or = np.stack([O.momentum_update(mom_before[m], g64[m], w0, wl.momentum, weight_decay) for m in range(M)])
    mom_gpu = np.stack([_np64(opt.tap(B.TAP_MOMENTUM, p_idx, m)) for m in range(M)])
    err = np.max(np.abs(mom_gpu - mom_or)) / max(np.max(np.abs(mom_or)), 1e-300)
    rep["momentum_relmax"] = max(rep.get("momentum_relmax", 0.0), float(err))
    assert err <= 2e-6, f"momentum mismatch {err} (param {p_idx})"

    gpu_bits = np.stack([O.unpack_bits(opt.tap(B.TAP_WORKER_BITS, p_idx, m).cpu().numpy(), d) for m in range(M)])
    n_words = (d + 31) // 32
    for m in range(M):
        words = opt.tap(B.TAP_WORKER_BITS, p_idx, m).cpu().numpy()
        assert words.size == 4 * n_words
        if d % 32:   # pad bits are zero
            last = int(np.frombuffer(words[-4:].tobytes(), dtype="<u4")[0])
            assert last >> (d % 32) == 0

    if p.kind == "matrix":
        for m in (range(M) if ns_workers is None else ns_workers):
            # ---- norm
            scales = opt.tap(B.TAP_NORM, p_idx, m).cpu().numpy().astype(np.float64)
            if power_start is None:
                sigma_arg = None
                sigma = max(O.frobenius_norm(mom_gpu[m]), 1e-12)
                assert abs(scales[1] * sigma - 1.0) <= 1e-5 and abs(scales[0] * sigma * sigma - 1.0) <= 2e-5
            else:   # scale = spectral: PowerIter on the GPU's own momentum from the same start vector
                sigma_arg = O.power_iter(mom_gpu[m], power_iters, 1e-12, _np64(power_start[m]))
                sigma = max(sigma_arg, 1e-12)
                rep["sigma_rel"] = max(rep.get("sigma_rel", 0.0), abs(scales[1] * sigma - 1.0))
                assert abs(scales[1] * sigma - 1.0) <= 2e-5 and abs(scales[0] * sigma * sigma - 1.0) <= 4e-5
                sigma_arg = 1.0 / float(scales[1])      # staged: Newton-Schulz is checked from the GPU's own scale
            # ---- Newton-Schulz on the GPU's own momentum
            if not check_polar:
                continue
            u_or = O.polar_ns_short_side(mom_gpu[m], K, 1e-12, sigma_arg)
            rms = math.sqrt(float(np.mean(u_or ** 2)))
            if K > 0 and (have_polar or c % 32 != 0):      # rows that do not hold whole words keep Y_K for the pack kernel
                u_gpu = _np64(opt.tap(B.TAP_POLAR, p_idx, m))
                rel = np.linalg.norm(u_gpu - u_or) / np.linalg.norm(u_or)
                rep["polar_relfro"] = max(rep.get("polar_relfro", 0.0), float(rel))
                assert rel <= 2e-2, f"NS output off by {rel} (param {p_idx}, worker {m})"
                # pack is bit-exact w.r.t. the GPU's own values
                assert np.array_equal(O.encode_bits(u_gpu).reshape(-1), gpu_bits[m]), "pack != sign of GPU polar"
            or_bits = O.encode_bits(u_or).reshape(-1)
            mism = or_bits != gpu_bits[m]
            frac = 1.0 - mism.mean()
            rep["sign_match_min"] = min(rep.get("sign_match_min", 1.0), float(frac))
            assert frac >= 0.999, f"sign agreement {frac}"
            if mism.any():
                worst = np.max(np.abs(u_or.reshape(-1)[mism]))
                rep["sign_mismatch_worst_over_rms"] = max(rep.get("sign_mismatch_worst_over_rms", 0.0),
                                                          float(worst / rms))
                assert worst < 1e-3 * rms, f"sign mismatch at |u|={worst} vs rms {rms}"
    else:
        for m in range(M):
            assert np.array_equal(O.encode_bits(mom_gpu[m]).reshape(-1), gpu_bits[m])

    # ---- vote from the GPU's own payload, bit-exact
    packed = [O.pack_bits(gpu_bits[m]) for m in range(M)]
    for m in range(M):
        assert np.array_equal(O.words_to_bytes(O.bytes_to_words(packed[m]), d),
                              opt.tap(B.TAP_WORKER_BITS, p_idx, m).cpu().numpy()[: (d + 7) // 8])
    vote_or = O.majority_vote_popcount(packed, d)
    vote_gpu = O.unpack_bits(opt.tap(B.TAP_VOTE_BITS, p_idx, 0).cpu().numpy(), d)
    assert np.array_equal(vote_or, vote_gpu), "vote differs from popcount of the GPU's own bits"
    assert np.array_equal(O.decode_bits(vote_or), O.majority_vote_sum(O.decode_bits(gpu_bits)))

    # ---- update given the GPU's vote
    s_bar = O.decode_bits(vote_gpu).reshape(r, c).astype(np.float64)
    w1_gpu = _np64(w_after).reshape(r, c)
    lp = wl.local_polar and p.kind == "matrix"
    if lp and K > 0:
        d_or = O.local_polar(s_bar, K, 1e-12, short_side=True)
    elif lp:
        d_or = s_bar / math.sqrt(r * c)
    else:
        d_or = s_bar
    w1_or = O.apply_update(w0, d_or, lr)
    if p.dtype == "f32":
        if lp and K > 0:
            d_gpu = (w0 - w1_gpu) / lr
            # weights carry ~1e-7 relative rounding: exclude it from the direction error
            noise = np.linalg.norm(np.abs(w0) * 1.2e-7 / lr)
            rel = max(np.linalg.norm(d_gpu - d_or) - noise, 0.0) / np.linalg.norm(d_or)
            rep["local_polar_relfro"] = max(rep.get("local_polar_relfro", 0.0), float(rel))
            assert rel <= 2e-2, f"local polar direction off by {rel}"
        else:
            # relative to the larger of the operands of W - eta D (the difference itself may cancel)
            scale = np.maximum(np.maximum(np.abs(w0), np.abs(w1_or)), lr * np.abs(d_or))
            rel = np.max(np.abs(w1_gpu - w1_or) / scale)
            rep["update_relmax"] = max(rep.get("update_relmax", 0.0), float(rel))
            assert rel <= 1e-6, f"weight update off: rel {rel}"
    else:
        rounded = O.round_to_bf16(w1_or).astype(np.float64)
        ulp = np.abs(rounded) * 2.0 ** -7 + 1e-40
        slack = (lr * 0.05 * np.max(np.abs(d_or))) if (lp and K > 0) else 0.0
        diff = np.abs(w1_gpu - w1_or)
        assert np.all(diff <= 0.5 * ulp * (1 + 1e-3) + slack + 1e-6 * np.abs(w1_or)), "bf16 weight update off"
        if not (lp and K > 0):
            neq = w1_gpu != rounded
            if neq.any():   # only allowed next to a rounding tie
                tie_dist = np.abs(np.abs(w1_or - rounded) - 0.5 * ulp)
                assert np.all(tie_dist[neq] <= 1e-6 * np.abs(w1_or[neq]) + 1e-3 * ulp[neq])
    return mom_or


def run_and_check(wl, steps: int, flags: int = B.FLAG_KEEP_POLAR, sample: Optional[Sequence[int]] = None,
                  device: str = "cuda:0", check_polar: bool = True, report: Optional[dict] = None,
                  ns_workers: Optional[Sequence[int]] = None, capture: Optional[dict] = None):
    """Runs `steps` optimizer steps of workload `wl` on the GPU and checks the sampled parameters
    (default: all) against the oracle after every step.  `capture` (a dict) receives the payload of every
    worker after every step and the final weights, for bit-level comparisons between two runs."""
    opt = make_optimizer(wl, flags=flags)
    weights = wlmod.make_weights(wl, device)
    signal = wlmod.make_signal(wl, device)
    sample = list(range(len(wl.params))) if sample is None else list(sample)
    mom_or = {p: None for p in sample}
    rep = report if report is not None else {}
    # (with K = 0 no scale is needed at all: the library then asks for no start vectors)
    spectral = wl.extra.get("ns_scale", "fro") == "spectral" and opt.power_start_size > 0
    for t in range(steps):
        grads = wlmod.make_grads(wl, signal, t, device)
        before = {p: weights[p].clone() for p in sample}
        starts = None
        if spectral:   # fresh start vectors every step, laid out as the library asks
            starts = wlmod.make_power_start(wl, t, device)
            flat = torch.zeros(opt.power_start_size, dtype=torch.float32, device=device)
            for p, v in enumerate(starts):
                if v is not None:
                    off, n = opt.power_start_segment(p)
                    assert n == wl.params[p].cols
                    flat[off: off + v.numel()] = v.reshape(-1)
            opt.set_power_start(flat)
        opt.step(weights, grads, wl.lr)
        torch.cuda.synchronize()
        assert opt.status() == B.OK, "device status word reports a timed-out wait"
        for p in sample:
            # the oracle momentum continues from the GPU's previous momentum (staged parity)
            mom_or[p] = check_param_step(opt, wl, p, before[p], weights[p], grads[p], mom_or[p], wl.lr,
                                         check_polar=check_polar, report=rep,
                                         power_start=None if starts is None else starts[p],
                                         power_iters=wl.extra.get("power_iters", 2), ns_workers=ns_workers,
                                         have_polar=bool(flags & B.FLAG_KEEP_POLAR))
            mom_or[p] = np.stack([_np64(opt.tap(B.TAP_MOMENTUM, p, m)) for m in range(wl.num_workers)])
        if capture is not None:
            capture.setdefault("payloads", []).append([opt.payload(m).clone() for m in range(wl.num_workers)])
    if capture is not None:
        capture["weights"] = [w.clone() for w in weights]
    opt.close()
    return rep
