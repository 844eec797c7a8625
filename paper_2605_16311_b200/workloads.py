"""Seeded synthetic workloads for the SignMuon optimizer step.

This module only describes parameter shapes and draws random inputs.  It holds
none of the method's arithmetic and is the one module that both the CUDA path's
tests/benchmark and the CPU oracle's tests may use.

The five workloads follow the shapes of the paper's experiments (ResNet-50 on
CIFAR-10, a GPT-2-style transformer) and stand in for them: no dataset or trained
model is involved, gradients are a fixed seeded "signal" shared by all workers plus
fresh seeded per-worker noise every step.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Tuple

import torch

BASE_SEED = 1337  # the seed the paper fixes for its language-model runs (Sec. 5.3, training configuration)


@dataclass(frozen=True)
class Param:
    rows: int
    cols: int
    kind: str = "matrix"         # "matrix" -> Newton-Schulz path, "plain" -> plain sign update
    dtype: str = "f32"           # storage type of weights and gradients: "f32" | "bf16"
    name: str = ""

    @property
    def numel(self) -> int:
        return self.rows * self.cols


@dataclass
class Workload:
    name: str
    params: List[Param]
    num_workers: int
    momentum: float = 0.9
    lr: float = 1e-3
    ns_steps: int = 5
    local_polar: bool = False
    steps: int = 10
    signal_std: float = 1e-3
    noise_std: float = 3e-3
    noise: str = "gauss"          # "gauss" | "student_t4"
    weight_std: float = 0.02
    config_id: int = 0
    extra: dict = field(default_factory=dict)

    @property
    def numel(self) -> int:
        return sum(p.numel for p in self.params)


# --------------------------------------------------------------------------- #
# shapes
# --------------------------------------------------------------------------- #
def resnet50_shapes() -> List[Tuple[int, int, str]]:
    """All 53 convolutions (out x in*kh*kw) and the 1000 x 2048 classifier of ResNet-50."""
    shapes = [(64, 3 * 7 * 7, "stem")]
    inplanes = 64
    for stage, (width, blocks) in enumerate(zip((64, 128, 256, 512), (3, 4, 6, 3))):
        for b in range(blocks):
            tag = f"s{stage}b{b}"
            shapes.append((width, inplanes, tag + ".conv1"))
            shapes.append((width, width * 9, tag + ".conv2"))
            shapes.append((width * 4, width, tag + ".conv3"))
            if b == 0:
                shapes.append((width * 4, inplanes, tag + ".down"))
            inplanes = width * 4
    shapes.append((1000, 2048, "fc"))
    return shapes


def gpt2_small_shapes():
    mats, plain = [], []
    for layer in range(12):
        mats += [(768, 2304, f"h{layer}.qkv"), (768, 768, f"h{layer}.attn_proj"),
                 (768, 3072, f"h{layer}.mlp_fc"), (3072, 768, f"h{layer}.mlp_proj")]
    plain += [(50257, 768, "wte"), (1024, 768, "wpe")]
    plain += [(1, 768, f"ln{i}") for i in range(25)]
    return mats, plain


def llama7b_layer_shapes():
    return [(4096, 4096, "q"), (4096, 4096, "k"), (4096, 4096, "v"), (4096, 4096, "o"),
            (4096, 11008, "mlp_up"), (11008, 4096, "mlp_down")]


# --------------------------------------------------------------------------- #
# the five configurations
# --------------------------------------------------------------------------- #
def config1() -> Workload:
    return Workload("c1_single_256", [Param(256, 256, "matrix", "f32", "w")], num_workers=4,
                    momentum=0.9, lr=0.02, ns_steps=5, local_polar=True, steps=10,
                    signal_std=1e-2, noise_std=1e-2, config_id=1)


def config2() -> Workload:
    ps = [Param(r, c, "matrix", "f32", n) for (r, c, n) in resnet50_shapes()]
    return Workload("c2_resnet50", ps, num_workers=4, lr=1e-3, ns_steps=5, local_polar=False,
                    steps=100, signal_std=1e-3, noise_std=3e-3, config_id=2)


def config3() -> Workload:
    mats, plain = gpt2_small_shapes()
    ps = [Param(r, c, "matrix", "bf16", n) for (r, c, n) in mats]
    ps += [Param(r, c, "plain", "bf16", n) for (r, c, n) in plain]
    return Workload("c3_gpt2_small", ps, num_workers=16, lr=1e-3, ns_steps=5, local_polar=True,
                    steps=100, signal_std=5e-4, noise_std=1e-3, noise="student_t4", config_id=3)


def config4(local_polar: bool = True) -> Workload:
    ps = [Param(r, c, "matrix", "bf16", n) for (r, c, n) in llama7b_layer_shapes()]
    return Workload("c4_llama7b_layer" + ("" if local_polar else "_nolp"), ps, num_workers=8, lr=1e-3,
                    ns_steps=5, local_polar=local_polar, steps=20, signal_std=1e-4, noise_std=5e-4,
                    config_id=4)


def sweep_shapes() -> List[Tuple[int, int]]:
    sq = [(n, n) for n in (512, 1024, 2048, 4096, 8192)]
    rect = [(512, 2048), (1024, 4096), (2048, 8192), (2048, 512), (4096, 1024), (8192, 2048)]
    return sq + rect


def config5(rows: int, cols: int, num_workers: int, ns_steps: int = 5, local_polar: bool = False) -> Workload:
    return Workload(f"c5_sweep_{rows}x{cols}_M{num_workers}_K{ns_steps}" + ("_lp" if local_polar else ""),
                    [Param(rows, cols, "matrix", "bf16", "w")], num_workers=num_workers, lr=1e-3,
                    ns_steps=ns_steps, local_polar=local_polar, steps=3, signal_std=1.0, noise_std=1.0,
                    weight_std=0.02, config_id=5)


def scaled_down(wl: Workload, max_params: int) -> Workload:
    """A prefix of a workload's parameter list (same hyper-parameters), for quick checks."""
    import copy
    out = copy.copy(wl)
    out.params = list(wl.params[:max_params])
    out.name = wl.name + f"_first{max_params}"
    return out


def by_name(name: str) -> Workload:
    table = {"c1": config1, "c2": config2, "c3": config3, "c4": config4,
             "c4_nolp": lambda: config4(False)}
    if name in table:
        return table[name]()
    if name in ("c3_plain", "c3_matrix"):   # the plain-sign / Newton-Schulz halves of config 3 (profiling cases)
        wl = config3()
        kind = "plain" if name == "c3_plain" else "matrix"
        wl.params = [p for p in wl.params if p.kind == kind]
        wl.name = name
        return wl
    if name in ("c2_short256", "c2_long"):   # the ResNet-50 matrices with a short side <= 256 / above (profiling cases)
        wl = config2()
        small = name == "c2_short256"
        wl.params = [p for p in wl.params if (min(p.rows, p.cols) <= 256) == small]
        wl.name = name
        return wl
    if name.startswith("c5:") or name.startswith("c5lp:"):           # c5:ROWSxCOLS:M[:K]; c5lp: local polar step on
        parts = name.split(":")
        r, c = (int(v) for v in parts[1].split("x"))
        m = int(parts[2])
        k = int(parts[3]) if len(parts) > 3 else 5
        return config5(r, c, m, k, local_polar=parts[0] == "c5lp")
    raise KeyError(name)


# --------------------------------------------------------------------------- #
# seeded draws
# --------------------------------------------------------------------------- #
_TORCH_DTYPE = {"f32": torch.float32, "bf16": torch.bfloat16}


def torch_dtype(name: str) -> torch.dtype:
    return _TORCH_DTYPE[name]


def _generator(device, *key: int) -> torch.Generator:
    seed = BASE_SEED
    for k in key:                       # simple reproducible key mixing (inputs only)
        seed = (seed * 1000003 + int(k) + 0x9E3779B9) % (2 ** 62)
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def make_weights(wl: Workload, device="cpu") -> List[torch.Tensor]:
    """W_0 ~ N(0, weight_std) per parameter, in the parameter's storage dtype."""
    out = []
    for p_idx, p in enumerate(wl.params):
        g = _generator(device, wl.config_id, 101, p_idx)
        w = torch.randn((p.rows, p.cols), generator=g, device=device, dtype=torch.float32) * wl.weight_std
        out.append(w.to(torch_dtype(p.dtype)).contiguous())
    return out


def make_signal(wl: Workload, device="cpu") -> List[torch.Tensor]:
    """The shared gradient signal G, fixed for the whole run (float32)."""
    out = []
    for p_idx, p in enumerate(wl.params):
        g = _generator(device, wl.config_id, 202, p_idx)
        out.append(torch.randn((p.rows, p.cols), generator=g, device=device, dtype=torch.float32)
                   * wl.signal_std)
    return out


def make_grads(wl: Workload, signal: List[torch.Tensor], step: int, device="cpu",
               out: Optional[List[torch.Tensor]] = None) -> List[torch.Tensor]:
    """Per-worker gradients G_m = G + E_m for one step: list of [M, rows, cols] tensors.

    Noise is redrawn from (config, step, parameter); Gaussian or Student-t with 4 degrees
    of freedom (a standard normal over sqrt(chi2_4 / 4)), scaled by noise_std.
    """
    res = []
    M = wl.num_workers
    for p_idx, p in enumerate(wl.params):
        g = _generator(device, wl.config_id, 303, step, p_idx)
        shape = (M, p.rows, p.cols)
        e = torch.randn(shape, generator=g, device=device, dtype=torch.float32)
        if wl.noise == "student_t4":
            v = torch.zeros(shape, device=device, dtype=torch.float32)
            for _ in range(4):
                z = torch.randn(shape, generator=g, device=device, dtype=torch.float32)
                v.addcmul_(z, z)
            e = e / torch.sqrt(v / 4.0)
            del v, z
        e.mul_(wl.noise_std).add_(signal[p_idx].unsqueeze(0))
        t = e.to(torch_dtype(p.dtype)).contiguous()
        if out is not None:
            out[p_idx].copy_(t)
            t = out[p_idx]
        res.append(t)
    return res


def make_power_start(wl: Workload, step: int, device="cpu") -> List[Optional[torch.Tensor]]:
    """Start vectors of the power iteration (the method "samples" them: here seeded standard normals),
    one [num_workers, cols] float32 tensor per matrix parameter, None for plain parameters."""
    out: List[Optional[torch.Tensor]] = []
    for p_idx, p in enumerate(wl.params):
        if p.kind != "matrix":
            out.append(None)
            continue
        g = _generator(device, wl.config_id, 404, step, p_idx)
        out.append(torch.randn((wl.num_workers, p.cols), generator=g, device=device, dtype=torch.float32))
    return out
