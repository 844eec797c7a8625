"""Shapes and seeded draws of the synthetic workloads (no method arithmetic involved)."""
import torch

from paper_2605_16311_b200 import workloads as wlmod


def test_resnet50_shapes():
    shapes = wlmod.resnet50_shapes()
    assert len(shapes) == 54                                   # 53 convolutions + classifier
    assert sum(r * c for r, c, _ in shapes) == 25_502_912
    assert sum(r * c for r, c, n in shapes if n != "fc") == 23_454_912
    assert all((r * c) % 32 == 0 for r, c, _ in shapes)
    assert [s[:2] for s in shapes[:5]] == [(64, 147), (64, 64), (64, 576), (256, 64), (256, 64)]
    assert len({s[:2] for s in shapes}) == 21


def test_gpt2_and_llama_shapes():
    mats, plain = wlmod.gpt2_small_shapes()
    assert sum(r * c for r, c, _ in mats) == 84_934_656
    assert sum(r * c for r, c, _ in plain) == 39_403_008
    assert sum(r * c for r, c, _ in wlmod.llama7b_layer_shapes()) == 157_286_400
    c3 = wlmod.config3()
    assert c3.num_workers == 16 and c3.local_polar and c3.noise == "student_t4"


def test_draws_are_seeded_and_shaped():
    wl = wlmod.config1()
    sig = wlmod.make_signal(wl)
    g0 = wlmod.make_grads(wl, sig, 0)
    g0b = wlmod.make_grads(wl, sig, 0)
    g1 = wlmod.make_grads(wl, sig, 1)
    assert g0[0].shape == (4, 256, 256) and g0[0].dtype == torch.float32
    assert torch.equal(g0[0], g0b[0]) and not torch.equal(g0[0], g1[0])
    # signal + noise: per-worker mean over workers approaches the signal
    assert abs(float(g0[0].std()) - (2 ** 0.5) * 1e-2) < 2e-3
    w = wlmod.make_weights(wl)
    assert abs(float(w[0].std()) - 0.02) < 2e-3


def test_student_t_noise_is_heavy_tailed():
    wl = wlmod.scaled_down(wlmod.config3(), 1)
    wl.params = [wlmod.Param(64, 256, "matrix", "bf16", "x")]
    wl.num_workers = 4
    sig = wlmod.make_signal(wl)
    g = wlmod.make_grads(wl, sig, 0)[0].float() - sig[0]
    z = g / 1e-3
    kurt = float((z ** 4).mean() / (z ** 2).mean() ** 2)
    assert g.dtype == torch.float32 and kurt > 4.0            # Gaussian would give 3
