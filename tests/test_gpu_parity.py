"""GPU parity tests: the CUDA path through the C ABI against the float64 oracle, stage by stage."""
import numpy as np
import pytest
import torch

from paper_2605_16311_b200 import binding as B
from paper_2605_16311_b200 import workloads as wlmod

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _lib():
    from paper_2605_16311_b200 import build as build_mod
    build_mod.build()
    assert torch.cuda.is_available()
    B.load_library()


def _wl(shapes, M, dtype="f32", K=5, local_polar=False, kinds=None, **kw):
    kinds = kinds or ["matrix"] * len(shapes)
    ps = [wlmod.Param(r, c, k, dtype, f"p{i}") for i, ((r, c), k) in enumerate(zip(shapes, kinds))]
    base = dict(momentum=0.9, lr=1e-3, ns_steps=K, local_polar=local_polar, steps=2, signal_std=1e-3,
                noise_std=3e-3, config_id=77)
    base.update(kw)
    return wlmod.Workload("t", ps, num_workers=M, **base)


def test_config1_simt_diagnostic_path():
    from parity_utils import run_and_check
    rep = run_and_check(wlmod.config1(), steps=2, flags=B.FLAG_KEEP_POLAR | B.FLAG_SIMT_GEMM)
    assert rep["sign_match_min"] >= 0.999


def test_one_cta_tile_variant_ragged_and_local_polar():
    """The 128 x 128 one-CTA shape of the tensor-core kernel (the default is CTA pairs on 256 x 256 tiles)."""
    from parity_utils import run_and_check
    flags = B.FLAG_KEEP_POLAR | B.FLAG_GEMM_1CTA
    run_and_check(_wl([(200, 328), (328, 200), (64, 147), (512, 640)], 3), steps=2, flags=flags)
    run_and_check(_wl([(200, 328), (328, 200), (256, 256)], 2, local_polar=True, lr=0.01), steps=1, flags=flags)


@pytest.mark.parametrize("P,K", [(0, 1), (1, 1), (2, 5), (3, 5), (2, 3)])
def test_spectral_scaling_power_iteration(P, K):
    """Alg. 4 with scale = spectral: sigma from P rounds of Alg. 5 on the momentum, start vectors passed in.
    With P < 2 the estimate can lie so far below the spectral norm that the cubic iteration leaves its
    basin (singular values of Y_0 above sqrt 3) and the result is decided by cancellation: those cases check
    sigma, the pack, the vote and the update, not the Newton-Schulz values."""
    from parity_utils import run_and_check
    shapes = [(200, 328), (328, 200), (64, 147), (256, 256), (1, 160)]
    wl = _wl(shapes, 3, K=K, extra={"ns_scale": "spectral", "power_iters": P})
    rep = run_and_check(wl, steps=2, check_polar=P >= 2)
    assert "sigma_rel" in rep
    print(rep)
    if P >= 2:
        wl = _wl([(128, 384), (384, 128)], 2, K=K, local_polar=True, lr=0.01,
                 extra={"ns_scale": "spectral", "power_iters": P})
        run_and_check(wl, steps=1)


def test_spectral_scaling_one_cta_variant_and_k0():
    """Split-precision products on the one-CTA tile shape, and the degenerate K = 0 (sign of the momentum)."""
    from parity_utils import run_and_check
    wl = _wl([(200, 328), (328, 200), (64, 147)], 2, extra={"ns_scale": "spectral", "power_iters": 2})
    run_and_check(wl, steps=1, flags=B.FLAG_KEEP_POLAR | B.FLAG_GEMM_1CTA)
    wl0 = _wl([(128, 384), (64, 147)], 2, K=0, extra={"ns_scale": "spectral", "power_iters": 2})
    run_and_check(wl0, steps=1)


def test_spectral_scaling_needs_start_vectors():
    wl = _wl([(64, 64)], 2, extra={"ns_scale": "spectral"})
    from parity_utils import make_optimizer
    opt = make_optimizer(wl)
    w = wlmod.make_weights(wl, "cuda:0")
    g = wlmod.make_grads(wl, wlmod.make_signal(wl, "cuda:0"), 0, "cuda:0")
    with pytest.raises(B.SignMuonError) as e:
        opt.step(w, g, 1e-3)
    assert e.value.code == -3
    opt.close()


def test_config1_ten_steps():
    from parity_utils import run_and_check
    rep = run_and_check(wlmod.config1(), steps=10)
    print(rep)


@pytest.mark.parametrize("M", [1, 2, 3, 8])
def test_ragged_shapes_wide_tall_and_stem(M):
    from parity_utils import run_and_check
    wl = _wl([(200, 328), (328, 200), (64, 147), (130, 64), (96, 96), (1, 160), (300, 1)], M)
    run_and_check(wl, steps=2)


def test_local_polar_ragged_and_eq2_scale():
    from parity_utils import run_and_check
    run_and_check(_wl([(200, 328), (328, 200), (64, 147), (256, 256)], 4, local_polar=True, lr=0.01), steps=2)


@pytest.mark.parametrize("K", [0, 1, 2, 3])
def test_ns_step_counts(K):
    from parity_utils import run_and_check
    run_and_check(_wl([(128, 384), (384, 128), (64, 147)], 2, K=K), steps=1)
    run_and_check(_wl([(128, 384), (64, 147)], 2, K=K, local_polar=True), steps=1)


def test_bf16_weights_matrix_and_plain_student_t():
    from parity_utils import run_and_check
    wl = _wl([(256, 768), (768, 256), (1000, 33), (1, 768), (515, 64)], 16, dtype="bf16", local_polar=True,
             kinds=["matrix", "matrix", "plain", "plain", "plain"], noise="student_t4", signal_std=5e-4,
             noise_std=1e-3)
    run_and_check(wl, steps=3)
    wl.local_polar = False
    run_and_check(wl, steps=2)


@pytest.mark.parametrize("M", [1, 5, 16, 32, 33, 100])
def test_vote_worker_counts(M):
    from parity_utils import run_and_check
    run_and_check(_wl([(64, 96), (40, 7)], M, K=1, kinds=["matrix", "plain"]), steps=1, check_polar=(M <= 16))


def test_resnet50_prefix_and_large_tiles():
    from parity_utils import run_and_check
    c2 = wlmod.config2()
    wl = wlmod.scaled_down(c2, 9)
    run_and_check(wl, steps=2)
    run_and_check(_wl([(512, 1152), (1024, 512)], 2), steps=1)


def test_gpt2_and_llama_like_shapes_bf16():
    from parity_utils import run_and_check
    run_and_check(_wl([(768, 2304), (3072, 768)], 2, dtype="bf16", local_polar=True, signal_std=5e-4,
                      noise_std=1e-3, noise="student_t4"), steps=1)
    run_and_check(_wl([(1024, 4096)], 2, dtype="bf16", signal_std=1e-4, noise_std=5e-4), steps=1)


def test_full_resnet50_config_sampled():
    """The benchmark's configuration at full size, parameters sampled for the oracle."""
    from parity_utils import run_and_check
    wl = wlmod.config2()
    names = [p.name for p in wl.params]
    sample = [0, 1, names.index("s0b0.conv3"), names.index("s1b0.conv2"), names.index("s2b0.down"),
              names.index("s3b2.conv2"), names.index("fc")]
    rep = run_and_check(wl, steps=2, sample=sample)
    print(rep)


@pytest.mark.parametrize("flags", [B.FLAG_KEEP_POLAR, 0])
def test_full_gpt2_config_sampled(flags):
    """Config 3 at full size (12 layers, embeddings and norm gains as plain parameters, M = 16, Student-t noise,
    local polar on): sampled parameters, Newton-Schulz compared for two of the sixteen workers; once with Y_K kept
    for the value comparison, once in the configuration the benchmark times (flags = 0)."""
    from parity_utils import run_and_check
    wl = wlmod.config3()
    names = [p.name for p in wl.params]
    sample = [names.index("h0.qkv"), names.index("h5.attn_proj"), names.index("h11.mlp_proj"), names.index("wpe"),
              names.index("ln7")]
    rep = run_and_check(wl, steps=1, sample=sample, ns_workers=[0, 15], flags=flags)
    assert rep["sign_match_min"] >= 0.999
    print(rep)


def test_full_llama_layer_config_sampled():
    """Config 4 at full size (4096 x 4096 x 4, 4096 x 11008, 11008 x 4096; M = 8; local polar on): a square and
    a rectangular matrix, Newton-Schulz compared for one worker each, plus the local polar direction."""
    from parity_utils import run_and_check
    wl = wlmod.config4()
    rep = run_and_check(wl, steps=1, sample=[1], ns_workers=[3])
    rep2 = run_and_check(wl, steps=1, sample=[5], ns_workers=[6])
    print(rep, rep2)


def test_llama_layer_without_local_polar_and_sweep_extremes():
    """Config 4 with the local polar step off (vote + update fused), and the corners of the kernel sweep:
    the largest square (8192 x 8192, K = 3) and a 1:4 rectangle with 32 workers (Newton-Schulz of the last worker)."""
    from parity_utils import run_and_check
    rep = run_and_check(wlmod.config4(False), steps=1, sample=[4], ns_workers=[0])
    rep2 = run_and_check(wlmod.config5(8192, 8192, 1, 3), steps=1)
    rep3 = run_and_check(wlmod.config5(2048, 8192, 32, 5), steps=1, ns_workers=[31])
    print(rep, rep2, rep3)


def _same_bits_and_weights(a: dict, b: dict):
    for pa, pb in zip(a["payloads"], b["payloads"]):
        for x, y in zip(pa, pb):
            assert torch.equal(x, y)
    for x, y in zip(a["weights"], b["weights"]):
        assert torch.equal(x, y)


def test_default_flags_path_against_oracle():
    """The configuration a caller (and the benchmark) runs: no FLAG_KEEP_POLAR, so the last apply epilogue
    writes payload words only and Y_K never reaches memory.  Worker sign bits against the oracle's PolarNS of
    the GPU's own momentum (>= 99.9 %, mismatches confined to |oracle| < 1e-3 RMS), vote and update from the
    GPU's own payload, and payload words + weights bit-identical to a run that also stores Y_K."""
    from parity_utils import run_and_check
    cases = [(wlmod.config1(), 3, None),
             (_wl([(200, 328), (328, 200), (64, 147), (130, 64), (96, 96), (1, 160), (300, 1)], 3), 2, None),
             (_wl([(256, 768), (768, 256), (1, 768)], 4, dtype="bf16", local_polar=True, lr=0.01,
                  kinds=["matrix", "matrix", "plain"]), 2, None)]
    c2 = wlmod.config2()
    names = [p.name for p in c2.params]
    cases.append((c2, 2, [0, 1, names.index("s0b0.conv3"), names.index("s1b0.conv2"), names.index("s2b0.down"),
                          names.index("s3b2.conv2"), names.index("fc")]))
    for wl, steps, sample in cases:
        plain, kept = {}, {}
        rep = run_and_check(wl, steps=steps, flags=0, sample=sample, capture=plain)
        assert rep["sign_match_min"] >= 0.999
        run_and_check(wl, steps=steps, flags=B.FLAG_KEEP_POLAR, sample=sample, capture=kept, check_polar=False)
        _same_bits_and_weights(plain, kept)


@pytest.mark.parametrize("K", [2, 5])
def test_gram_space_iteration_against_oracle_and_full_matrix_iteration(K):
    """Short sides up to 256 iterate in Gram space (one Gram launch, the on-chip chain, one apply launch).  Both that
    path and the per-iteration path (FLAG_NO_GRAM_SPACE) are held to the oracle's Alg. 4 at the same tolerances; their
    sign bits agree with each other wherever the oracle's value is not next to zero (both are confined to 1e-3 RMS)."""
    import numpy as np
    from parity_utils import run_and_check
    shapes = [(64, 576), (576, 64), (100, 328), (129, 520), (200, 200), (256, 1024), (1024, 256), (256, 256),
              (64, 147), (8, 64), (320, 512)]
    wl = _wl(shapes, 3, K=K)
    rep_gs, rep_full, cap_gs, cap_full = {}, {}, {}, {}
    run_and_check(wl, steps=2, report=rep_gs, capture=cap_gs)
    run_and_check(wl, steps=2, flags=B.FLAG_KEEP_POLAR | B.FLAG_NO_GRAM_SPACE, report=rep_full, capture=cap_full)
    print("gram space:", rep_gs, "\nper iteration:", rep_full)
    assert rep_gs["polar_relfro"] <= 2e-2 and rep_full["polar_relfro"] <= 2e-2
    for m in range(wl.num_workers):
        a = cap_gs["payloads"][0][m].cpu().numpy().view(np.uint8)
        b = cap_full["payloads"][0][m].cpu().numpy().view(np.uint8)
        differing = int(np.unpackbits(a ^ b).sum())
        assert differing <= 2e-3 * wl.numel
    # default flags (no stored Y_K) on the same set
    run_and_check(wl, steps=1, flags=0)


@pytest.mark.parametrize("K", [2, 5])
def test_gram_space_chain_through_memory_against_oracle_and_full_matrix_iteration(K):
    """Longer short sides iterate in Gram space as a chain of symmetric s x s products through memory (upper tiles
    computed, hi part mirrored).  Held to the oracle's Alg. 4 like the per-iteration path, on shapes with ragged
    tiles, wide and tall, and with the default flags as well."""
    import numpy as np
    from parity_utils import run_and_check
    shapes = [(512, 2048), (2048, 512), (320, 512), (300, 1000), (1000, 300), (768, 2304), (264, 4096), (520, 520)]
    wl = _wl(shapes, 3, K=K)
    # the path under test is the one taken: 2K launches for the square matrix, 2K - 1 more for the chain
    from parity_utils import make_optimizer
    opt = make_optimizer(wl, flags=0)
    assert opt.ns_launches_per_step == (4 * K - 1, 0)
    opt.close()
    opt = make_optimizer(wl, flags=B.FLAG_NO_GRAM_SPACE)
    assert opt.ns_launches_per_step == (2 * K, 0)
    opt.close()
    rep_gs, rep_full, cap_gs, cap_full = {}, {}, {}, {}
    run_and_check(wl, steps=2, report=rep_gs, capture=cap_gs)
    run_and_check(wl, steps=2, flags=B.FLAG_KEEP_POLAR | B.FLAG_NO_GRAM_SPACE, report=rep_full, capture=cap_full)
    print("gram space:", rep_gs, "\nper iteration:", rep_full)
    assert rep_gs["polar_relfro"] <= 2e-2 and rep_full["polar_relfro"] <= 2e-2
    for m in range(wl.num_workers):
        a = cap_gs["payloads"][0][m].cpu().numpy().view(np.uint8)
        b = cap_full["payloads"][0][m].cpu().numpy().view(np.uint8)
        assert int(np.unpackbits(a ^ b).sum()) <= 2e-3 * wl.numel
    run_and_check(wl, steps=1, flags=0)
    run_and_check(wl, steps=1, flags=B.FLAG_KEEP_POLAR | B.FLAG_GEMM_1CTA)


def test_local_polar_step_in_gram_space_against_oracle_and_full_matrix_iteration():
    """The local polar step also iterates in Gram space where the workers' iterations do (FP8 Gram of the vote matrix,
    the on-chip chain or the chain through memory, one apply launch that updates the weights).  Both that path and the per-iteration
    one are held to the oracle's Alg. 4 on the vote matrix; the Gram-space path, whose product with the exact +-1 matrix
    carries only the rounding of F_K, is the more accurate of the two."""
    from parity_utils import run_and_check
    shapes = [(64, 576), (576, 64), (100, 328), (200, 200), (256, 1024), (1024, 256), (64, 147), (16, 2048), (320, 512),
              (512, 2048), (1000, 300), (520, 520), (768, 2304)]
    wl = _wl(shapes, 4, local_polar=True, lr=0.01)
    rep_gs = run_and_check(wl, steps=2)
    rep_full = run_and_check(wl, steps=2, flags=B.FLAG_KEEP_POLAR | B.FLAG_NO_GRAM_SPACE)
    print("gram space:", rep_gs, "\nper iteration:", rep_full)
    assert rep_gs["local_polar_relfro"] <= 2e-3
    assert rep_full["local_polar_relfro"] <= 2e-2


def test_default_flags_path_full_llama_layer_sampled():
    """Config 4 at full size in the benchmark's launch configuration (flags = 0, local polar on)."""
    from parity_utils import run_and_check
    rep = run_and_check(wlmod.config4(), steps=1, flags=0, sample=[0, 4], ns_workers=[5])
    assert rep["sign_match_min"] >= 0.999
    print(rep)


def test_weight_decay_and_step_lr_override():
    from parity_utils import check_param_step, make_optimizer
    import numpy as np
    wl = _wl([(96, 160)], 3)
    opt = B.SignMuon(wl.params, 3, momentum=0.8, lr=123.0, ns_steps=5, weight_decay=0.05, flags=B.FLAG_KEEP_POLAR)
    wl.momentum = 0.8
    w = wlmod.make_weights(wl, "cuda:0")
    sig = wlmod.make_signal(wl, "cuda:0")
    g = wlmod.make_grads(wl, sig, 0, "cuda:0")
    before = w[0].clone()
    opt.step(w, g, 0.004)                     # per-step learning rate overrides the configured one
    torch.cuda.synchronize()
    check_param_step(opt, wl, 0, before, w[0], g[0], None, 0.004, weight_decay=0.05)
    opt.close()


def test_stage_calls_equal_one_step_and_determinism():
    wl = _wl([(256, 320), (320, 256), (64, 147), (1, 99)], 4, local_polar=True,
             kinds=["matrix", "matrix", "matrix", "plain"])
    sig = wlmod.make_signal(wl, "cuda:0")
    g = wlmod.make_grads(wl, sig, 0, "cuda:0")
    outs = []
    for mode in range(3):
        opt = B.SignMuon(wl.params, 4, lr=0.01, local_polar=True)
        w = wlmod.make_weights(wl, "cuda:0")
        if mode == 1:
            for st in (B.STAGE_MOMENTUM, B.STAGE_NS, B.STAGE_VOTE, B.STAGE_LOCAL_POLAR):
                opt.step(w, g, stages=st)
        else:
            opt.step(w, g)
        torch.cuda.synchronize()
        assert opt.status() == B.OK
        outs.append(([x.clone() for x in w], opt.payload(0).clone(), opt.payload(3).clone()))
        opt.close()
    for other in outs[1:]:
        for a, b in zip(outs[0][0], other[0]):
            assert torch.equal(a, b)                       # bit-identical weights
        assert torch.equal(outs[0][1], other[1]) and torch.equal(outs[0][2], other[2])


def test_long_contractions_are_bit_reproducible_run_to_run():
    """Two threads issue the tensor-core instructions of a tile, alternating K blocks; a token keeps them in K order,
    so the fp32 accumulation order - and every payload and weight bit - must not depend on timing.  Long contractions
    (many K blocks per tile, both operand majors, the split-precision products of a short-side matrix) over three
    fresh contexts."""
    wl = _wl([(1024, 4096), (4096, 1024), (256, 2048), (768, 768)], 3, dtype="bf16", local_polar=True, lr=0.01)
    sig = wlmod.make_signal(wl, "cuda:0")
    g = wlmod.make_grads(wl, sig, 0, "cuda:0")
    outs = []
    for _ in range(3):
        opt = B.SignMuon(wl.params, 3, lr=0.01, local_polar=True)
        w = wlmod.make_weights(wl, "cuda:0")
        for _step in range(2):
            opt.step(w, g)
        torch.cuda.synchronize()
        assert opt.status() == B.OK
        outs.append(([x.clone() for x in w], [opt.payload(m).clone() for m in range(3)]))
        opt.close()
    for other in outs[1:]:
        for a, b in zip(outs[0][0], other[0]):
            assert torch.equal(a, b)
        for a, b in zip(outs[0][1], other[1]):
            assert torch.equal(a, b)


@pytest.mark.parametrize("local_polar", [False, True])
def test_step_captured_in_a_cuda_graph_replays_bit_identically(local_polar):
    """signmuon_step only enqueues work (no allocation, no synchronisation, no upload once the pointer set is known):
    a step recorded into a CUDA graph - cluster launches, the programmatic dependent launch of the update kernel and the
    Gram-space chain included - replays to the same bits as the same steps enqueued directly."""
    wl = _wl([(256, 512), (512, 1024), (64, 147), (1, 96)], 3, local_polar=local_polar, lr=0.01,
             kinds=["matrix", "matrix", "matrix", "plain"])
    sig = wlmod.make_signal(wl, "cuda:0")
    g = wlmod.make_grads(wl, sig, 0, "cuda:0")
    eager = B.SignMuon(wl.params, 3, lr=0.01, local_polar=local_polar)
    graphed = B.SignMuon(wl.params, 3, lr=0.01, local_polar=local_polar)
    w_e = wlmod.make_weights(wl, "cuda:0")
    w_g = [x.clone() for x in w_e]
    eager.step(w_e, g)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        graphed.step(w_g, g)                       # warm-up on the capture stream: the pointer table is uploaded here
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        graphed.step(w_g, g)
    # the capture itself runs nothing: three replays against three more eager steps
    for _ in range(3):
        graph.replay()
        eager.step(w_e, g)
    torch.cuda.synchronize()
    assert eager.status() == B.OK and graphed.status() == B.OK
    for a, b in zip(w_e, w_g):
        assert torch.equal(a, b)
    for m in range(3):
        assert torch.equal(eager.payload(m), graphed.payload(m))
    eager.close(); graphed.close()


def test_bounded_wait_runs_out_and_the_context_recovers():
    """Failure detection without a fault: a one-thread kernel performs the Newton-Schulz kernels' bounded wait on
    a barrier that nothing signals, with a 1 ms limit.  The kernel returns, the status word reports the timeout,
    a new bind clears it, and the context then steps exactly like a fresh one."""
    wl = _wl([(256, 320), (64, 147)], 3, local_polar=True, lr=0.01)
    sig = wlmod.make_signal(wl, "cuda:0")
    g = wlmod.make_grads(wl, sig, 0, "cuda:0")
    opt = B.SignMuon(wl.params, 3, lr=0.01, local_polar=True)
    assert opt.status() == B.OK
    opt.selftest_wait_timeout(1_000_000)
    assert opt.status() == B.ERR_TIMEOUT
    assert opt.status() == B.ERR_TIMEOUT          # stays until the next bind
    with pytest.raises(B.SignMuonError):
        opt.selftest_wait_timeout(0)              # a limit is mandatory
    opt.rebind()
    assert opt.status() == B.OK
    opt.set_wait_limit(500_000_000)               # a shorter (still generous) limit for the real kernels
    w = wlmod.make_weights(wl, "cuda:0")
    opt.step(w, g)
    assert opt.status() == B.OK
    fresh = B.SignMuon(wl.params, 3, lr=0.01, local_polar=True)
    w2 = wlmod.make_weights(wl, "cuda:0")
    fresh.step(w2, g)
    assert fresh.status() == B.OK
    for a, b in zip(w, w2):
        assert torch.equal(a, b)
    assert torch.equal(opt.payload(1), fresh.payload(1))
    opt.close(); fresh.close()


def test_pointer_table_cache_with_more_buffer_sets_than_slots():
    """Six gradient buffer sets used in rotation (the device keeps four pointer tables) against one context
    that always sees the same buffers: identical weights and payloads after every step."""
    wl = _wl([(128, 256), (64, 147), (1, 40)], 3, kinds=["matrix", "matrix", "plain"])
    sig = wlmod.make_signal(wl, "cuda:0")
    sets = [wlmod.make_grads(wl, sig, t, "cuda:0") for t in range(6)]
    fixed = [torch.empty_like(x) for x in sets[0]]
    a, b = B.SignMuon(wl.params, 3), B.SignMuon(wl.params, 3)
    wa, wb = wlmod.make_weights(wl, "cuda:0"), wlmod.make_weights(wl, "cuda:0")
    for t in range(14):
        gs = sets[(t * 5) % 6] if t % 3 else sets[t % 6]
        a.step(wa, gs)
        for dst, src in zip(fixed, gs):
            dst.copy_(src)
        b.step(wb, fixed)
        torch.cuda.synchronize()
        for x, y in zip(wa, wb):
            assert torch.equal(x, y)
        assert torch.equal(a.payload(2), b.payload(2))
    assert a.status() == B.OK and b.status() == B.OK
    a.close(); b.close()


@pytest.mark.parametrize("dtype,M,K", [("f32", 4, 5), ("bf16", 3, 3), ("f32", 1, 1)])
def test_muon_rule_against_oracle(dtype, M, K):
    """The full-precision Muon comparison optimizer on the same kernels (one momentum of the mean gradient,
    W <- W - eta PolarNS(Mom), no sign, no vote): momentum at the momentum tolerance, update direction within 2e-2
    relative Frobenius error of the oracle's step from the GPU's own momentum; plain parameters keep the
    majority-vote sign update."""
    import oracle as O
    from parity_utils import _np64
    shapes = [(200, 328), (328, 200), (64, 147), (256, 256), (1, 160)]
    wl = _wl(shapes, M, dtype=dtype, K=K, kinds=["matrix"] * 4 + ["plain"], lr=0.01)
    opt = B.SignMuon(wl.params, M, momentum=0.9, lr=0.01, ns_steps=K, update_rule="muon", weight_decay=0.01)
    w = wlmod.make_weights(wl, "cuda:0")
    sig = wlmod.make_signal(wl, "cuda:0")
    cfg = O.OracleConfig(num_workers=M, momentum=0.9, lr=0.01, ns_steps=K, weight_decay=0.01)
    mom_prev = [np.zeros((p.rows, p.cols)) for p in wl.params[:4]]
    for t in range(2):
        g = wlmod.make_grads(wl, sig, t, "cuda:0")
        before = [x.clone() for x in w]
        opt.step(w, g)
        torch.cuda.synchronize()
        assert opt.status() == B.OK
        for p in range(4):
            spec = O.ParamSpec(wl.params[p].rows, wl.params[p].cols, "matrix", dtype)
            w0 = _np64(before[p])
            mom_or, _, _ = O.muon_step_param(spec, cfg, mom_prev[p], w0, _np64(g[p]), short_side=True)
            mom_gpu = _np64(opt.tap(B.TAP_MOMENTUM, p, 0))
            assert np.max(np.abs(mom_gpu - mom_or)) <= 2e-6 * np.max(np.abs(mom_or))
            u_or = O.polar_ns_short_side(mom_gpu, K, 1e-12)               # staged: from the GPU's own momentum
            w1 = _np64(w[p])
            if dtype == "f32":
                d_gpu = (w0 - w1) / 0.01
                noise = np.linalg.norm(np.abs(w0) * 1.2e-7 / 0.01)
                rel = max(np.linalg.norm(d_gpu - u_or) - noise, 0.0) / np.linalg.norm(u_or)
                assert rel <= 2e-2, rel
            else:
                w1_or = w0 - 0.01 * u_or
                ulp = np.abs(O.round_to_bf16(w1_or).astype(np.float64)) * 2.0 ** -7 + 1e-40
                assert np.all(np.abs(w1 - w1_or) <= 0.5 * ulp * (1 + 1e-3) + 0.01 * 0.05 * np.max(np.abs(u_or)))
            mom_prev[p] = mom_gpu
            with pytest.raises(B.SignMuonError):
                opt.tap(B.TAP_WORKER_BITS, p, 0)                          # nothing is packed for a matrix under this rule
        # the plain parameter: majority-vote sign update of its M momenta
        d = wl.params[4].numel
        packed = [opt.tap(B.TAP_WORKER_BITS, 4, m).cpu().numpy()[: (d + 7) // 8] for m in range(M)]
        vote = O.decode_bits(O.majority_vote_popcount(packed, d)).reshape(1, d).astype(np.float64)
        want = O.round_to_bf16(_np64(before[4]) - 0.01 * vote) if dtype == "bf16" else _np64(before[4]) - 0.01 * vote
        scale = np.maximum(np.maximum(np.abs(_np64(before[4])), np.abs(want)), 0.01)   # operands of W - eta S
        assert np.max(np.abs(_np64(w[4]) - want) / scale) <= 1e-6
    with pytest.raises(B.SignMuonError):
        B.SignMuon(wl.params, M, ns_steps=0, update_rule="muon")
    opt.close()


def test_muon_rule_with_the_chain_through_memory():
    """The Muon rule on a matrix large enough (one batch slot, 9.4 M entries) for its iteration to run in Gram space as
    a chain through memory, whose last apply launch then updates the weights: direction against the oracle's PolarNS of
    the GPU's own momentum."""
    import oracle as O
    from parity_utils import _np64
    K, M = 5, 2
    wl = _wl([(2048, 4608)], M, dtype="f32", K=K, lr=0.01)
    opt = B.SignMuon(wl.params, M, momentum=0.9, lr=0.01, ns_steps=K, update_rule="muon")
    assert opt.ns_launches_per_step == (2 + 2 * K - 1, 0)     # Gram, 2K - 1 chain launches, apply
    w = wlmod.make_weights(wl, "cuda:0")
    sig = wlmod.make_signal(wl, "cuda:0")
    g = wlmod.make_grads(wl, sig, 0, "cuda:0")
    w0 = _np64(w[0])
    opt.step(w, g)
    torch.cuda.synchronize()
    assert opt.status() == B.OK
    u_or = O.polar_ns_short_side(_np64(opt.tap(B.TAP_MOMENTUM, 0, 0)), K, 1e-12)
    d_gpu = (w0 - _np64(w[0])) / 0.01
    noise = np.linalg.norm(np.abs(w0) * 1.2e-7 / 0.01)
    rel = max(np.linalg.norm(d_gpu - u_or) - noise, 0.0) / np.linalg.norm(u_or)
    print("muon, chain through memory: direction off by", rel)
    assert rel <= 2e-3
    opt.close()


@pytest.mark.parametrize("flags", [0, B.FLAG_GEMM_1CTA])
def test_local_polar_first_gram_in_fp8_equals_bf16_bit_for_bit(flags):
    """The local polar step's first Gram product reads the vote matrix as E4M3 bytes (+-1 are exact, the fp32
    sums of +-1 products are exact integers): the weights after the step equal, bit for bit, those of a run
    whose first Gram product uses the bf16 copy.  Wide, tall, square and ragged shapes; K-major and MN-major tiles."""
    shapes = [(200, 328), (328, 200), (64, 147), (256, 256), (512, 1152), (1152, 512), (130, 48)]
    for dtype, M in (("f32", 3), ("bf16", 4)):
        wl = _wl(shapes, M, dtype=dtype, local_polar=True, lr=0.01)
        sig = wlmod.make_signal(wl, "cuda:0")
        outs = []
        for extra in (0, B.FLAG_LP_GRAM_BF16):
            opt = B.SignMuon(wl.params, M, lr=0.01, local_polar=True, flags=flags | extra)
            w = wlmod.make_weights(wl, "cuda:0")
            for t in range(2):
                opt.step(w, wlmod.make_grads(wl, sig, t, "cuda:0"))
            torch.cuda.synchronize()
            assert opt.status() == B.OK
            outs.append(w)
            opt.close()
        for a, b in zip(*outs):
            assert torch.equal(a, b)


def test_garbage_worker_is_outvoted():
    """One worker sending NaN gradients maps to -1 everywhere; the vote still equals the popcount rule."""
    from parity_utils import check_param_step
    wl = _wl([(64, 128), (1, 64)], 5, kinds=["matrix", "plain"])
    opt = B.SignMuon(wl.params, 5, flags=B.FLAG_KEEP_POLAR)
    w = wlmod.make_weights(wl, "cuda:0")
    sig = wlmod.make_signal(wl, "cuda:0")
    g = wlmod.make_grads(wl, sig, 0, "cuda:0")
    for t in g:
        t[2].fill_(float("nan"))
    opt.step(w, g)
    torch.cuda.synchronize()
    for p in range(2):
        bits = opt.tap(B.TAP_WORKER_BITS, p, 2).cpu().numpy()
        assert not bits.any()                              # NaN >= 0 is false -> bit 0
        import oracle as O
        d = wl.params[p].numel
        packed = [opt.tap(B.TAP_WORKER_BITS, p, m).cpu().numpy()[: (d + 7) // 8] for m in range(5)]
        vote = O.unpack_bits(opt.tap(B.TAP_VOTE_BITS, p, 0).cpu().numpy(), d)
        assert np.array_equal(vote, O.majority_vote_popcount(packed, d))
    opt.close()


def test_degenerate_cases_tiny_matrices_zero_gradient_and_255_workers():
    """The degenerate ends of the method: matrices of one row, one column or a few entries as MATRIX parameters (the
    Gram matrix is then 1 x 1 or 2 x 2 and PolarNS keeps the signs), an all-zero gradient (sigma = 0 -> Y = 0 -> every
    sign bit 1, Alg. 3's note, pad bits 0, W <- W - eta), and the largest worker count the vote supports."""
    from parity_utils import run_and_check, make_optimizer
    run_and_check(_wl([(1, 96), (96, 1), (2, 2), (8, 8), (3, 5), (1, 1)], 3), steps=2)
    run_and_check(_wl([(1, 96), (8, 8), (5, 3)], 2, local_polar=True, lr=0.01), steps=1)
    run_and_check(_wl([(16, 32), (24, 8), (1, 40)], 255, K=2, kinds=["matrix", "matrix", "plain"]), steps=1,
                  ns_workers=[0, 254])
    # all-zero gradients
    wl = _wl([(64, 96), (40, 7), (1, 33)], 4, kinds=["matrix", "matrix", "plain"])
    opt = make_optimizer(wl)
    w = wlmod.make_weights(wl, "cuda:0")
    before = [x.clone() for x in w]
    g = [torch.zeros_like(x) for x in wlmod.make_grads(wl, wlmod.make_signal(wl, "cuda:0"), 0, "cuda:0")]
    opt.step(w, g, wl.lr)
    torch.cuda.synchronize()
    assert opt.status() == B.OK
    import oracle as O
    for p_idx, p in enumerate(wl.params):
        d = p.rows * p.cols
        for m in range(wl.num_workers):
            bits = O.unpack_bits(opt.tap(B.TAP_WORKER_BITS, p_idx, m).cpu().numpy(), d)
            assert bits.all()
        assert O.unpack_bits(opt.tap(B.TAP_VOTE_BITS, p_idx, 0).cpu().numpy(), d).all()
        assert torch.allclose(w[p_idx], before[p_idx] - wl.lr, rtol=0, atol=1e-9)
    opt.close()


def test_sign_agreement_counts_match_the_payload():
    """Per worker, the number of sign bits equal to the vote, against plain counting on the GPU's own bits
    (ragged parameters: pad bits must not be counted)."""
    import oracle as O
    wl = _wl([(64, 147), (200, 328), (1, 37), (5, 9)], 5, kinds=["matrix", "matrix", "plain", "plain"])
    opt = B.SignMuon(wl.params, 5, flags=B.FLAG_KEEP_POLAR | B.FLAG_SIGN_AGREEMENT)
    w = wlmod.make_weights(wl, "cuda:0")
    sig = wlmod.make_signal(wl, "cuda:0")
    for t in range(2):
        opt.step(w, wlmod.make_grads(wl, sig, t, "cuda:0"))
    agree, entries = opt.sign_agreement()
    assert entries == wl.numel
    want = [0] * 5
    for p, prm in enumerate(wl.params):
        vote = O.unpack_bits(opt.tap(B.TAP_VOTE_BITS, p, 0).cpu().numpy(), prm.numel)
        for m in range(5):
            mine = O.unpack_bits(opt.tap(B.TAP_WORKER_BITS, p, m).cpu().numpy(), prm.numel)
            want[m] += int((mine == vote).sum())
    assert agree == want
    assert all(a > entries // 2 for a in agree)       # a majority vote agrees with most workers on most entries
    opt.close()
    plain = B.SignMuon(wl.params, 5)
    with pytest.raises(B.SignMuonError):
        plain.sign_agreement()
    plain.close()


@pytest.mark.parametrize("case", ["plain_params", "matrices_only", "matrices_local_polar", "weight_decay"])
def test_host_resident_step_matches_device_step(case):
    """Six host-buffer steps issued back to back (the gradient copies run one step ahead on the library's own stream;
    without plain parameters and weight decay the weights travel there too and only the vote stage waits for them)
    against six device-buffer steps on the same inputs: bit-identical weights, also when the caller changes the host
    weights between two calls."""
    kinds = ["matrix", "matrix", "plain"] if case == "plain_params" else ["matrix", "matrix", "matrix"]
    shapes = [(128, 256), (64, 147), (1, 40)] if case == "plain_params" else [(128, 256), (64, 147), (320, 512)]
    lp = case == "matrices_local_polar"
    wd = 0.01 if case == "weight_decay" else 0.0
    wl = _wl(shapes, 3, kinds=kinds, local_polar=lp, lr=0.01 if lp else 1e-3)
    sig = wlmod.make_signal(wl, "cuda:0")
    gs = [wlmod.make_grads(wl, sig, t, "cuda:0") for t in range(6)]
    w_dev = wlmod.make_weights(wl, "cuda:0")
    w_host = [x.cpu().pin_memory() for x in w_dev]
    g_host = [[x.cpu().pin_memory() for x in g] for g in gs]
    a = B.SignMuon(wl.params, 3, local_polar=lp, lr=wl.lr, weight_decay=wd)
    b = B.SignMuon(wl.params, 3, local_polar=lp, lr=wl.lr, weight_decay=wd, host_staging=True)
    for t, g in enumerate(gs):
        if t == 3:      # the caller edits the weights between two steps (after synchronising, as the contract asks)
            torch.cuda.synchronize()
            for x, y in zip(w_dev, w_host):
                x.mul_(0.5)
                y.mul_(0.5)
        a.step(w_dev, g)
        b.step_host(w_host, g_host[t])
    torch.cuda.synchronize()
    assert a.status() == B.OK and b.status() == B.OK
    for x, y in zip(w_dev, w_host):
        assert torch.equal(x.cpu(), y)
    a.close(); b.close()
