"""signmuon_momentum_norm_noalloc against the regular momentum stage.

The entry point exists for callers that may not allocate device memory while an optimizer step is being
issued (a frozen memory plan, a host framework's allocator that must not grow, a loop that cannot take the
allocator lock); it keeps its reduction scratch in a fixed array inside the library.  This file is named so
that pytest collects it last: a run that stops at the first failure has then already run everything else.
The test drives two calls in a row through the C ABI - the second one reuses the built-in scratch that the
first left behind - and compares momentum, bf16 operand and norm factors with what signmuon_run_stages
produces for the same inputs, and with the float64 oracle's momentum recursion and Frobenius norm.
"""
import numpy as np
import pytest
import torch

import oracle as O

from paper_2605_16311_b200 import binding as B
from paper_2605_16311_b200 import workloads as wlmod


def test_noalloc_rejects_oversize_and_bad_arguments_without_a_gpu():
    from paper_2605_16311_b200 import build as build_mod
    build_mod.build()
    f = B.signmuon_momentum_norm_noalloc
    ok_ptr = 4096
    # capacity: 64 workers x ceil(8192*8192/8192) = 524288 partial sums > 65536
    assert f(ok_ptr, B.F32, 0, B.F32, ok_ptr, ok_ptr, ok_ptr, 8192, 8192, 64, 0.9, 0.0, 1e-12, 0) == B.ERR_TOO_LARGE
    assert f(ok_ptr, B.F32, 0, B.F32, ok_ptr, ok_ptr, ok_ptr, 3, 5, 2, 0.9, 0.0, 1e-12, 0) == -2     # d % 8 != 0
    assert f(0, B.F32, 0, B.F32, ok_ptr, ok_ptr, ok_ptr, 8, 8, 2, 0.9, 0.0, 1e-12, 0) == -1          # null grads
    assert f(ok_ptr, B.F32, 0, B.F32, ok_ptr, ok_ptr, ok_ptr, 8, 8, 2, 0.9, 0.1, 1e-12, 0) == -1     # decay w/o weights
    assert f(ok_ptr + 4, B.F32, 0, B.F32, ok_ptr, ok_ptr, ok_ptr, 8, 8, 2, 0.9, 0.0, 1e-12, 0) == -8  # misaligned
    assert B.load_library().signmuon_error_string(B.ERR_TOO_LARGE).decode().startswith("problem exceeds")


@pytest.mark.gpu
@pytest.mark.parametrize("dtype,rows,cols,M,wd", [("f32", 200, 328, 4, 0.0), ("bf16", 768, 1024, 3, 0.05)])
def test_noalloc_matches_regular_momentum_stage_twice(dtype, rows, cols, M, wd):
    assert torch.cuda.is_available()
    dev = "cuda:0"
    wl = wlmod.Workload("noalloc", [wlmod.Param(rows, cols, "matrix", dtype, "w")], num_workers=M, ns_steps=0,
                        config_id=55)
    # regular path: K = 0 so that the bf16 operand (Y_0) stays readable through the polar tap
    opt = B.SignMuon(wl.params, M, momentum=0.9, ns_steps=0, weight_decay=wd, flags=B.FLAG_KEEP_POLAR)
    weights = wlmod.make_weights(wl, dev)
    signal = wlmod.make_signal(wl, dev)
    d = rows * cols
    dt = B._DT[dtype]
    mom = torch.zeros(M, d, dtype=torch.float32, device=dev)           # caller-owned outputs
    operand = torch.empty(M, d, dtype=torch.bfloat16, device=dev)
    scales = torch.empty(M, 2, dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream().cuda_stream
    w64 = weights[0].float().cpu().numpy().astype(np.float64)
    mom_or = np.zeros((M, rows, cols))                                 # the oracle's momentum, evolved alongside
    for step in range(2):                                              # two calls in a row, shared scratch
        grads = wlmod.make_grads(wl, signal, step, dev)
        opt.step(weights, grads, stages=B.STAGE_MOMENTUM)
        rc = B.signmuon_momentum_norm_noalloc(grads[0].data_ptr(), dt, weights[0].data_ptr(), dt, mom.data_ptr(),
                                              operand.data_ptr(), scales.data_ptr(), rows, cols, M, 0.9, wd,
                                              1e-12, stream)
        assert rc == B.OK
        torch.cuda.synchronize()
        for m in range(M):
            ref_mom = opt.tap(B.TAP_MOMENTUM, 0, m).reshape(-1)
            # same arithmetic in the same order: the tests' momentum tolerance (2e-6 of the largest entry)
            assert (mom[m] - ref_mom).abs().max() <= 2e-6 * ref_mom.abs().max()
            ref_op = opt.tap(B.TAP_POLAR, 0, m).reshape(-1).float()
            assert (operand[m].float() - ref_op).abs().max() <= 2e-6 * ref_op.abs().max() + 2 ** -8 * 2e-6
            ref_sc = opt.tap(B.TAP_NORM, 0, m)
            assert torch.allclose(scales[m], ref_sc, rtol=1e-5, atol=0)
        # against the oracle (Alg. 2 momentum, Alg. 4 sigma = ||Mom||_F): the tolerances of the staged parity tests
        g64 = grads[0].float().cpu().numpy().astype(np.float64)
        mom_gpu = mom.cpu().numpy().astype(np.float64).reshape(M, rows, cols)
        for m in range(M):
            mom_or[m] = O.momentum_update(mom_or[m], g64[m], w64, 0.9, wd)
            assert np.max(np.abs(mom_gpu[m] - mom_or[m])) <= 2e-6 * np.max(np.abs(mom_or[m]))
            sigma = max(O.frobenius_norm(mom_gpu[m]), 1e-12)
            sc = scales[m].cpu().numpy().astype(np.float64)
            assert abs(sc[1] * sigma - 1.0) <= 1e-5 and abs(sc[0] * sigma * sigma - 1.0) <= 2e-5
            assert np.array_equal(operand[m].float().cpu().numpy().reshape(rows, cols),
                                  O.round_to_bf16(mom_gpu[m]))          # the operand is the rounded momentum
        mom_or = mom_gpu.copy()                                         # staged: continue from the GPU's state
    opt.close()
