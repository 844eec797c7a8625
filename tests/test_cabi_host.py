"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the
header declares, validates its arguments and reports sizes that follow from the payload format."""
import ctypes as C
import os
import re

import pytest

from paper_2605_16311_b200 import binding as B
from paper_2605_16311_b200 import build as build_mod
from paper_2605_16311_b200 import workloads as wlmod

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built_library():
    build_mod.build()
    return B.load_library()


def test_library_exports_every_declared_symbol(built_library):
    header = open(os.path.join(ROOT, "include", "signmuon.h")).read()
    declared = set(re.findall(r"\b(signmuon_[a-z_]+)\s*\(", header))
    assert declared == set(B.EXPORTS)
    for name in declared:
        assert hasattr(built_library, name)


def _cfg(params, **kw):
    arr = (B.ParamStruct * len(params))(*[B.ParamStruct(*p) for p in params])
    vals = dict(num_workers=4, momentum=0.9, lr=1e-3, ns_steps=5, local_polar=0, weight_decay=0.0, eps=1e-12,
                update_scale=0, flags=0)
    vals.update(kw)
    cfg = B.ConfigStruct(len(params), arr, vals["num_workers"], vals["momentum"], vals["lr"], vals["ns_steps"],
                         vals["local_polar"], vals["weight_decay"], vals["eps"], vals["update_scale"], vals["flags"])
    cfg._keep = arr
    return cfg


def test_create_rejects_bad_arguments():
    good = [(64, 64, 0, 0, 0)]
    assert B.signmuon_create_raw(None)[0] == -1
    for kw in (dict(num_workers=0), dict(num_workers=256), dict(momentum=1.0), dict(momentum=-0.1),
               dict(ns_steps=-1), dict(weight_decay=-1.0), dict(update_scale=2), dict(local_polar=3),
               dict(lr=float("nan"))):
        code, h = B.signmuon_create_raw(_cfg(good, **kw))
        assert code == -1 and h is None, kw
    for bad in ([(0, 64, 0, 0, 0)], [(64, -1, 0, 0, 0)], [(1 << 25, 4, 0, 0, 0)]):
        assert B.signmuon_create_raw(_cfg(bad))[0] == -2
    assert B.signmuon_create_raw(_cfg([(64, 64, 7, 0, 0)]))[0] == -1
    assert B.signmuon_create_raw(_cfg([(64, 64, 0, 5, 0)]))[0] == -1
    empty = _cfg(good)
    empty.num_params = 0
    assert B.signmuon_create_raw(empty)[0] == -1
    assert B.load_library().signmuon_create(C.byref(_cfg(good)), None) == -1


def test_unbound_context_refuses_device_calls():
    ctx = B.signmuon_create([(64, 64, 0, 0, 0)], 2, 0.9, 1e-3, 5, False)
    lib = B.load_library()
    arr = (C.c_void_p * 1)(C.c_void_p(256))
    assert lib.signmuon_step(ctx, arr, arr, 0.1, None) == -3
    assert lib.signmuon_status(ctx, None) == -3
    p = C.c_void_p()
    assert lib.signmuon_packed_payload(ctx, 0, C.byref(p), None, None) == -3
    assert lib.signmuon_packed_payload(ctx, 2, None, None, None) == -1      # worker out of range
    assert lib.signmuon_bind(ctx, None, 0, None, 0, None, 0, 1, None) == -1
    assert lib.signmuon_bind(ctx, C.c_void_p(1024), 16, C.c_void_p(1024), 16, None, 0, 1, None) == -4
    B.signmuon_destroy(ctx)
    assert B.load_library().signmuon_error_string(-6).decode().startswith("a bounded")


@pytest.mark.parametrize("name", ["c1", "c2", "c3", "c4"])
def test_payload_is_one_bit_per_entry(name):
    wl = wlmod.by_name(name)
    tuples = [(p.rows, p.cols, B._KIND[p.kind], B._DT[p.dtype], B._DT[p.dtype]) for p in wl.params]
    ctx = B.signmuon_create(tuples, wl.num_workers, wl.momentum, wl.lr, wl.ns_steps, wl.local_polar)
    _, nbytes, entries = B.signmuon_packed_payload(ctx, 0, want_ptr=False)
    assert entries == wl.numel
    assert nbytes * 8 == entries                      # exactly one bit per entry at these shapes
    assert 4 * entries / nbytes == 32                 # 32x smaller than float32
    off = 0
    for i, p in enumerate(wl.params):
        o, w = B.signmuon_payload_segment(ctx, i)
        assert o == off and w == (p.numel + 31) // 32
        off += w
    state, ws, staging = B.signmuon_state_bytes(ctx)
    assert state >= 4 * wl.num_workers * wl.numel     # one float32 momentum per worker and entry
    assert state < 4 * wl.num_workers * wl.numel + 256 * len(wl.params) + 1
    assert ws > wl.num_workers * nbytes
    flops = B.signmuon_ns_flops_per_step(ctx)
    expect = sum(4.0 * min(p.rows, p.cols) ** 2 * max(p.rows, p.cols) * wl.ns_steps *
                 (wl.num_workers + (1 if wl.local_polar else 0)) for p in wl.params if p.kind == "matrix")
    assert flops == pytest.approx(expect, rel=1e-12)
    B.signmuon_destroy(ctx)


def test_ragged_parameter_pads_to_words():
    ctx = B.signmuon_create([(3, 11, 0, 0, 0), (1, 5, 1, 0, 0)], 3, 0.9, 1e-3, 2, False)
    _, nbytes, entries = B.signmuon_packed_payload(ctx, 1, want_ptr=False)
    assert entries == 38 and nbytes == 4 * (2 + 1)
    assert B.signmuon_payload_segment(ctx, 1) == (2, 1)
    # momentum, norms, plain kernel; the 3 x 11 matrix iterates in Gram space (first Gram product, on-chip chain, last
    # apply product); fallback pack (11 columns do not fill words), vote, update
    assert B.signmuon_launches_per_step(ctx) == 2 + 1 + 3 + 1 + 2
    full = B.signmuon_create([(3, 11, 0, 0, 0), (1, 5, 1, 0, 0)], 3, 0.9, 1e-3, 2, False, flags=B.FLAG_NO_GRAM_SPACE)
    assert B.signmuon_launches_per_step(full) == 2 + 1 + 4 + 1 + 2          # 2 x 2 products on the full matrix
    B.signmuon_destroy(full)
    B.signmuon_destroy(ctx)


def test_power_start_layout_and_errors():
    lib = B.load_library()
    # Frobenius scale: no start vectors
    ctx = B.signmuon_create([(8, 12, 0, 0, 0)], 2, 0.9, 1e-3, 5, False)
    assert B.signmuon_power_start_size(ctx) == 0
    assert lib.signmuon_power_start_segment(ctx, 0, None, None) == -1
    B.signmuon_destroy(ctx)
    # spectral scale: [M][cols] floats per matrix parameter, in creation order; plain parameters have none
    params = [(8, 12, 0, 0, 0), (1, 40, 1, 0, 0), (20, 6, 0, 0, 0)]
    ctx = B.signmuon_create(params, 3, 0.9, 1e-3, 5, False, ns_scale=1, power_iters=2)
    assert B.signmuon_power_start_size(ctx) == 3 * 12 + 3 * 6
    assert B.signmuon_power_start_segment(ctx, 0) == (0, 12)
    assert B.signmuon_power_start_segment(ctx, 2) == (36, 6)
    assert lib.signmuon_power_start_segment(ctx, 1, None, None) == -1      # plain parameter
    assert lib.signmuon_set_power_start(ctx, C.c_void_p(4096), 54) == -3     # not bound yet
    # momentum, start norm + 2 rounds x 4 + final matvec + sigma, 5 x 2 NS products, fallback pack, vote, plain kernel
    assert B.signmuon_launches_per_step(ctx) == 1 + (3 + 8) + 10 + 1 + 2 + 1
    B.signmuon_destroy(ctx)
    for kw in (dict(ns_scale=2), dict(ns_scale=-1), dict(power_iters=-1), dict(power_iters=65)):
        cfg = _cfg([(64, 64, 0, 0, 0)])
        for k, v in kw.items():
            setattr(cfg, k, v)
        assert B.signmuon_create_raw(cfg)[0] == -1, kw


def test_header_is_plain_c(tmp_path):
    """include/signmuon.h must compile as C (no C++ in the boundary) and a C caller must link against the library."""
    import subprocess
    src = tmp_path / "use.c"
    src.write_text('#include "signmuon.h"\n'
                   '#include <stdio.h>\n'
                   'int main(void) {\n'
                   '  signmuon_param p = {64, 64, SIGNMUON_PARAM_MATRIX, SIGNMUON_F32, SIGNMUON_F32};\n'
                   '  signmuon_config c = {0};\n'
                   '  signmuon_ctx* ctx = NULL;\n'
                   '  size_t bytes = 0, entries = 0;\n'
                   '  c.num_params = 1; c.params = &p; c.num_workers = 4; c.momentum = 0.9f; c.lr = 1e-3f; c.ns_steps = 5;\n'
                   '  if (signmuon_create(&c, &ctx) != SIGNMUON_OK) return 1;\n'
                   '  if (signmuon_packed_payload(ctx, 0, NULL, &bytes, &entries) != SIGNMUON_OK) return 2;\n'
                   '  printf("%zu %zu %s\\n", bytes, entries, signmuon_error_string(SIGNMUON_ERR_TIMEOUT));\n'
                   '  signmuon_destroy(ctx);\n'
                   '  return 0;\n'
                   '}\n')
    exe = tmp_path / "use"
    libdir = os.path.dirname(B.LIB_PATH)
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Werror", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe),
                    "-L", libdir, "-l:libsignmuon.so", "-Wl,-rpath," + libdir], check=True)
    out = subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.split(maxsplit=2)
    assert out[0] == "512" and out[1] == "4096"          # 64 x 64 entries, one bit each
    assert out[2].startswith("a bounded")


def test_worker_shard_arguments_and_payload_buffer_layout():
    """A context may compute a block of the workers only (the others' payload rows arrive by the exchange):
    argument checks, state sized for the own workers, payload buffer with one 128-byte-aligned row per worker."""
    lib = B.load_library()
    params = [(64, 96, 0, 0, 0), (1, 40, 1, 0, 0)]
    full = B.signmuon_create(params, 8, 0.9, 1e-3, 5, False)
    part = B.signmuon_create(params, 8, 0.9, 1e-3, 5, False, worker_offset=4, local_workers=2)
    st_full, _, _ = B.signmuon_state_bytes(full)
    st_part, _, _ = B.signmuon_state_bytes(part)
    assert st_part == 2 * 64 * 96 * 4 + 512 and st_full == 8 * 64 * 96 * 4 + 1280    # momenta of 2 of the 8 workers (256-byte slabs)
    _, pitch, rows = B.signmuon_payload_buffer(part, want_ptr=False)
    _, nbytes, _ = B.signmuon_packed_payload(part, 7, want_ptr=False)
    assert rows == 8 and pitch % 128 == 0 and pitch >= nbytes == 4 * (64 * 96 // 32 + 2)
    p = C.c_void_p()
    assert lib.signmuon_payload_buffer(part, C.byref(p), None, None) == -3          # not bound yet
    # a sharded context cannot run the whole step in one call: the exchange sits between the stages
    arr = (C.c_void_p * 2)(4096, 8192)
    assert lib.signmuon_step(part, arr, arr, C.c_float(1e-3), None) == -1
    for bad in (dict(worker_offset=7, local_workers=2), dict(worker_offset=-1, local_workers=1),
                dict(worker_offset=0, local_workers=9)):
        with pytest.raises(B.SignMuonError):
            B.signmuon_create(params, 8, 0.9, 1e-3, 5, False, **bad)
    B.signmuon_destroy(full); B.signmuon_destroy(part)
