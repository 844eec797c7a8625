"""Workers sharded over several contexts (Alg. 2 / Alg. 3 across GPUs).

CPU part: two gloo ranks exchange oracle-packed payloads through the package's exchange module (1-bit all-gather and
int8 SUM all-reduce) and vote; the result equals the single-process vote bit for bit.
GPU part (one GPU, the shards run one after the other, nothing waits on anything): sharded contexts + a copy of the
payload rows against one context that holds all workers - payloads, vote and weights bit-identical.
"""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import oracle as O
from paper_2605_16311_b200 import exchange
from paper_2605_16311_b200 import workloads as wlmod


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


D_ENTRIES = 1000          # not a multiple of 32: the last word is padded
M_WORKERS = 6


def _worker_bits():
    rng = np.random.default_rng(77)
    return (rng.normal(size=(M_WORKERS, D_ENTRIES)) + 0.3 >= 0).astype(np.uint8)


def _rank_main(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    bits = _worker_bits()
    per = M_WORKERS // world
    words = (D_ENTRIES + 31) // 32
    pitch = 32 * ((words + 31) // 32)                   # rows padded to 128 bytes, as in the library's buffer
    rows = torch.zeros(M_WORKERS, pitch, dtype=torch.int32)
    for m in range(rank * per, (rank + 1) * per):       # this rank packs its own workers only
        w = O.bytes_to_words(O.pack_bits(bits[m])).astype(np.uint32).view(np.int32)
        rows[m, :words] = torch.from_numpy(w.copy())
    exchange.all_gather_payload(rows, rank * per, per, dist)
    packed = [O.words_to_bytes(rows[m, :words].numpy().view(np.uint32), D_ENTRIES) for m in range(M_WORKERS)]
    vote_gather = O.majority_vote_popcount(packed, D_ENTRIES)
    # Alg. 2: int8 sums of the own workers' signs, SUM all-reduce, sign of the sum (ties -> +1)
    sums = torch.from_numpy(O.decode_bits(bits[rank * per:(rank + 1) * per]).astype(np.int64).sum(axis=0).astype(np.int8))
    exchange.all_reduce_sign_sums(sums, dist)
    vote_sum = (sums.numpy() >= 0).astype(np.uint8)
    np.save(os.path.join(out_dir, f"gather{rank}.npy"), vote_gather)
    np.save(os.path.join(out_dir, f"sum{rank}.npy"), vote_sum)
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_sharded_vote_equals_single_process(tmp_path):
    world = 2
    mp.spawn(_rank_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    bits = _worker_bits()
    want = O.majority_vote_popcount([O.pack_bits(bits[m]) for m in range(M_WORKERS)], D_ENTRIES)
    assert np.array_equal(O.decode_bits(want), O.majority_vote_sum(O.decode_bits(bits)))
    for rank in range(world):
        assert np.array_equal(np.load(tmp_path / f"gather{rank}.npy"), want)
        assert np.array_equal(np.load(tmp_path / f"sum{rank}.npy"), want)


def test_all_gather_payload_refuses_unequal_blocks():
    class FakeDist:
        @staticmethod
        def get_world_size(group=None): return 2
        @staticmethod
        def get_rank(group=None): return 1
    rows = torch.zeros(6, 32, dtype=torch.int32)
    with pytest.raises(ValueError):
        exchange.all_gather_payload(rows, 2, 2, FakeDist)        # 2 ranks x 2 workers != 6
    with pytest.raises(ValueError):
        exchange.all_gather_payload(rows, 0, 3, FakeDist)        # rank 1 must own workers 3..5
    vol = exchange.payload_volume_bytes(32 * 1024, 16, 8)
    assert vol["all_gather_1bit"] == 4096 * 16 * 7 / 8 and vol["all_reduce_int8"] == 2 * 32768 * 7 / 8


# ------------------------------------------------------------------------------------------------ GPU
def _mixed_workload(M, local_polar, dtype="f32"):
    ps = [wlmod.Param(200, 328, "matrix", dtype, "a"), wlmod.Param(64, 147, "matrix", dtype, "stem"),
          wlmod.Param(256, 256, "matrix", dtype, "sq"), wlmod.Param(1, 200, "plain", dtype, "g"),
          wlmod.Param(40, 33, "plain", dtype, "ragged")]
    return wlmod.Workload("shard", ps, num_workers=M, lr=0.01 if local_polar else 1e-3, ns_steps=5,
                          local_polar=local_polar, signal_std=1e-3, noise_std=3e-3, config_id=91)


@pytest.mark.gpu
@pytest.mark.parametrize("M,shards,local_polar,dtype", [(4, 2, False, "f32"), (8, 4, True, "bf16"), (6, 3, True, "f32")])
def test_sharded_contexts_equal_one_context(M, shards, local_polar, dtype):
    from paper_2605_16311_b200 import binding as B
    from paper_2605_16311_b200 import build as build_mod
    build_mod.build()
    dev = "cuda:0"
    wl = _mixed_workload(M, local_polar, dtype)
    per = M // shards
    full = B.SignMuon(wl.params, M, lr=wl.lr, local_polar=local_polar)
    parts = [B.SignMuon(wl.params, M, lr=wl.lr, local_polar=local_polar, worker_offset=r * per, local_workers=per)
             for r in range(shards)]
    sig = wlmod.make_signal(wl, dev)
    w_full = wlmod.make_weights(wl, dev)
    w_parts = [wlmod.make_weights(wl, dev) for _ in range(shards)]      # every "rank" holds a replica of the weights
    for t in range(3):
        grads = wlmod.make_grads(wl, sig, t, dev)
        full.step(w_full, grads)
        local = [[g[r * per:(r + 1) * per].contiguous() for g in grads] for r in range(shards)]
        for r, opt in enumerate(parts):                                 # own workers' stages
            opt.step(w_parts[r], local[r], stages=B.STAGE_MOMENTUM | B.STAGE_NS)
        torch.cuda.synchronize()
        own_rows = [opt.payload_rows()[r * per:(r + 1) * per].clone() for r, opt in enumerate(parts)]
        for r, opt in enumerate(parts):
            if r % 2 == 0:      # the exchange written straight into the payload buffer (what an in-place all-gather does)
                for q in range(shards):
                    if q != r:
                        opt.payload_rows()[q * per:(q + 1) * per].copy_(own_rows[q])
                opt.step(w_parts[r], local[r], stages=B.STAGE_VOTE | B.STAGE_LOCAL_POLAR)
            else:               # payload pointers handed to signmuon_vote_update (gathered elsewhere)
                ptrs = [None if m // per == r else own_rows[m // per][m % per] for m in range(M)]
                opt.vote_update(w_parts[r], local[r], payloads=ptrs)
        torch.cuda.synchronize()
        for r, opt in enumerate(parts):
            assert opt.status() == B.OK
            for m in range(M):
                assert torch.equal(opt.payload(m), full.payload(m))
            for a, b in zip(w_parts[r], w_full):
                assert torch.equal(a, b)
            for p in range(len(wl.params)):
                assert torch.equal(opt.tap(B.TAP_VOTE_BITS, p), full.tap(B.TAP_VOTE_BITS, p))
    with pytest.raises(B.SignMuonError):
        parts[0].step(w_parts[0], local[0])                 # a sharded context has no one-call step
    with pytest.raises(B.SignMuonError):
        parts[0].tap(B.TAP_MOMENTUM, 0, M - 1)              # not one of its own workers
    for opt in parts + [full]:
        opt.close()


@pytest.mark.gpu
def test_int8_sum_exchange_equals_bit_gather():
    """Alg. 2 (int8 sums, SUM all-reduce, sign) against Alg. 3 (1-bit all-gather, popcount vote): the reduced sums
    of two shards, added here on the device, give bit-identical votes and weights; the sums themselves equal the
    oracle's integer sum of the GPU's own sign bits."""
    from paper_2605_16311_b200 import binding as B
    from paper_2605_16311_b200 import build as build_mod
    build_mod.build()
    dev = "cuda:0"
    M, per = 6, 3
    wl = _mixed_workload(M, True)
    full = B.SignMuon(wl.params, M, lr=wl.lr, local_polar=True)
    parts = [B.SignMuon(wl.params, M, lr=wl.lr, local_polar=True, worker_offset=r * per, local_workers=per) for r in range(2)]
    sig = wlmod.make_signal(wl, dev)
    grads = wlmod.make_grads(wl, sig, 0, dev)
    w_full = wlmod.make_weights(wl, dev)
    w_parts = [wlmod.make_weights(wl, dev) for _ in range(2)]
    full.step(w_full, grads)
    local = [[g[r * per:(r + 1) * per].contiguous() for g in grads] for r in range(2)]
    sums = []
    for r, opt in enumerate(parts):
        opt.step(w_parts[r], local[r], stages=B.STAGE_MOMENTUM | B.STAGE_NS)
        sums.append(opt.local_sign_sum())
    total = sums[0] + sums[1]                                   # what the SUM all-reduce leaves on every rank
    for r, opt in enumerate(parts):
        opt.vote_update_from_sums(total, w_parts[r], local[r])
    torch.cuda.synchronize()
    words = full.payload(0).numel() // 4
    d_bits = words * 32
    signs = np.stack([O.decode_bits(O.unpack_bits(full.payload(m).cpu().numpy(), d_bits)) for m in range(M)])
    assert np.array_equal(total.cpu().numpy().astype(np.int64), signs.astype(np.int64).sum(axis=0))
    assert np.array_equal(sums[1].cpu().numpy().astype(np.int64), signs[per:].astype(np.int64).sum(axis=0))
    for r, opt in enumerate(parts):
        assert opt.status() == B.OK
        for a, b in zip(w_parts[r], w_full):
            assert torch.equal(a, b)
        for p in range(len(wl.params)):
            assert torch.equal(opt.tap(B.TAP_VOTE_BITS, p), full.tap(B.TAP_VOTE_BITS, p))
    for opt in parts + [full]:
        opt.close()


@pytest.mark.gpu
@pytest.mark.parametrize("local_polar", [False, True])
def test_fused_exchange_peer_stores_on_one_gpu(local_polar):
    """The exchange fused into the pack: two sharded contexts on one GPU name each other's payload buffer as a
    peer, so every payload word either of them packs (tensor-core epilogue, stand-alone pack kernel, plain-parameter
    kernel) lands in both buffers, and the flag hand-shake lets the vote start.  The contexts run one after the
    other on one stream - each flag is set before anything waits for it - and must match one full context."""
    from paper_2605_16311_b200 import binding as B
    from paper_2605_16311_b200 import build as build_mod
    build_mod.build()
    dev = "cuda:0"
    M, per = 4, 2
    wl = _mixed_workload(M, local_polar)
    full = B.SignMuon(wl.params, M, lr=wl.lr, local_polar=local_polar)
    parts = [B.SignMuon(wl.params, M, lr=wl.lr, local_polar=local_polar, worker_offset=r * per, local_workers=per)
             for r in range(2)]
    parts[0].set_payload_peers(0, 2, [parts[1]])
    parts[1].set_payload_peers(1, 2, [parts[0]])
    assert parts[0].launches_per_step == full.launches_per_step + 2          # publish + await
    sig = wlmod.make_signal(wl, dev)
    w_full = wlmod.make_weights(wl, dev)
    w_parts = [wlmod.make_weights(wl, dev) for _ in range(2)]
    for t in range(3):
        grads = wlmod.make_grads(wl, sig, t, dev)
        full.step(w_full, grads)
        local = [[g[r * per:(r + 1) * per].contiguous() for g in grads] for r in range(2)]
        for r, opt in enumerate(parts):          # both pack (and publish) before either votes
            opt.step(w_parts[r], local[r], stages=B.STAGE_MOMENTUM | B.STAGE_NS)
        for r, opt in enumerate(parts):
            opt.step(w_parts[r], local[r], stages=B.STAGE_VOTE | B.STAGE_LOCAL_POLAR)
        torch.cuda.synchronize()
        for r, opt in enumerate(parts):
            assert opt.status() == B.OK
            for m in range(M):
                assert torch.equal(opt.payload(m), full.payload(m))
            for a, b in zip(w_parts[r], w_full):
                assert torch.equal(a, b)
    # a missing peer: rank 1 never packs, so rank 0's bounded wait for its flag runs out and is reported
    parts[0].set_wait_limit(2_000_000)
    grads = wlmod.make_grads(wl, sig, 3, dev)
    local0 = [g[:per].contiguous() for g in grads]
    parts[0].step(w_parts[0], local0, stages=B.STAGE_MOMENTUM | B.STAGE_NS)
    parts[0].step(w_parts[0], local0, stages=B.STAGE_VOTE | B.STAGE_LOCAL_POLAR)
    assert parts[0].status() == B.ERR_TIMEOUT
    for opt in parts + [full]:
        opt.close()
