"""Host side of the vocabulary-sharded verification, on CPU: the column partition the library
prescribes, and the collectives of a step over torch.distributed with the gloo backend (world
size 2) against the in-process stand-in that the one-GPU tests use."""
import os
import types

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2401_06706_b200 import binding, build


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build()
    binding.load_library()


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("vocab", [1, 7, 1000, 4096, 4097, 32000, 50272, 65536])
def test_column_partition(vocab, dtype):
    for g in (1, 2, 3, 4, 8, 32):
        parts = [binding.mcsd_shard_columns(vocab, dtype, g, s) for s in range(g)]
        eps = parts[0][2]
        assert all(p[2] == eps for p in parts) and g * eps >= 1 and (g == 1 or (g - 1) * eps < 32 + eps)
        pos = 0
        for begin, n, _ in parts:
            if n:
                assert begin == pos            # contiguous, in order
                pos += n
        assert pos == vocab                    # the whole vocabulary, once
        run = parts[0][1] // eps if (parts[0][1] % eps == 0 and g > 1 and parts[0][1] < vocab) else None
        if run:
            assert all(b % run == 0 for b, n, _ in parts if n)   # shards start at run boundaries
    lib = binding.load_library()
    assert lib.mcsd_shard_columns(vocab, 0, 0, 0, None, None, None) == -2
    assert lib.mcsd_shard_columns(vocab, 0, 2, 2, None, None, None) == -2
    assert lib.mcsd_shard_columns(vocab, 9, 2, 0, None, None, None) == -3


def test_rounds_follow_the_widest_node():
    from paper_2401_06706_b200 import synth
    lib = binding.load_library()
    for kc, want in (("", 0), ("1x1", 0), ("2", 1), ("4x2x2x1", 3), ("8x1", 7), ("2x32", 31)):
        parent = synth.tree_from_kconfig(synth.parse_kconfig(kc))
        assert lib.mcsd_shard_rounds(parent.ctypes.data, parent.shape[0]) == want
    bad = np.array([-1, 1], dtype=np.int32)
    assert lib.mcsd_shard_rounds(bad.ctypes.data, 2) == -6


def _fake_shard(rank, world, n_items=5, eps=3):
    g = torch.Generator().manual_seed(100 + rank)
    sh = types.SimpleNamespace(shard=rank)
    sh.part = torch.rand((n_items, eps, 4), generator=g)
    sh.part_all = torch.zeros((world, n_items, eps, 4))
    sh.totals = torch.rand((2, eps), generator=g, dtype=torch.float64)
    sh.totals_all = torch.zeros((world, 2, eps), dtype=torch.float64)
    sh.endpoint_part = torch.tensor([-1, 40 + rank, -1 if rank else 7], dtype=torch.int32)
    return sh


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    sh = _fake_shard(rank, world)
    comm = binding.DistComm()
    comm.all_gather([sh], "part", "part_all")
    comm.all_gather([sh], "totals", "totals_all")
    comm.all_reduce_max([sh], "endpoint_part")
    torch.save({"part_all": sh.part_all, "totals_all": sh.totals_all, "endpoint": sh.endpoint_part},
               os.path.join(out_dir, f"rank{rank}.pt"))
    dist.barrier()
    dist.destroy_process_group()


def test_collectives_over_two_gloo_ranks_match_the_in_process_stand_in(tmp_path):
    world = 2
    port = 29700 + os.getpid() % 200
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    shards = [_fake_shard(r, world) for r in range(world)]
    local = binding.LocalComm()
    local.all_gather(shards, "part", "part_all")
    local.all_gather(shards, "totals", "totals_all")
    local.all_reduce_max(shards, "endpoint_part")
    for r in range(world):
        got = torch.load(tmp_path / f"rank{r}.pt")
        assert torch.equal(got["part_all"], shards[r].part_all)          # [shard][node][entry][4], shard-major
        assert torch.equal(got["totals_all"], shards[r].totals_all)
        assert got["endpoint"].tolist() == [-1, 41, 7] == shards[r].endpoint_part.tolist()
    assert torch.equal(shards[0].part_all[1], _fake_shard(1, world).part)
