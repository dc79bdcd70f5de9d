"""world_size-2 gloo run of the image sharding used for several GPUs (CPU only; the worker is the oracle)."""
import os
import socket

import numpy as np
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
import workloads as wl
from paper_2108_09413_b200 import multi

N0, N, SIGMA, ALPHA, ID0 = 20, 60, 0.25, 0.001, 40


def _oracle_worker(model):
    om = oracle.Model(model)

    def fn(block, first_id):
        res = [oracle.certify(om, x, wl.NOISE_SEED, first_id + i, N0, N, SIGMA, ALPHA) for i, x in enumerate(block)]
        return (np.array([r[0] for r in res], np.int32), np.array([r[1] for r in res], np.float64),
                np.stack([r[2] for r in res]), np.stack([r[3] for r in res]))
    return fn


def _rank_main(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), OMP_NUM_THREADS="2")
    dist.init_process_group("gloo", rank=rank, world_size=world)
    images = wl.images(5, seed=123)
    res = multi.certify_sharded(_oracle_worker(wl.tiny_cnn()), images, image_id0=ID0)
    slowest = multi.max_over_ranks(10.0 + rank)
    np.savez(os.path.join(out_dir, f"rank{rank}.npz"), cls=res[0], rad=res[1], c0=res[2], c1=res[3], slowest=slowest)
    dist.barrier()
    dist.destroy_process_group()


def test_image_blocks_partition_the_images():
    for n in (0, 1, 5, 8, 500):
        for world in (1, 2, 3, 8):
            blocks = [multi.image_block(r, world, n) for r in range(world)]
            assert blocks[0][0] == 0 and blocks[-1][1] == n
            assert all(blocks[i][1] == blocks[i + 1][0] for i in range(world - 1))
            sizes = [e - b for b, e in blocks]
            assert max(sizes) - min(sizes) <= 1


def test_two_ranks_equal_one_process(tmp_path):
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    mp.spawn(_rank_main, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    images = wl.images(5, seed=123)
    single = _oracle_worker(wl.tiny_cnn())(images, ID0)
    for rank in range(2):
        got = np.load(tmp_path / f"rank{rank}.npz")
        np.testing.assert_array_equal(got["cls"], single[0])
        np.testing.assert_array_equal(got["rad"], single[1])
        np.testing.assert_array_equal(got["c0"], single[2])
        np.testing.assert_array_equal(got["c1"], single[3])
        assert float(got["slowest"]) == 11.0
