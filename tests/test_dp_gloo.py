"""Two gloo ranks on CPU: token-sharded data parallelism reproduces the single-process result.

The ranks run the CPU oracle on their token shards with the library's sharding helper; the
all-reduced grad_W equals the unsharded one and the MVUE draws are those of the unsharded batch
(global group counter), so the outcome does not depend on the data-parallel degree.
"""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2409_09099_b200 import synth


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import sste_oracle as orc
    from paper_2409_09099_b200 import dp
    O, I, T = 128, 256, 512
    W, X, dY = (synth.gaussian_bf16(11, (O, I), 0.02), synth.gaussian_bf16(12, (T, I), 1.0),
                synth.gaussian_bf16(13, (T, O), 1e-2))
    t0, n = dp.token_shard(T, rank, world)
    beta32 = np.float32(orc.beta(W)[0])                          # identical on every rank: a function of W only
    vals, meta, dense = orc.project_compress(W, beta32)
    Xs, dYs = X[t0:t0 + n].copy(), dY[t0:t0 + n].copy()
    Y = orc.linear_fwd(Xs, orc.BF16, vals, meta, orc.BF16)
    gv, gm, _, _ = orc.mvue(dYs, seed=5, tensor_id=2, step=7, token_offset=t0)
    dW = torch.from_numpy(orc.linear_bwd_weight(gv, gm, orc.BF16, Xs, orc.BF16))
    dX = orc.linear_bwd_input(dYs, orc.BF16, dense, orc.BF16)
    for h in dp.allreduce_grad_w([dW]):
        h.wait()
    gathered = [torch.zeros_like(torch.from_numpy(gv.astype(np.int32))) for _ in range(world)]
    dist.all_gather(gathered, torch.from_numpy(gv.astype(np.int32)))
    if rank == 0:
        # unsharded reference
        gv_full, gm_full, _, _ = orc.mvue(dY, seed=5, tensor_id=2, step=7)
        dW_full = orc.linear_bwd_weight(gv_full, gm_full, orc.BF16, X, orc.BF16)
        gv_cat = np.concatenate([g.numpy().astype(np.uint16) for g in gathered], axis=1)
        np.save(os.path.join(out_dir, "ok.npy"), np.array([
            np.array_equal(gv_cat, gv_full),
            np.allclose(dW.numpy(), dW_full, rtol=1e-12, atol=1e-15),
            np.allclose(Y, orc.linear_fwd(X, orc.BF16, vals, meta, orc.BF16)[t0:t0 + n]),
            np.allclose(dX, orc.linear_bwd_input(dY, orc.BF16, dense, orc.BF16)[t0:t0 + n]),
        ]))
    dist.barrier()
    dist.destroy_process_group()


def test_token_sharding_matches_single_process(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    ok = np.load(tmp_path / "ok.npy")
    assert ok.all(), ok


def test_token_shard_helper():
    from paper_2409_09099_b200 import dp
    assert dp.token_shard(1024, 0, 2) == (0, 512) and dp.token_shard(1024, 1, 2) == (512, 512)
    assert dp.token_shard(8192, 3, 8) == (3072, 1024)
    assert dp.allreduce_grad_w([torch.zeros(2)]) == []       # no process group: nothing to exchange
