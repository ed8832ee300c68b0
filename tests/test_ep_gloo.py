"""Expert-parallel plumbing on the CPU: the ownership map and the reduction of the ranks' partial outputs,
with two gloo ranks.  (The kernels of a shard are checked on one GPU in tests/test_gpu_ep.py.)"""
import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from paper_2602_16052_b200 import ep  # noqa: E402


@pytest.mark.parametrize("n_experts,world", [(64, 1), (64, 2), (64, 8), (8, 2), (8, 8), (128, 3), (7, 4)])
def test_every_expert_has_exactly_one_owner(n_experts, world):
    seen = []
    for r in range(world):
        first, count = ep.expert_range(r, world, n_experts)
        assert count >= 1
        seen += list(range(first, first + count))
    assert seen == list(range(n_experts))                       # contiguous blocks, in rank order, no gaps
    sizes = [ep.expert_range(r, world, n_experts)[1] for r in range(world)]
    assert max(sizes) - min(sizes) <= 1
    for e in (0, n_experts // 2, n_experts - 1):
        first, count = ep.expert_range(ep.owner_of(e, world, n_experts), world, n_experts)
        assert first <= e < first + count
    with pytest.raises(ValueError):
        ep.expert_range(world, world, n_experts)


def test_sum_in_rank_order_is_the_left_to_right_fp32_sum():
    # three values whose fp32 sum depends on the order: (1 + 2^-24) + 2^-24 = 1, but 1 + (2^-24 + 2^-24) > 1
    a = torch.tensor([1.0], dtype=torch.float32)
    b = torch.tensor([2.0 ** -24], dtype=torch.float32)
    assert ep.sum_in_rank_order([a, b, b]).item() == 1.0
    assert ep.sum_in_rank_order([b, b, a]).item() == 1.0 + 2.0 ** -23


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    g = torch.Generator().manual_seed(100 + rank)
    partial = torch.randn((5, 16), generator=g, dtype=torch.float32)
    partial[rank] = 0.0                                          # a token with no resident kept expert on this rank
    ordered = ep.reduce_partials(partial, ordered=True)
    allred = ep.reduce_partials(partial, ordered=False)
    out[rank] = (partial, ordered, allred)
    dist.barrier()
    dist.destroy_process_group()


def test_reduction_of_partial_outputs_two_ranks():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
        res = dict(out)
    parts = [res[r][0] for r in range(world)]
    want = ep.sum_in_rank_order(parts)
    for r in range(world):
        assert torch.equal(res[r][1], want)                     # the ordered form is bitwise the rank-order sum
        assert torch.allclose(res[r][2], want, rtol=0, atol=1e-6)
    assert torch.equal(res[0][1], res[1][1])


def test_single_process_reduction_is_identity():
    x = torch.arange(6, dtype=torch.float32).view(2, 3)
    assert torch.equal(ep.reduce_partials(x), x)
