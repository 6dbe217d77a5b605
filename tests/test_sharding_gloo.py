"""Whole-block sharding over ranks (host logic), run as two gloo processes on
the CPU: each rank steps only its own blocks with the float64 oracle, the
results are gathered, and must equal the unsharded run bit for bit."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import step as ostep
from paper_2406_16793_b200 import sharding, workloads as W

HP = dict(lr=1e-3, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.1)


def small_model():
    return W.Workload("mini-llama", 31, W.llama_like(2, 64, 4, 2, 176, 96, grad_dtype=W.BF16),
                      W.GradRecipe(-4.0, -1.0), steps=3)


@pytest.mark.parametrize("world", [1, 2, 3, 8])
def test_pieces_tile_every_tensor_once_and_balance(world):
    for w in (small_model(), W.llama2_7b(), W.flat_sweep(1 << 30), W.flat_sweep(128, numel=1 << 20)):
        shards = sharding.shard_by_blocks(w.tensors, world)
        assert len(shards) == world
        flat = [p for r in shards for p in r]
        cursor = {}
        for p in flat:                                    # table order, contiguous, whole blocks
            assert p.block_begin == cursor.get(p.tensor, 0) and p.block_end > p.block_begin
            cursor[p.tensor] = p.block_end
            assert p.block_len == w.tensors[p.tensor].block_len
        assert cursor == {i: t.n_blocks for i, t in enumerate(w.tensors)}
        assert [p.tensor for p in flat] == sorted(p.tensor for p in flat)
        loads = [sum(p.numel for p in r) for r in shards]
        assert sum(loads) == w.numel
        biggest_block = max(t.block_len for t in w.tensors)
        assert max(loads) - min(loads) <= 2 * biggest_block + world


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, result_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = small_model()
    mine = sharding.shard_by_blocks(w.tensors, world)[rank]
    # every rank draws the full (seeded) inputs and keeps only its blocks
    state = []
    for piece in mine:
        p0 = W.gen_param(w, piece.tensor)[piece.elem_begin:piece.elem_end]
        state.append([ostep.widen(p0), np.zeros(piece.numel), np.zeros(piece.block_end - piece.block_begin)])
    for step in range(1, w.steps + 1):
        for piece, st in zip(mine, state):
            g = W.gen_grad(w, piece.tensor, step)[piece.elem_begin:piece.elem_end].contiguous()
            spec = piece.spec(w.tensors[piece.tensor])
            ostep.adammini_step(st[0], st[1], st[2], g, spec.block_len, step=step,
                                apply_wd=bool(spec.apply_weight_decay), **HP)
    # gather (what a trainer's all-gather of updated parameters would do)
    payload = [(piece.tensor, piece.elem_begin, piece.v_begin, st[0], st[1], st[2]) for piece, st in zip(mine, state)]
    gathered = [None] * world
    dist.all_gather_object(gathered, payload)
    if rank == 0:
        torch.save(gathered, os.path.join(result_dir, "gathered.pt"))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_equal_the_unsharded_step(tmp_path):
    world = 2
    mp.spawn(_rank_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    gathered = torch.load(os.path.join(tmp_path, "gathered.pt"), weights_only=False)
    w = small_model()
    ref = ostep.OracleState([W.gen_param(w, i) for i in range(len(w.tensors))],
                            [t.block_len for t in w.tensors], [bool(t.apply_weight_decay) for t in w.tensors])
    for step in range(1, w.steps + 1):
        ref.step([W.gen_grad(w, i, step) for i in range(len(w.tensors))], step, **HP)
    v_all = np.concatenate(ref.v)
    seen = 0
    for rank_payload in gathered:
        assert rank_payload, "a rank owned nothing"
        for tensor, e0, v0, p, m, v in rank_payload:
            assert np.array_equal(p, ref.p[tensor][e0:e0 + p.size])
            assert np.array_equal(m, ref.m[tensor][e0:e0 + m.size])
            assert np.array_equal(v, v_all[v0:v0 + v.size])
            seen += p.size
    assert seen == w.numel


# ----------------------------------------------------------------------------
# flat shards that cut blocks: tiling, and the one exchange of partial sums
# ----------------------------------------------------------------------------
def odd_model():
    T = W.TensorSpec
    tensors = W.llama_like(1, 64, 4, 2, 176, 96, grad_dtype=W.BF16) + [
        T("odd.rows", 9, 1001, W.ROWS, grad_dtype=W.BF16), T("odd.short", 50, 36, W.ROWS, grad_dtype=W.F32),
        T("odd.whole", 1, 7777, W.WHOLE, grad_dtype=W.F32)]
    return W.Workload("odd", 32, tensors, W.GradRecipe(-4.0, -1.0), steps=2)


@pytest.mark.parametrize("world", [1, 2, 3, 7, 16])
def test_flat_pieces_tile_and_parts_stay_inside_one_block(world):
    for w in (small_model(), odd_model(), W.llama2_7b(n_layers=2), W.flat_sweep(1 << 30)):
        shards = sharding.shard_flat(w.tensors, world)
        cursor = {}
        for r in shards:
            for p in r:
                t = w.tensors[p.tensor]
                assert p.elem_begin == cursor.get(p.tensor, 0) and p.elem_end > p.elem_begin
                cursor[p.tensor] = p.elem_end
                assert p.block_len == t.block_len
                if p.part:
                    assert p.elem_begin // t.block_len == (p.elem_end - 1) // t.block_len == p.block
                else:
                    assert p.elem_begin % t.block_len == 0 and p.elem_end % t.block_len == 0
                    item = 2 if t.grad_dtype == W.BF16 else 4
                    assert (p.elem_begin * item) % 16 == 0                     # whole-block runs stay 16-byte aligned
        assert cursor == {i: t.numel for i, t in enumerate(w.tensors)}
        loads = [sum(p.numel for p in r) for r in shards]
        assert max(loads) - min(loads) <= 16


def _flat_rank_main(rank, world, port, result_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = odd_model()
    plan = sharding.FlatExchangePlan(w.tensors, world, rank)
    grads = [ostep.widen(W.gen_grad(w, i, 1)) for i in range(len(w.tensors))]
    local = torch.zeros(plan.max_parts, dtype=torch.float64)
    k = 0
    for p in plan.pieces:
        if p.part:
            g = grads[p.tensor][p.elem_begin:p.elem_end]
            local[k] = float((g * g).sum())
            k += 1
    gathered = sharding.all_gather_exchange(local)                      # the step's one exchange, as the GPU path calls it
    assert gathered.shape == (world, plan.max_parts) and torch.equal(gathered[rank], local)
    totals = plan.combine(gathered)
    torch.save((plan.part_keys, totals[:plan.n_parts]), os.path.join(result_dir, f"rank{rank}.pt"))
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
def test_exchange_gives_every_holder_the_whole_block_sum(tmp_path, world):
    mp.spawn(_flat_rank_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    w = odd_model()
    grads = [ostep.widen(W.gen_grad(w, i, 1)) for i in range(len(w.tensors))]
    seen = {}
    for rank in range(world):
        keys, totals = torch.load(os.path.join(tmp_path, f"rank{rank}.pt"), weights_only=False)
        for (tensor, block), tot in zip(keys, totals.tolist()):
            L = w.tensors[tensor].block_len
            g = grads[tensor][block * L:(block + 1) * L]
            want = float((g * g).sum())
            assert abs(tot - want) <= 1e-12 * want
            assert seen.setdefault((tensor, block), tot) == tot             # every holder has the same bits
    assert seen, "no block was cut"
