"""The multi-rank plumbing on CPU: two gloo ranks shard the tokens, share the parameters, and agree on
the max-over-ranks time and the whole-job throughput."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp


def _free_port():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); p = s.getsockname()[1]; s.close(); return p


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    from paper_2601_05732_b200 import dist as D, synth
    assert D.env_rank_world() == (rank, rank, world)
    D.init(world, backend="gloo")
    inp = synth.make_layer_inputs(4, 16, 8, seed=1, bias_std=0.1, shard=D.shard_of(rank))
    D.barrier(world, cuda=False)
    ms = D.max_over_ranks(10.0 + 5.0 * rank, world)            # rank 1 is the slow one
    value = D.job_tokens_per_s(8, world, steps=3, ms_max=ms)
    # parameters identical across ranks, tokens different
    w = torch.from_numpy(inp["W"].copy()); x = torch.from_numpy(inp["x"].astype(np.int32))
    ws = [torch.empty_like(w) for _ in range(world)]; xs = [torch.empty_like(x) for _ in range(world)]
    torch.distributed.all_gather(ws, w); torch.distributed.all_gather(xs, x)
    out.put((rank, ms, value, bool((ws[0] == ws[1]).all()), bool((xs[0] == xs[1]).all())))
    D.shutdown()


def test_two_gloo_ranks_shard_tokens_and_take_max_time():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, value, same_w, same_x in res:
        assert ms == 15.0                                        # max over ranks, on every rank
        assert value == pytest.approx(2 * 8 * 3 / 15e-3)        # all ranks' tokens over the slowest time
        assert same_w and not same_x


def _grad_worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    from oracle import mhclite_oracle as O
    from paper_2601_05732_b200 import dist as D, synth
    D.init(world, backend="gloo")
    inp = synth.make_layer_inputs(3, 8, 5, seed=2, bias_std=0.1, shard=D.shard_of(rank))
    f = synth.bf16_bits_to_f64
    w = [inp[k].astype(np.float64) for k in ("W", "b", "alpha", "gain")]
    bw = O.layer_bwd(f(inp["x"]), f(inp["y"]), *w, 1e-6, f(inp["g"]), f(inp["du"]))
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.float64))
    dW, db, dal, dg = t(bw["dW"]), t(bw["db"]), t(bw["dalpha"]), t(bw["dgain"])
    mine = [x.clone() for x in (dW, db, dal, dg)]
    bucket = D.all_reduce_param_grads(dW, db, dal, dg, world)
    out.put((rank, [m.numpy() for m in mine], [x.numpy().copy() for x in (dW, db, dal, dg)], bucket.numel()))
    D.shutdown()


def test_parameter_gradients_sum_over_token_shards():
    # data parallelism over tokens: each rank's dW, db, dalpha, dgain cover its shard; one all-reduce sums them
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_grad_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted((q.get(timeout=120) for _ in range(world)), key=lambda r: r[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (_, mine0, red0, n0), (_, mine1, red1, n1) = res
    assert n0 == n1 == sum(m.size for m in mine0)
    for a0, a1, r0, r1 in zip(mine0, mine1, red0, red1):
        assert not np.array_equal(a0, a1)                       # different token shards
        np.testing.assert_allclose(r0, a0 + a1, rtol=1e-14, atol=0)
        np.testing.assert_array_equal(r0, r1)                   # every rank ends with the same sum


def test_single_process_defaults():
    from paper_2601_05732_b200 import dist as D
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE"):
        os.environ.pop(k, None)
    assert D.env_rank_world() == (0, 0, 1)
    assert D.max_over_ranks(3.5, 1) == 3.5
    assert D.job_tokens_per_s(100, 1, 2, 4.0) == 50000.0
    assert D.all_reduce_param_grads(torch.zeros(2, 2), torch.zeros(2), torch.zeros(3), torch.zeros(2), 1) is None
