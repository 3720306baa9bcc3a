"""Data parallelism over tokens on the CUDA path (paper Appendix A: DDP): each rank runs the library's
forward + backward on its own token shard, the ranks sum their parameter gradients with one all-reduce,
and the sum equals the oracle's gradient over all tokens.  The two ranks are two processes that share the
one GPU of the test box (their kernels never wait on one another; the exchange runs over gloo)."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

pytestmark = pytest.mark.gpu


def _free_port():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); p = s.getsockname()[1]; s.close(); return p


def _rank(rank, world, port, n, C, T, seed, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK="0", WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    from paper_2601_05732_b200 import dist as D, layer as L, synth
    from paper_2601_05732_b200.binding import MhcLite
    D.init(world, backend="gloo")
    dev = "cuda:0"
    inp = synth.make_layer_inputs(n, C, T, seed, bias_std=0.1, gain_std=0.1, shard=D.shard_of(rank))
    ctx = MhcLite(n, C, 0)
    P = L.LayerParams(inp["W"], inp["b"], inp["alpha"], inp["gain"], dev)
    B = L.LayerBuffers(ctx, T)
    x, y, g, du = (L.to_device_bf16(inp[k], dev) for k in ("x", "y", "g", "du"))
    L.pre_fwd(ctx, P, B, x); L.post_fwd(ctx, B, x, y)
    L.post_bwd(ctx, B, x, y, g); L.tail_bwd(ctx, P, B, x, g, du)
    torch.cuda.synchronize()
    ctx.device_status()
    mine = [t.detach().cpu().numpy().copy() for t in (B.dW, B.db, B.dalpha, B.dgain)]
    D.all_reduce_param_grads(B.dW, B.db, B.dalpha, B.dgain, world)     # CUDA tensors through gloo
    torch.cuda.synchronize()
    red = [t.detach().cpu().numpy().copy() for t in (B.dW, B.db, B.dalpha, B.dgain)]
    out.put((rank, mine, red))
    D.barrier(world)
    D.shutdown()


@pytest.mark.parametrize("n,C,T", [(4, 256, 1000), (5, 64, 300)])
def test_two_gpu_ranks_all_reduce_matches_full_batch_oracle(n, C, T):
    from oracle import mhclite_oracle as O
    from paper_2601_05732_b200 import synth
    from parity_utils import check_f32
    world, port, seed = 2, _free_port(), 90 + n
    mpc = mp.get_context("spawn")
    q = mpc.Queue()
    procs = [mpc.Process(target=_rank, args=(r, world, port, n, C, T, seed, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted((q.get(timeout=600) for _ in range(world)), key=lambda r: r[0])
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    # the oracle over the full batch: both shards' tokens, one set of parameters
    f = synth.bf16_bits_to_f64
    shards = [synth.make_layer_inputs(n, C, T, seed, bias_std=0.1, gain_std=0.1, shard=r) for r in range(world)]
    cat = lambda k: np.concatenate([f(s[k]) for s in shards], axis=0)
    w = [shards[0][k].astype(np.float64) for k in ("W", "b", "alpha", "gain")]
    bw = O.layer_bwd(cat("x"), cat("y"), *w, 1e-6, cat("g"), cat("du"))
    for rank, mine, red in res:
        for name, got in zip(("dW", "db", "dalpha", "dgain"), red):
            check_f32(f"{name} summed over shards (rank {rank})", got.astype(np.float64), bw[name], 1e-3)
    for a, b in zip(res[0][2], res[1][2]):
        np.testing.assert_array_equal(a, b)                      # every rank ends with the same sum
    assert not np.array_equal(res[0][1][0], res[1][1][0])        # the shards' own gradients differ
