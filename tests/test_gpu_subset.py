"""The subset-of-permutations variant (paper Section 5, "larger n"): Eq. (5) over K sampled permutation
matrices given as a device table, against the oracle's `table` route, element by element."""
import math

import numpy as np
import pytest
import torch

from oracle import mhclite_oracle as O
from paper_2601_05732_b200 import synth
from paper_2601_05732_b200.binding import MhcLite, ERR_BAD_ARG
from parity_utils import DEV, GpuLayer, check_bf16, compare_backward, compare_forward, host, oracle_bwd, oracle_fwd

pytestmark = pytest.mark.gpu

CASES = [  # (n, K, C, T)
    (5, 8, 256, 333), (5, 24, 320, 700), (5, 64, 136, 161), (5, 120, 64, 70), (4, 7, 256, 300), (4, 16, 1024, 257),
    (3, 2, 72, 130), (2, 1, 64, 50),
]


@pytest.mark.parametrize("n,K,C,T", CASES)
@pytest.mark.parametrize("fused", [True, False])
def test_subset_layer_parity(n, K, C, T, fused):
    tab = synth.sample_perm_table(n, K, seed=200 + K)
    inp = synth.make_layer_inputs(n, C, T, seed=30 + n, bias_std=0.5, alpha=[1.0, 0.7, 1.3], w_std=0.05, gain_std=0.1, n_res=K)
    G = GpuLayer(inp, table=tab)
    assert G.B.a_saved.shape == (T, K) and G.B.dW.shape == (n * C, K + 2 * n)
    G.forward(fused)
    compare_forward(G, oracle_fwd(inp, table=tab), coeff_rel=2e-4)
    Hr = host(G.B.H_res)
    assert Hr.min() >= 0 and np.abs(Hr.sum(1) - 1).max() < 1e-6 and np.abs(Hr.sum(2) - 1).max() < 1e-6
    G.backward(fused)
    compare_backward(G, oracle_bwd(inp, table=tab), grad_rel=2e-3, fused=fused)
    G.ctx.device_status()


def test_subset_at_benchmark_distribution_and_one_hot():
    # the benchmark's near-uniform logits (alpha = 0.01): the mappings at 1e-5
    n, K, C, T = 5, 24, 512, 600
    tab = synth.sample_perm_table(n, K, seed=5)
    inp = synth.make_layer_inputs(n, C, T, seed=77, bias_std=0.1, n_res=K)
    G = GpuLayer(inp, table=tab)
    G.forward(); compare_forward(G, oracle_fwd(inp, table=tab))
    G.backward(); compare_backward(G, oracle_bwd(inp, table=tab))
    # one-hot weight on row k of the table: H_res = P_k exactly, and x_next takes stream sigma_k(i) in row i
    for k in (0, 3, K - 1):
        inp1 = synth.make_layer_inputs(n, 64, 5, seed=3, n_res=K)
        inp1["W"][:] = 0; inp1["b"][:K] = -200.0; inp1["b"][k] = 0.0
        G1 = GpuLayer(inp1, table=tab); G1.forward()
        expect = np.zeros((n, n)); expect[np.arange(n), tab[k]] = 1.0
        assert (host(G1.B.H_res) == expect[None]).all(), k
        check_bf16("x_next", host(G1.B.x_next), oracle_fwd(inp1, table=tab)["x_next"])


def test_full_table_as_subset_matches_the_default_path():
    n, C, T = 4, 256, 200
    inp = synth.make_layer_inputs(n, C, T, seed=12, bias_std=0.5, alpha=[1.0, 1.0, 1.0], w_std=0.05)
    G0 = GpuLayer(inp); G0.forward(); G0.backward()
    G1 = GpuLayer(inp, table=O.perm_table(n)); G1.forward(); G1.backward()
    ref_f, ref_b = oracle_fwd(inp), oracle_bwd(inp)
    compare_forward(G1, ref_f, coeff_rel=2e-4); compare_backward(G1, ref_b, grad_rel=2e-3)
    assert np.abs(host(G0.B.H_res) - host(G1.B.H_res)).max() < 2e-6
    # detaching the subset restores the n! columns
    G1.ctx.set_perm_subset(None)
    assert G1.ctx.nfact == math.factorial(n)


def test_bad_tables_are_rejected():
    ctx = MhcLite(4, 64)
    dev = lambda rows: torch.tensor(rows, dtype=torch.uint8, device=DEV)
    lib, h = ctx.lib, ctx._h
    for rows in ([[0, 1, 2, 2]], [[0, 1, 2, 3], [0, 1, 2, 3]], [[0, 1, 2, 4]]):
        t = dev(rows)
        assert lib.mhclite_set_perm_subset(h, t.shape[0], t.data_ptr()) == ERR_BAD_ARG
    t = dev([[0, 1, 2, 3]] * 25)
    assert lib.mhclite_set_perm_subset(h, 25, t.data_ptr()) == ERR_BAD_ARG          # K > n!
    good = dev([[1, 0, 3, 2], [0, 1, 2, 3]])
    assert lib.mhclite_set_perm_subset(h, 2, good.data_ptr()) == 0
    assert lib.mhclite_workspace_bytes_subset(4, 64, 1000, 2) > 0
    assert lib.mhclite_workspace_bytes_subset(4, 64, 1000, 25) == 0
