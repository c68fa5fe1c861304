"""Pins for the host cost evaluator and fit against numbers the paper prints (no GPU)."""
import os

import numpy as np

from paper_2608_13057_b200 import costmodel as C

GOLD = {}
with open(os.path.join(os.path.dirname(__file__), "golden", "paper_cost_numbers.txt")) as fh:
    for line in fh:
        line = line.split("#")[0].split()
        if line:
            GOLD[line[0]] = [float(v) for v in line[1:]]


def test_figure_1b_toy_batch():
    b, beta = GOLD["fig1b_b"][0], GOLD["fig1b_beta"][0]
    hot, cold = 600, 30
    token_bal = [[hot // 2] + [cold // 2] * 6] * 2                 # everything split: 7 floors per GPU
    act_bal = [[hot, cold, cold, cold], [cold, cold, cold]]        # whole experts, 4 vs 3
    time_bal = [[hot // 2, cold, cold, cold]] * 2                  # only the hot expert split
    t_tok = C.makespan(0, b, 0, beta, token_bal)
    t_act = C.makespan(0, b, 0, beta, act_bal)
    t_time = C.makespan(0, b, 0, beta, time_bal)
    assert abs(t_tok - GOLD["fig1b_token_balancing_us"][0]) < 1e-9
    assert abs(t_act - GOLD["fig1b_activation_balancing_us"][0]) < 1e-9
    assert abs(t_time - GOLD["fig1b_time_balancing_us"][0]) < 1e-9
    assert abs(t_tok / t_time - GOLD["fig1b_ratio"][0]) < 1e-9


def test_n_star_reproduces_the_printed_table():
    for key in ("tab_params_qwen3_30b", "tab_params_dsv2_lite", "tab_params_dsv3", "tab_params_dsv3_bf16"):
        b, beta, printed = GOLD[key]
        assert abs(C.n_star(b, beta) - printed) <= 1.0            # the table rounds ("approximately")


def test_weight_bytes_formula_and_win_boundary():
    assert abs(3 * 7168 * 2048 / 1e6 - GOLD["dsv3_expert_mbytes"][0]) < 0.05
    assert round((16.4 + 2.99 * 13 - 25.0) / 0.10) == GOLD["bstar_a2a_tokens"][0]


def test_tile_term_counts_extra_tiles_only():
    # Eq. 3: T - G extra tiles; decode region (every instance <= 128 rows) is untouched by b2
    assert C.tiles_of([1, 128, 129, 256, 0]) == 1 + 1 + 2 + 2
    t0 = C.block_time(34.9, 3.95, 34.8, 0.0154, 8, 8 * 100)
    t1 = C.block_time(34.9, 3.95, 34.8, 0.0154, 8, 8 * 100, b2=1.23, tiles=8)
    assert t0 == t1
    t2 = C.block_time(34.9, 3.95, 34.8, 0.0154, 8, 8 * 129, b2=1.23, tiles=16)
    assert abs(t2 - (34.9 + 3.95 * 8 + 1.23 * 8)) < 1e-9


def test_fit_recovers_a_planted_profile():
    Gs = np.array([1, 2, 4, 8, 16, 32, 64])
    Ns = np.array([1, 8, 32, 64, 128, 129, 160, 192, 256, 512, 1024, 2048, 4096])
    G, n = [a.reshape(-1) for a in np.meshgrid(Gs, Ns, indexing="ij")]
    N = G * n
    tiles = G * -(-n // 128)
    t = C.block_time(35.0, 4.0, 30.0, 0.016, G, N)
    fit = C.fit_max_affine(G, N, t)
    assert abs(fit["b"] - 4.0) < 1e-6 and abs(fit["beta"] - 0.016) < 1e-9 and fit["fit_err"] < 1e-9
    assert abs(fit["n_star"] - 250.0) < 1e-3
    t = C.block_time(35.0, 4.0, 30.0, 0.016, G, N, b2=1.3, tiles=tiles)
    fit = C.fit_max_affine(G, N, t, tiles=tiles, tile_aware=True)
    assert abs(fit["b"] - 4.0) < 1e-6 and abs(fit["b2"] - 1.3) < 1e-6 and fit["fit_err"] < 1e-9
