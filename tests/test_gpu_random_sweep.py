"""Seeded random sweep of verify calls (chains and candidate trees) on the two small shapes:
batch 1-4, with and without guidance, 1-3 forced rows, 0-12 drafts, fill levels drawn over the
whole cache including empty and exactly-full, drafters near to and far from the target.  Every
case goes through the same end-to-end and replay checks as the hand-picked ones."""
import numpy as np
import pytest

import helpers as H
from test_gpu_tree import _check_tree
from test_gpu_verify import _check_end_to_end
from vvs_synth.configs import B7_SMALL, XL_SMALL

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("sweep_seed", [1, 7])
def test_random_chain_and_tree_calls(sweep_seed):
    rng = np.random.default_rng(sweep_seed)
    paths = {"chain": 0, "tree": 0, "whole_chain_kernel": 0, "per_projection": 0}
    for i in range(20):
        ms = XL_SMALL if rng.random() < 0.7 else B7_SMALL
        n_images, n_cfg = int(rng.integers(1, 5)), int(rng.integers(1, 3))
        f, k = int(rng.integers(1, 4)), int(rng.integers(0, 13))
        t_len = f + k
        fills = [int(x) for x in rng.integers(0, ms.s_max - t_len + 1, size=n_images)]
        if rng.random() < 0.2:
            fills[0] = ms.s_max - t_len
        if rng.random() < 0.2:
            fills[-1] = 0
        tree = rng.random() < 0.5 and k > 0
        cfg_scale = 2.0 if n_cfg == 2 else 1.0
        q_noise = float(rng.choice([0.3, 1.0, 2.5]))
        seed = 5000 * sweep_seed + i
        if tree:
            parent = [-1] + list(range(f - 1)) + [int(rng.integers(f - 1, c)) for c in range(f, t_len)]
            case = H.build_tree_case(ms, seed, n_images, n_cfg, f, parent, fills, cfg_scale=cfg_scale, q_noise=q_noise)
            run = H.GpuRunner(ms, case["w"], n_images * n_cfg, t_len, deterministic=bool(i & 1), chain_kernels=bool(i & 2))
            gpu = H.run_tree_gpu(run, case)
            _check_tree(case, gpu, H.run_tree_oracle(case))
        else:
            case = H.build_case(ms, seed, n_images, n_cfg, f, k, fills, cfg_scale=cfg_scale, q_noise=q_noise)
            run = H.GpuRunner(ms, case["w"], n_images * n_cfg, t_len, deterministic=bool(i & 1), chain_kernels=bool(i & 2))
            gpu = run.verify(case)
            _check_end_to_end(case, gpu, H.run_oracle(case))
        run.close()
        paths["tree" if tree else "chain"] += 1
        paths["whole_chain_kernel" if gpu["launches"] < 20 else "per_projection"] += 1
    print("sweep", sweep_seed, paths)
    assert min(paths.values()) > 0          # the sweep reaches both kinds of call and both kernel paths


def test_random_relaxed_and_ragged_calls():
    """Relaxed acceptance with 1-64 neighbours and thresholds from 0 to infinity, ragged draft
    counts (including images with no draft at all), up to five images."""
    from vvs_synth.configs import MODE_RELAXED, MODE_STRICT
    rng = np.random.default_rng(3)
    n_relaxed = 0
    for i in range(16):
        ms = XL_SMALL if rng.random() < 0.7 else B7_SMALL
        n_images, n_cfg = int(rng.integers(1, 6)), int(rng.integers(1, 3))
        f, k = int(rng.integers(1, 4)), int(rng.integers(1, 13))
        t_len = f + k
        fills = [int(x) for x in rng.integers(0, ms.s_max - t_len + 1, size=n_images)]
        relaxed = rng.random() < 0.6
        nbr_k = int(rng.choice([1, 4, 16, 64])) if relaxed else 1
        delta = float(rng.choice([0.0, 0.05, 0.3, np.inf])) if relaxed else float("inf")
        n_draft = [int(x) for x in rng.integers(0, k + 1, size=n_images)]
        case = H.build_case(ms, 9000 + i, n_images, n_cfg, f, k, fills, cfg_scale=2.0 if n_cfg == 2 else 1.0,
                            mode=MODE_RELAXED if relaxed else MODE_STRICT, nbr_k=nbr_k, delta=delta,
                            q_noise=float(rng.choice([0.3, 1.0, 2.5])), n_draft=n_draft)
        run = H.GpuRunner(ms, case["w"], n_images * n_cfg, t_len, max_nbr_k=nbr_k)
        gpu = run.verify(case)
        _check_end_to_end(case, gpu, H.run_oracle(case))
        assert (gpu["accept_len"] <= np.asarray(n_draft)).all()
        run.close()
        n_relaxed += int(relaxed)
    assert 0 < n_relaxed < 16
