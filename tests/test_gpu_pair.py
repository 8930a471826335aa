"""GPU parity of the CTA-pair attention kernel (tcgen05.mma with cta_group::2), selected explicitly: the same oracle
comparison as the other attention paths, on the five configurations, ragged and tree-shaped batches."""
import numpy as np
import pytest

from lr_workloads import make_config, make_random_mid, make_random_small, make_random_tree, make_tree
from paper_2506_19830_b200 import binding as B

from gpu_util import REL_LARGE, run_and_check_pass

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("cfg", [2, 3, 4, 5])
def test_configs(cfg):
    run_and_check_pass(make_config(cfg), path=B.PATH_PAIR)


@pytest.mark.parametrize("cfg", [2, 5])
def test_configs_with_the_carry_in_token(cfg):
    run_and_check_pass(make_config(cfg, carry_in=True), path=B.PATH_PAIR)


@pytest.mark.parametrize("seed", list(range(12)))
def test_ragged_small(seed):
    run_and_check_pass(make_random_small(1000 + seed, head_dim=128), path=B.PATH_PAIR, rel_large=REL_LARGE)


@pytest.mark.parametrize("seed", list(range(6)))
def test_random_trees(seed):
    run_and_check_pass(make_random_tree(600 + seed, head_dim=128), path=B.PATH_PAIR, rel_large=REL_LARGE)


@pytest.mark.parametrize("W,gamma,size", [(2, 3, "layer"), (2, 2, "serving")])
def test_full_trees(W, gamma, size):
    run_and_check_pass(make_tree(W, gamma, size=size), path=B.PATH_PAIR)


def test_mid_size_batches():
    for seed in range(6):
        w = make_random_mid(seed)
        if w.batch.model.head_dim != 128:
            continue
        rng = np.random.Generator(np.random.PCG64(seed))
        pick = sorted(set(int(x) for x in rng.integers(0, w.batch.n_branch, size=min(3, w.batch.n_branch))))
        run_and_check_pass(w, path=B.PATH_PAIR, check_rows_of_branches=pick, rel_large=REL_LARGE)
