"""The whole loop on the GPU (rollout -> GAE -> PPO gradient -> Adam, evaluation blocks in between) learns the task.

Parity ties every block to the oracle; this ties the blocks together and their signs to the task itself: on the
small level-based-foraging workload a randomly initialised policy collects almost nothing, and a few dozen
iterations of the loop must raise the mean greedy return substantially (1.0 = every food item collected).
All seeds are fixed, so the run is reproducible.
"""
import pytest

from paper_2107_01460_b200 import binding, train

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("precision", [binding.MAVA_PRECISION_BF16, binding.MAVA_PRECISION_FP32])
def test_the_loop_learns_to_forage(precision):
    history = train.train(workload=1, n_envs=512, T=64, iters=60, epochs=4, lr=1e-3, eval_every=30, precision=precision,
                          log=lambda *_: None)
    first, last = history[0][1], history[-1][1]
    assert first < 0.05, history
    assert last > 0.5, history
    assert all(b[1] >= a[1] - 0.05 for a, b in zip(history, history[1:])), history


def test_the_loop_improves_the_mappo_shape_too():
    """15x15, four agents, five food items, centralised critic: a harder task, so only a clear improvement is asked."""
    history = train.train(workload=3, n_envs=512, T=64, iters=60, epochs=4, lr=1e-3, eval_every=60, log=lambda *_: None)
    assert history[0][1] < 0.01 and history[-1][1] > 0.04, history
