"""The paper's 2-D example (Appendix) run end to end: gradient steps on the host, the population
operators through the library, against the same loop with the oracle's operators."""
import numpy as np
import pytest

import oracle
from paper_2405_17517_b200 import toy2d

pytestmark = pytest.mark.gpu


class OracleOps:
    def __init__(self):
        self.pop = oracle.Population(2, [2], [0], toy2d.ROW, 0)

    def shuffle(self, stack, step, p, seed):
        oracle.shuffle(self.pop, stack.reshape(-1), p, seed, step)

    def ema(self, stack, alpha):
        oracle.papa_ema(self.pop, stack.reshape(-1), alpha)


@pytest.mark.parametrize("method,noise", [("wash", 0.0), ("wash", 0.5), ("papa", 0.5)])
def test_trajectories_are_bit_identical_to_the_oracles(method, noise):
    lib = toy2d.LibraryOps()
    got, want = [], []
    end = toy2d.run(method, lib, noise=noise, seed=3, steps=400, p=0.05, trace=got)
    ref = toy2d.run(method, OracleOps(), noise=noise, seed=3, steps=400, p=0.05, trace=want)
    lib.close()
    assert all((a == b).all() for a, b in zip(got, want))
    assert (end.view(np.uint32) == ref.view(np.uint32)).all()


def test_shuffling_moves_both_models_out_of_their_local_minima():
    """Without noise the only randomness is the shuffle: apart, the models stop in (3, 8) and (8, 3);
    with WASH both reach the global minimum at (10, 10) (the picture of the paper's 2-D example)."""
    lib = toy2d.LibraryOps()
    apart = toy2d.run("baseline", lib)
    wash = toy2d.run("wash", lib)
    lib.close()
    assert np.abs(apart[0] - (3, 8)).max() < 0.2 and np.abs(apart[1] - (8, 3)).max() < 0.2
    assert np.abs(wash - 10.0).max() < 0.2
    assert toy2d.loss(*wash[0]) < toy2d.loss(*apart[0]) and toy2d.loss(*wash[1]) < toy2d.loss(*apart[1])
