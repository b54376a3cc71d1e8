"""The extensions work together: sampled episodes, simulated run times,
advantages, the policy gradient and an Adam step, all on the device, lower the
mean simulated run time of a small graph (the REINFORCE loop of the paper's
Appendix A.1 with a terminal reward). This checks the sign and the wiring of
the whole chain, not a learning curve: a loose bound on a seeded run."""
from __future__ import annotations

import numpy as np
import pytest

from paper_1906_08879_b200.examples import reinforce_demo

pytestmark = pytest.mark.gpu


def test_reinforce_lowers_the_simulated_run_time():
    history = reinforce_demo.train(reinforce_demo.demo_config(), iterations=40)
    first, last = np.mean(history[:3]), np.mean(history[-3:])
    assert np.isfinite(history).all()
    assert last < 0.9 * first, (first, last)
