"""Repetition code on many small random cases, including more adversaries than the code tolerates: the selected
values, the flags and the count of coordinates without a majority must equal the oracle's bit for bit on the same
received matrix, whatever the adversaries did (Algorithm 2 is deterministic)."""
import numpy as np
import pytest
import torch

import draco_inputs as di
from oracle import draco_oracle as orc
from gpu_util import dev, host

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("stream_seed", [21, 22])
def test_random_small_cases_match_the_oracle_bit_for_bit(stream_seed):
    import paper_1803_09877_b200 as dr
    rng = np.random.default_rng(stream_seed)
    for case in range(60):
        n = int(rng.integers(3, 70))
        s = int(rng.integers(0, min(9, (n - 1) // 2) + 1))
        n_adv = int(rng.integers(0, min(n, s + 3) + 1))              # up to two more than tolerated
        d = int(rng.choice([255, 1000, 4096, 10001]))
        seed = int(rng.integers(1, 1 << 30))
        G = di.gradient_rows(seed, n, d)
        R = orc.rep_encode(G, n, s)
        adv = di.choose_adversaries(seed + 1, n, n_adv) if n_adv else np.zeros(0, dtype=np.int32)
        if n_adv:
            # constant adversaries collude (identical values); the other two models give every adversary its own values
            model = [int(rng.choice([di.ADV_REVGRAD, di.ADV_CONST, di.ADV_GAUSS])) for _ in range(n_adv)]
            param = [{di.ADV_REVGRAD: 100.0, di.ADV_CONST: 1e4, di.ADV_GAUSS: 1e3}[m] for m in model]
            di.apply_adversaries(R, adv, model, param, seed=seed + 2)
        want = orc.rep_decode(R, n, s)
        plan = dr.Plan(n, s, d, dr.REP)
        g = len(orc.rep_groups(n, s))
        u = torch.empty(d, dtype=torch.float32, device="cuda")
        maj = torch.empty((g, d), dtype=torch.float32, device="cuda")
        flags = torch.full((n,), 7, dtype=torch.uint8, device="cuda")
        plan.rep_vote(dev(R), u, maj, flags)
        info = plan.info()
        what = f"case {case}: n={n} s={s} adv={adv.tolist()} d={d} seed={seed}"
        np.testing.assert_array_equal(host(maj).view(np.uint32), want["maj"].view(np.uint32), err_msg=what)
        np.testing.assert_array_equal(host(flags).astype(bool), want["flags"], err_msg=what)
        assert info["no_majority"] == want["no_majority"], what
        seq = np.zeros(d, dtype=np.float32)
        for row in want["maj"]:                                       # groups ascending, fp32
            seq = seq + row
        np.testing.assert_array_equal(host(u).view(np.uint32), seq.view(np.uint32), err_msg=what)
        plan.close()
