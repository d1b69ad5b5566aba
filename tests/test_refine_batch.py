"""CPU: integer refinement of the TPOT-feasible batch against brute force on synthetic monotone curves."""
import importlib.util
import os
import random

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _load(pdlib):
    import paper_2603_04716_b200.configs as cfgs
    return cfgs


def test_refinement_finds_largest_feasible_integer(pdlib):
    cfgs = _load(pdlib)
    rnd = random.Random(5)
    for _ in range(200):
        a, b0 = rnd.uniform(1e-5, 2e-4), rnd.uniform(1e-3, 5e-3)
        curve = lambda b: b0 + a * b                         # TPOT grows with the batch
        sweep = [1, 2, 4, 8, 16, 32, 64, 128, 256, 512]
        tp = [curve(b) for b in sweep]
        slo = rnd.uniform(b0 + a, b0 + 600 * a)
        calls = []
        b_all, t_all, probes = cfgs.refine_feasible_batch(lambda b: (calls.append(b), curve(b))[1], sweep, tp, slo,
                                                          max_probes=12)
        got = pdlib.pd_allocate(1e5, 512, 512, 2.0, slo, 5e4, b_all, t_all)["feasible_batch"]
        feas = [b for b in range(1, 513) if curve(b) <= slo]
        if not feas:
            assert got == 0 and not calls
        elif max(feas) == 512:
            assert got == 512 and not calls            # capped by the sweep: nothing to refine
        else:
            assert got == max(feas) and t_all[b_all.index(got)] == curve(got)
            assert len(calls) <= 9 and [p[0] for p in probes] == calls
