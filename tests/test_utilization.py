"""Compute-utilisation model (the paper's Sec. 5.2 simulator): oracle pins and product parity (CPU).

The paper prints the simulator's outputs (Table 1, the appendix ablation table, three sentences of
Sec. 5.2) but not its two inputs, the step time and the payload size.  The pins: fit exactly those
two constants -- the step time on the one absolute statement (GlobalM1, fully hidden, reaches 1 T
tokens in about 16 weeks), the payload on ONE utilisation cell (DiLoCo, M = 8, H = 100, 100 Mbps) --
and require the oracle to reproduce every other printed cell, the DiLoCo wall-clock figure and the
minimum-H statement.  A wrong transfer volume, a blocking / non-blocking mix-up, a missing factor for
the momentum or the subset, or a wrong batch scaling each break several cells.
"""
import os

import pytest

from oracle import utilization as oracle_util
from paper_2606_22768_b200 import utilization as util

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "table1_compute_utilization.txt")
WEEK = 7 * 24 * 3600.0
TOKENS_PER_STEP = 512 * 1024          # global batch 512 sequences of 1024 tokens (Sec. 5.1)


def _rows():
    out = []
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        f = line.split()
        out.append(dict(name=f[0], M=int(f[1]), H=int(f[2]), GBS=int(f[3]), mix1=f[4], mix2=f[5], frac=float(f[6]),
                        state=bool(int(f[7])), u100=float(f[8]), u200=float(f[9])))
    return out


def _fit():
    """(t_step at M = 8 / GBS = 512, payload bytes) from the two anchor statements."""
    t_step = 16 * WEEK / (1e12 / TOKENS_PER_STEP)                 # GlobalM1 at 200 Mbps runs at 100 %
    # DiLoCo, M = 8, H = 100, 100 Mbps prints 36 %: compute / (compute + all-reduce) = 0.36
    allreduce = 100 * t_step * (1 / 0.36 - 1)
    payload = allreduce / (2 * 7 / 8) * 100e6 / 8
    return t_step, payload


def _t_step(row, t8):
    return t8 * (row["GBS"] / row["M"]) / (512 / 8)               # step time follows the per-worker batch


def test_fitted_constants_are_plausible():
    t_step, payload = _fit()
    assert 4.0 < t_step < 6.0                                     # seconds per step of 64 sequences on one GPU
    assert 5.5e9 < payload < 7.5e9                                # about 1.5 B parameters in fp32
    assert payload == pytest.approx(1.5 * 2 ** 30 * 4, rel=1e-6)  # in fact 6 GiB to six digits: the two anchors agree


@pytest.mark.parametrize("row", _rows(), ids=lambda r: f"{r['name']}-M{r['M']}-H{r['H']}-GBS{r['GBS']}")
def test_oracle_reproduces_the_printed_cells(row):
    t8, payload = _fit()
    for bw, want in ((100e6, row["u100"]), (200e6, row["u200"])):
        got = 100 * oracle_util.simulate(row["mix1"], row["mix2"], row["M"], row["H"], _t_step(row, t8), payload, bw,
                                         mix2_fraction=row["frac"], state_in_mix1=row["state"])
        assert abs(got - want) <= 1.0, f"{row['name']} at {bw / 1e6:.0f} Mbps: {got:.2f} vs the printed {want}"


def test_oracle_reproduces_the_sentences_of_sec_5_2():
    t8, payload = _fit()
    # Sec. 5.2's wall-clock figures for 10^12 tokens at 200 Mbps, M = 8, H = 100: about 16 weeks (GlobalM1,
    # the anchor of the fit) against about 29 weeks for DiLoCo
    steps = 1e12 / TOKENS_PER_STEP
    u = oracle_util.simulate("none", "global", 8, 100, t8, payload, 200e6)
    assert steps * t8 / u / WEEK == pytest.approx(29, rel=0.06)
    # Sec. 5.2: Mix1 is fully hidden from about H = 180 at 100 Mbps and about H = 90 at 200 Mbps
    for bw, want in ((100e6, 180), (200e6, 90)):
        hidden = [H for H in range(1, 400) if oracle_util.simulate("global", "none", 8, H, t8, payload, bw) > 1 - 1e-12]
        assert abs(hidden[0] - want) <= 5
    # all-reduce moves at most about twice what pairwise gossip moves
    assert oracle_util.transfer_seconds("global", 8, 1.0, 1.0) / oracle_util.transfer_seconds("local", 8, 1.0, 1.0) == pytest.approx(1.75)
    # failures: DiLoCo degrades, LocalM1M2 is unaffected
    base = oracle_util.simulate("none", "global", 8, 100, t8, payload, 200e6)
    hurt = oracle_util.simulate("none", "global", 8, 100, t8, payload, 200e6, p_fail=0.05, rounds=4000, seed=1)
    assert hurt < base - 0.02
    assert oracle_util.simulate("local", "local", 8, 100, t8, payload, 200e6, p_fail=0.05, rounds=50, seed=1) == \
        pytest.approx(oracle_util.simulate("local", "local", 8, 100, t8, payload, 200e6), rel=1e-13)


# ------------------------------------------------------------------ the library's closed form against the oracle
KINDS = ("none", "local", "global")


@pytest.mark.parametrize("M,H,bw", [(8, 100, 100e6), (8, 500, 200e6), (16, 100, 100e6), (4, 37, 1e9), (8, 100, 50e6)])
def test_closed_form_equals_the_timeline_without_failures(M, H, bw):
    t8, payload = _fit()
    for mix1 in KINDS:
        for mix2 in KINDS:
            for frac, state in ((1.0, False), (0.43, False), (1.0, True), (0.43, True)):
                d = util.Deployment(M, H, t8, payload, bw, t_outer=0.7)
                got = util.utilization(mix1, mix2, d, mix2_fraction=frac, state_in_mix1=state)
                ref = oracle_util.simulate(mix1, mix2, M, H, t8, payload, bw, t_outer=0.7, mix2_fraction=frac,
                                           state_in_mix1=state, rounds=3)
                assert got == pytest.approx(ref, rel=1e-12)


@pytest.mark.parametrize("mix1,mix2", [("none", "global"), ("global", "none"), ("global", "local"), ("global", "global"), ("local", "local")])
def test_closed_form_expectation_under_failures(mix1, mix2):
    t8, payload = _fit()
    d = util.Deployment(8, 100, t8, payload, 200e6)
    got = util.utilization(mix1, mix2, d, p_fail=0.05)
    ref = oracle_util.simulate(mix1, mix2, 8, 100, t8, payload, 200e6, p_fail=0.05, rounds=60000, seed=7)
    assert got == pytest.approx(ref, rel=5e-3)                    # Monte-Carlo noise of 60 000 rounds
    assert got <= util.utilization(mix1, mix2, d) + 1e-15


def test_min_inner_steps_for_hidden_mix1():
    t8, payload = _fit()
    for bw in (100e6, 200e6):
        d = util.Deployment(8, 1, t8, payload, bw)
        H = util.min_inner_steps_for_hidden_mix1("global", d)
        assert oracle_util.simulate("global", "none", 8, H, t8, payload, bw) == pytest.approx(1.0)
        assert oracle_util.simulate("global", "none", 8, H - 1, t8, payload, bw) < 1.0
