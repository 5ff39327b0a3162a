"""Oracle of the paper's compute-utilisation simulator (Sec. 5.2) -- TEST INFRASTRUCTURE ONLY.

PARITY UNPINNED BY THE PAPER'S TEXT ALONE: the paper names the simulator's four components
(forward/backward compute, outer-optimizer compute, Mix1 communication, Mix2 communication) and
its one assumption (a fixed per-link bandwidth between any pair of workers) but prints neither the
step time nor the payload size nor the restart policy.  The readings taken here:
  * one round = H inner steps of t_step seconds while Mix1 (launched at the top of the round,
    Algorithm 1) uses the link, then the blocking Mix2 transfer, then t_outer seconds of outer
    optimizer; utilisation = time spent in inner steps / wall time;
  * a worker's link (the bandwidth is per link and fixed) carries one transfer at a time: if Mix1 is still
    running when the inner steps end, Mix2 queues behind what is left of it, so the round's
    communication ends at max(compute, Mix1) + Mix2 -- this is the reading under which the printed
    GlobalM1LocalM2 cells (36 % at 100 Mbps where Mix1 is not hidden) come out; letting the two
    transfers overlap at full rate each gives 50 % there;
  * a global average is a bandwidth-optimal ring all-reduce, 2 (M-1)/M payloads per link
    (Sec. 5.2 puts it at no more than roughly double what gossip moves); pairwise gossip is one
    full-duplex exchange, one payload per link;
  * a worker's step time is proportional to its batch (GBS / M sequences);
  * Mix2 on a subset moves that fraction of the payload; Mix1 "with state" moves two payloads;
  * failures (Sec. 5.2, last paragraph): every all-reduce ATTEMPT fails as a whole with
    probability q = 1 - (1 - p)^M (any of the ring's M links) and is started again; a failed
    gossip exchange is skipped (weaker mixing) and costs no extra time.
The two unknown constants are fitted by the TEST on two printed cells and every other printed
cell is then a pin (tests/golden/table1_compute_utilization.txt).

Written as an explicit timeline, round by round, so that it can be read against Algorithm 1.
"""
from __future__ import annotations

import random


def transfer_seconds(kind: str, M: int, payload_bytes: float, bandwidth_bps: float) -> float:
    """Time of one attempt of a mix: "none" 0, "local" one exchange, "global" a ring all-reduce."""
    per_link = payload_bytes * 8.0 / bandwidth_bps
    if kind == "none":
        return 0.0
    if kind == "local":
        return per_link
    if kind == "global":
        return 2.0 * (M - 1) / M * per_link
    raise ValueError(kind)


def simulate(mix1: str, mix2: str, M: int, H: int, t_step: float, payload_bytes: float, bandwidth_bps: float,
             *, t_outer: float = 0.0, mix2_fraction: float = 1.0, state_in_mix1: bool = False,
             p_fail: float = 0.0, rounds: int = 1, seed: int = 0) -> float:
    """Utilisation over `rounds` rounds of the timeline.  Deterministic for p_fail = 0."""
    rng = random.Random(seed)
    q = 1.0 - (1.0 - p_fail) ** M            # an all-reduce attempt fails if any ring link does

    def duration(kind, payload):
        one = transfer_seconds(kind, M, payload, bandwidth_bps)
        total = one
        if kind == "global":
            while rng.random() < q:          # restart from scratch
                total += one
        return total

    clock = 0.0
    busy = 0.0
    for _ in range(rounds):
        start = clock
        mix1_done = start + duration(mix1, payload_bytes * (2.0 if state_in_mix1 else 1.0))   # launched, not awaited
        clock += H * t_step                                                               # inner steps
        busy += H * t_step
        clock = max(clock, mix1_done)                                                     # the link is busy until Mix1 is through
        clock += duration(mix2, payload_bytes * mix2_fraction)                            # blocking
        clock += t_outer                                                                  # outer optimizer
    return busy / clock
