"""Compute-utilisation model of a Factored Gossip DiLoCo deployment (the paper's Sec. 5.2 simulator).

Host-side planning arithmetic, no GPU involved: given the worker count, the inner steps per round,
the step time, the payload size and the per-link bandwidth it returns the fraction of wall time
the workers spend computing, in closed form -- including the expectation under transient
failures, where an all-reduce attempt that loses any link is started again and a missed gossip
exchange just weakens the mix (Sec. 1, Sec. 5.2).  One round (Algorithm 1):
    Mix1 launched (non-blocking) | H inner steps | wait for the link | Mix2 (blocking) | outer optimizer.
A global average costs a ring all-reduce, 2 (M-1)/M payloads per link; pairwise gossip one payload.
"""
from __future__ import annotations

import math
from dataclasses import dataclass


@dataclass(frozen=True)
class Deployment:
    M: int                        # workers
    H: int                        # inner steps per round
    t_step: float                 # seconds per inner step of one worker
    payload_bytes: float          # bytes of one copy of the communicated parameters
    bandwidth_bps: float          # per-link bandwidth, bits per second
    t_outer: float = 0.0          # seconds of outer-optimizer compute per round


def mix_seconds(kind: str, d: Deployment, payload_scale: float = 1.0) -> float:
    link = d.payload_bytes * payload_scale * 8.0 / d.bandwidth_bps
    return {"none": 0.0, "local": link, "global": 2.0 * (d.M - 1) / d.M * link}[kind]


def _expected_attempts_time(kind: str, one: float, q: float) -> float:
    """Expected time of a transfer whose all-reduce attempts fail with probability q and restart."""
    return one / (1.0 - q) if kind == "global" and q > 0.0 else one


def _expected_hidden(kind: str, one: float, q: float, compute: float) -> float:
    """E[max(compute, attempts * one)]: when the link is free for Mix2 (geometric number of attempts)."""
    if kind != "global" or q <= 0.0 or one == 0.0:
        return max(compute, one)
    total, n, p_n = 0.0, 1, 1.0 - q
    while p_n > 1e-18 and n <= 10000:          # (the neglected tail of the geometric law is below 1e-16 of the sum)
        total += p_n * max(compute, n * one)
        n += 1
        p_n *= q
    return total


def utilization(mix1: str, mix2: str, d: Deployment, *, mix2_fraction: float = 1.0, state_in_mix1: bool = False,
                p_fail: float = 0.0) -> float:
    """Expected compute utilisation of the configuration (Mix1, Mix2) in {"none", "local", "global"}^2.

    A worker's link carries one transfer at a time, so Mix2 starts when both the inner steps and
    Mix1 are through: round = max(compute, Mix1) + Mix2 + outer optimizer.  Exact for p_fail = 0;
    with failures it is expected compute over expected round time (the long-run utilisation)."""
    q = 1.0 - (1.0 - p_fail) ** d.M
    compute = d.H * d.t_step
    m1_one = mix_seconds(mix1, d, 2.0 if state_in_mix1 else 1.0)
    m2_one = mix_seconds(mix2, d, mix2_fraction)
    round_t = _expected_hidden(mix1, m1_one, q, compute) + _expected_attempts_time(mix2, m2_one, q) + d.t_outer
    return compute / round_t


def min_inner_steps_for_hidden_mix1(mix1: str, d: Deployment, *, state_in_mix1: bool = False) -> int:
    """Smallest H whose compute hides Mix1 completely (the paper quotes H of about 180 / 90 at 100 / 200 Mbps)."""
    return int(math.ceil(mix_seconds(mix1, d, 2.0 if state_in_mix1 else 1.0) / d.t_step))
