"""Seeded agent traces: request order, prompt lengths and token ids.

Every agent resends its whole conversation each turn, so turn t's prompt is the first
``n_tokens`` ids of that agent's token stream (pure appends: the cache-stable prompt
length equals the previous prompt's length).  Request times come from a closed loop
with zero service time, so the order does not depend on how fast anything runs.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, List

import numpy as np

from .shapes import CONFIGS, TraceConfig


@dataclass(frozen=True)
class Request:
    time_ms: int
    agent: int
    turn: int
    n_tokens: int


@dataclass
class Trace:
    config: TraceConfig
    requests: List[Request]
    agent_tokens: Dict[int, np.ndarray]  # agent -> int32[max prompt length of that agent]
    # agent -> int64[turns]: tool/agent time in ms between the end of turn t-1 and turn t
    # (entry 0 is 0).  ``requests`` is the open-loop order these gaps give with zero service
    # time; a closed-loop replay takes the gaps and lengths and orders the calls itself.
    agent_gaps_ms: Dict[int, np.ndarray] = None
    agent_lengths: Dict[int, np.ndarray] = None   # agent -> int64[turns] prompt lengths

    def prompt(self, req: Request) -> np.ndarray:
        return self.agent_tokens[req.agent][: req.n_tokens]

    @property
    def total_prompt_tokens(self) -> int:
        return sum(r.n_tokens for r in self.requests)


def make_trace(cfg, seed=None, agents=None, turns=None) -> Trace:
    """Build the trace of a named configuration (or a TraceConfig).

    ``agents``/``turns`` shrink the trace for tests; the draw order is fixed
    (all lengths first, then times, then tokens per agent) so a given seed always
    yields the same trace for the same arguments.
    """
    if isinstance(cfg, str):
        cfg = CONFIGS[cfg]
    assert isinstance(cfg, TraceConfig)
    seed = cfg.seed if seed is None else seed
    A = cfg.agents if agents is None else agents
    T = cfg.turns if turns is None else turns
    rng = np.random.default_rng(seed)

    # prompt lengths per agent and turn
    lengths = np.zeros((A, T), dtype=np.int64)
    for a in range(A):
        n = min(cfg.first_prompt, cfg.context_cap)
        for t in range(T):
            if t > 0:
                draw = int(np.floor(rng.lognormal(np.log(cfg.append_median), cfg.append_sigma)))
                n = n + min(draw, cfg.context_cap - n)
            lengths[a, t] = n

    # request times
    times = np.zeros((A, T), dtype=np.int64)
    gaps_ms = np.zeros((A, T), dtype=np.int64)
    if cfg.interleave == "round_robin":
        for t in range(T):
            for a in range(A):
                times[a, t] = t * A + a
    else:
        start = np.zeros(A, dtype=np.float64)
        if cfg.interleave == "poisson_start":
            start = np.cumsum(rng.exponential(cfg.start_gap_mean_ms, size=A))
        for a in range(A):
            gaps = rng.exponential(cfg.tool_gap_mean_ms, size=T)
            gaps[0] = 0.0
            times[a] = np.floor(start[a] + np.cumsum(gaps)).astype(np.int64)
            gaps_ms[a] = np.floor(gaps).astype(np.int64)

    # token ids: independent stream per agent, after an optional prefix common to all agents
    agent_tokens = {}
    for a in range(A):
        agent_tokens[a] = rng.integers(0, cfg.vocab, size=int(lengths[a, -1]), dtype=np.int32)
    if cfg.shared_prefix_tokens > 0:
        common = rng.integers(0, cfg.vocab, size=cfg.shared_prefix_tokens, dtype=np.int32)
        for a in range(A):
            k = min(len(common), len(agent_tokens[a]))
            agent_tokens[a][:k] = common[:k]

    reqs = [Request(int(times[a, t]), a, t, int(lengths[a, t])) for a in range(A) for t in range(T)]
    reqs.sort(key=lambda r: (r.time_ms, r.agent, r.turn))
    return Trace(cfg, reqs, agent_tokens,
                 agent_gaps_ms={a: gaps_ms[a].copy() for a in range(A)},
                 agent_lengths={a: lengths[a].copy() for a in range(A)})
