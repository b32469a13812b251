"""Random interleavings of overlapping requests whose host writes are deferred: begin, later store,
later finish, with other requests' lookups in between.  One generator of operations serves the
oracle's own pins and the parity tests (it holds none of the method's arithmetic)."""
import random

import numpy as np


class Prompts:
    """A few agents whose prompts grow by appends and share a system prefix."""

    def __init__(self, rng, block, agents=5, system_blocks=3, vocab=50000):
        self.rng, self.b = rng, block
        self.system = [rng.randrange(vocab) for _ in range(system_blocks * block)]
        self.tokens = {a: list(self.system) for a in range(agents)}
        self.vocab = vocab

    def next_prompt(self, agent, max_tokens):
        t = self.tokens[agent]
        if len(t) > max_tokens * 3 // 4 or self.rng.random() < 0.1:       # the agent starts a new task
            t = self.tokens[agent] = list(self.system)
        grow = self.rng.randrange(1, 4 * self.b)
        t.extend(self.rng.randrange(self.vocab) for _ in range(grow))
        del t[max_tokens:]
        return list(t)


def operations(seed, steps, block, max_tokens, max_open=4, agents=5):
    """Yields ("begin", rid, agent, tokens, now_ms) / ("store", rid) / ("finish", rid).  A request is
    stored once, after its begin, and finished after its store; at most ``max_open`` are open."""
    rng = random.Random(seed)
    prompts = Prompts(rng, block, agents)
    begun, stored = [], []            # waiting for their store / for their finish
    busy_agents = set()
    rid, now = 0, 0
    for _ in range(steps):
        now += rng.randrange(0, 4000)
        choices = []
        if len(begun) + len(stored) < max_open and len(busy_agents) < agents:
            choices += ["begin"] * 3
        if begun:
            choices += ["store"] * 2
        if stored:
            choices += ["finish"] * 2
        op = rng.choice(choices)
        if op == "begin":
            agent = rng.choice([a for a in range(agents) if a not in busy_agents])
            rid += 1
            # the caller reports through send() whether the request was admitted to the GPU
            admitted = yield ("begin", rid, agent, prompts.next_prompt(agent, max_tokens), now)
            if admitted:
                begun.append((rid, agent))
                busy_agents.add(agent)
        elif op == "store":
            r = begun.pop(rng.randrange(len(begun)))
            stored.append(r)
            yield ("store", r[0])
        else:
            r = stored.pop(rng.randrange(len(stored)))
            busy_agents.discard(r[1])
            yield ("finish", r[0])
    for r in begun:
        yield ("store", r[0])
    for r in begun + stored:
        yield ("finish", r[0])


def drive(ops, on_begin, on_store, on_finish):
    """Runs the generator; on_begin returns whether the request was admitted."""
    gen = ops
    try:
        op = next(gen)
        while True:
            if op[0] == "begin":
                op = gen.send(bool(on_begin(*op[1:])))
                continue
            if op[0] == "store":
                on_store(op[1])
            else:
                on_finish(op[1])
            op = next(gen)
    except StopIteration:
        pass


def as_keys(x):
    return np.asarray(x, dtype=np.uint64)
