"""Host-tier reference model and write admission.

Reference model (Appendix D, "Reference model" and "Recency order of the host tier"):
an LRU list of capacity K_H chunks, empty at time zero.  Referencing a resident chunk is a hit
and makes it the most recent entry.  An admitted miss appends the chunk as the most recent entry;
if the list already has K_H entries its least recent one is dropped first.  A miss that is
declined changes nothing.

Write rule (Eq. 6): with n prompt tokens and a host-resident prefix of h tokens, the request
would add u = floor(n/b) - floor(h/b) full chunks, and save(r) = not (p_t and u > kappa),
decided once per request.  p_t is 0 for plain offload (write-all), 1 for fixed write
admission, and the pressure signal of Eq. 10 for capacity-conditioned admission:
p_t = [ (A_t - 1) N_t beta > C_H ] and [ o_t >= theta and e_t > 0 ].  Copy-time
deduplication falls out of the model: a resident chunk is a hit and is never copied.

Readings taken where the paper is silent (integers only, virtual time in ms):
  * windows are (now - W, now]; A_t counts distinct agents with a request in the window
    including the current one; N_t is the mean of the last <= 256 prompt lengths
    including the current one; e_t counts capacity evictions in the window before the
    current request inserts anything; o_t uses the resident count at that same moment;
  * C_H is taken as K_H * b * beta, so beta cancels: (A_t-1) * sum_len > K_H * b * count;
  * slots come from a free stack that first yields 0, 1, 2, ...; an evicted chunk's slot
    is the next one handed out;
  * a request with more full chunks than K_H is refused and changes nothing.

Tier reports (Appendix D, "Pressure signal" and the parameter table: the tier publishes the number
of registered chunks, K_H and e_t every second; a report older than 5 seconds is not fresh; with
nothing fresh to read (nothing published yet, say) p_t reduces to its working-set factor).  With ``telemetry_period_ms`` = P > 0 the second factor is read from the latest report
instead of from the tier itself: reports are published at the virtual times P, 2P, 3P, ...; the
report of time t describes the tier as the requests before t left it (registered chunks, and the
evictions with a time in (t - W, t)); a request at time ``now`` reads the report of time
floor(now / P) * P, which exists from P on; it is fresh while now - t <= ``telemetry_max_age_ms``
(0: any age).  The paper's scheduler reads reports every 0.5 s; since that divides its 1 s report
interval, a read always sees the latest report, so the read interval is no parameter here.
P = 0 is the synchronous reading above.
"""
from collections import OrderedDict, deque

WRITE_ALL = 0
FILTER_FIXED = 1
FILTER_CONDITIONED = 2


class CapacityError(Exception):
    pass


class StepResult:
    __slots__ = ("hit", "admit", "slot", "evicted", "save", "pressure", "new_chunks",
                 "host_prefix_blocks")

    def __init__(self):
        self.hit = []
        self.admit = []
        self.slot = []
        self.evicted = []        # (key, slot) in eviction order
        self.save = True
        self.pressure = False
        self.new_chunks = 0
        self.host_prefix_blocks = 0


class HostTier:
    def __init__(self, capacity_blocks, block_size, policy=WRITE_ALL, kappa_blocks=8,
                 theta_percent=95, window_ms=60_000, len_window=256, telemetry=True,
                 telemetry_period_ms=0, telemetry_max_age_ms=0):
        self.K = int(capacity_blocks)
        self.period = int(telemetry_period_ms)
        self.max_age = int(telemetry_max_age_ms)
        self.report = None                            # (time, registered chunks, e_t) of the latest report
        self.b = int(block_size)
        self.policy = policy
        self.kappa = int(kappa_blocks)
        self.theta_percent = int(theta_percent)
        self.window_ms = int(window_ms)
        self.telemetry = telemetry
        self.order = OrderedDict()                    # key -> slot, least recent first
        self.free = list(range(self.K - 1, -1, -1))   # pop() yields 0, 1, 2, ...
        self.agent_last = {}                          # agent -> time of latest request
        self.lengths = deque(maxlen=int(len_window))
        self.evict_times = deque()
        self.stats = dict(requests=0, references=0, hits=0, admitted=0, declined=0,
                          evicted=0, declined_requests=0, pressure_requests=0)

    # ---- lookups that do not change recency -------------------------------------------
    def __contains__(self, key):
        return key in self.order

    def slot_of(self, key):
        return self.order[key]

    def leading_run(self, keys):
        n = 0
        for k in keys:
            if k not in self.order:
                break
            n += 1
        return n

    # ---- published reports ----------------------------------------------------------------
    def _publish(self, now_ms):
        """Bring the latest report up to date before a request at ``now_ms`` changes anything:
        if a publication time has passed since the last report, the tier as it stands is what
        that publication saw (every earlier request came before it)."""
        if self.period <= 0:
            return
        t = (now_ms // self.period) * self.period
        if t >= self.period and (self.report is None or self.report[0] < t):
            e = sum(1 for x in self.evict_times if t - self.window_ms < x < t)
            self.report = (t, len(self.order), e)

    # ---- Eq. 10 ---------------------------------------------------------------------------
    def _pressure(self, agent, n_tokens, now_ms):
        self.agent_last[agent] = now_ms
        self.lengths.append(int(n_tokens))
        lo = now_ms - self.window_ms
        while self.evict_times and self.evict_times[0] <= lo:
            self.evict_times.popleft()
        if self.policy == WRITE_ALL:
            return False
        if self.policy == FILTER_FIXED:
            return True
        active = sum(1 for t in self.agent_last.values() if t > lo)
        estimate_exceeds = (active - 1) * sum(self.lengths) > self.K * self.b * len(self.lengths)
        if not self.telemetry:
            return estimate_exceeds
        if self.period > 0:
            fresh = self.report is not None and (self.max_age <= 0 or now_ms - self.report[0] <= self.max_age)
            if not fresh:
                return estimate_exceeds
            _, registered, evicted = self.report
            return estimate_exceeds and 100 * registered >= self.theta_percent * self.K and evicted > 0
        full = 100 * len(self.order) >= self.theta_percent * self.K
        evicting = len(self.evict_times) > 0
        return estimate_exceeds and full and evicting

    # ---- one request ----------------------------------------------------------------------
    def step(self, keys, n_tokens, agent, now_ms, decided=None):
        """``decided``: None for the request's first lookup.  A later lookup of the same request
        (after a preemption; Appendix D: the store/skip choice made at the first lookup
        also holds for the request's further lookups) passes the choice made then: the walk is the same, but the request is not
        registered again in the activity and prompt-length windows, which count first lookups."""
        if len(keys) > self.K:
            raise CapacityError("request references more blocks than the tier holds")
        self._publish(now_ms)
        res = StepResult()
        H = self.leading_run(keys)
        res.host_prefix_blocks = H
        res.new_chunks = n_tokens // self.b - (H * self.b) // self.b
        st = self.stats
        if decided is None:
            res.pressure = self._pressure(agent, n_tokens, now_ms)
            res.save = not (res.pressure and res.new_chunks > self.kappa)
            st["requests"] += 1
            st["pressure_requests"] += int(res.pressure)
            st["declined_requests"] += int(not res.save)
        else:
            res.pressure = False
            res.save = bool(decided)
        for k in keys:
            st["references"] += 1
            if k in self.order:
                self.order.move_to_end(k)
                res.hit.append(1); res.admit.append(0); res.slot.append(self.order[k])
                st["hits"] += 1
            elif res.save:
                if len(self.order) >= self.K:
                    vk, vs = self.order.popitem(last=False)
                    self.free.append(vs)
                    res.evicted.append((vk, vs))
                    self.evict_times.append(now_ms)
                    st["evicted"] += 1
                s = self.free.pop()
                self.order[k] = s
                res.hit.append(0); res.admit.append(1); res.slot.append(s)
                st["admitted"] += 1
            else:
                res.hit.append(0); res.admit.append(0); res.slot.append(-1)
                st["declined"] += 1
        return res


def simulate_stream(stream, capacity, declined=frozenset()):
    """Bare reference model over a flat stream of chunk keys.  ``declined`` holds the
    reference indices whose miss is not inserted.  Returns the list of hit flags."""
    order = OrderedDict()
    hits = []
    for i, k in enumerate(stream):
        if k in order:
            order.move_to_end(k)
            hits.append(True)
            continue
        hits.append(False)
        if i in declined:
            continue
        if len(order) >= capacity:
            order.popitem(last=False)
        order[k] = True
    return hits
