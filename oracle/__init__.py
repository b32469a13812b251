"""CPU oracle for the paged-KV offload path -- TEST INFRASTRUCTURE ONLY.

A plain, slow, obviously-correct restatement of what the path computes, written from
the paper (EfficientAgent) and the problem statement, in pure Python / numpy.  It
shares no code with the CUDA library and must never be imported by the product path:
only the tests, the smoke check and the benchmark's CPU-baseline leg may use it.

Modules
  hash        polynomial prefix hash of token blocks (keys depend on the whole prefix)
  match       longest resident prefix on the GPU / host tier, restore run, fresh tokens
  tier        LRU host tier reference model with write-all / filtered admission
  storeload   byte-exact store (paged pool -> host slots) and load (inverse)
  stackdist   reuse (stack) distances, Mattson hit prediction, coverage prediction
  sizing      KV footprint, working-set scale, pressure ratios, offload benefit ratio
  trace       whole-trace driver: one agent turn = hash, match, tier step, load, store
  audit       declined-chunk audit and threshold sensitivity
  closedloop  closed-loop replay: active pool, first-come-first-served engine, Eq. 2 service times
  eakv_oracle.c / c_oracle   the same hash, store/load and LRU tier (write-all, fixed admission) in plain C,
              checked against the modules above; the timed CPU baseline

Parity unpinned: the paper's trace-level results (its prediction tables, replay table
and declined-chunk shares) need the authors' recorded trajectories, which are not
available; nothing here is checked against them.
"""
