"""Store and load of KV blocks as opaque bytes (Section 2: host writes and restores;
Appendix D: a chunk is copied only if the tier lacks it, straight out of the paged blocks that hold it).

Layouts
  pool : list of 2L numpy uint8 arrays, pool[2*l + kv] has shape [NB, piece_bytes]
         (layer l's K for kv = 0, V for kv = 1, paged [NB][b][H][d] flattened per block)
  tier : numpy uint8 array [K_H, 2L, piece_bytes] (slot-major)
"""


def store(pool, tier, block_table, admit, host_slots):
    """Copy every piece of each admitted block j from pool block block_table[j] to tier
    slot host_slots[j].  Non-admitted entries are not touched."""
    for j in range(len(block_table)):
        if not admit[j]:
            continue
        for q in range(len(pool)):
            tier[host_slots[j], q, :] = pool[q][block_table[j], :]


def load(pool, tier, host_slots, block_table):
    """Copy every piece of tier slot host_slots[j] into pool block block_table[j]."""
    for j in range(len(block_table)):
        for q in range(len(pool)):
            pool[q][block_table[j], :] = tier[host_slots[j], q, :]
