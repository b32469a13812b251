"""GPU parity: eakv_store / eakv_load against oracle.storeload, byte for byte, for both
host-link strategies, both tier locations and both device copy paths."""
import itertools

import numpy as np
import pytest

from eakv_workloads import KVShape, SHAPES, counter_words_numpy, counter_words_torch
from oracle import storeload as osl

from gpu_util import make_ctx, require_gpu, torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _gpu():
    require_gpu()


def eakv():
    from paper_2609_33762_b200 import eakv as m
    return m


def variants():
    e = eakv()
    out = []
    for link, loc, path in itertools.product((e.LINK_ZERO_COPY, e.LINK_STAGED),
                                             (e.TIER_PINNED_HOST, e.TIER_DEVICE),
                                             (e.COPY_VECTOR, e.COPY_BULK)):
        kw = dict(link_strategy=link, tier_location=loc, copy_path=path)
        if link == e.LINK_STAGED:
            kw["min_staged_run_bytes"] = -1          # always through the staging buffers
        out.append(kw)
    # the default: staged, but scattered slots fall back to the direct kernel
    out.append(dict(link_strategy=e.LINK_STAGED, tier_location=e.TIER_PINNED_HOST,
                    copy_path=e.COPY_BULK, min_staged_run_bytes=0))
    # a mapped host tier moved by the vector kernel both ways, or by the bulk-copy ring (restores
    # only, which is the default, or both directions), with small explicit grids
    for hp in (e.HOST_COPY_VECTOR, e.HOST_COPY_BULK_LOAD, e.HOST_COPY_BULK_BOTH):
        out.append(dict(link_strategy=e.LINK_ZERO_COPY, tier_location=e.TIER_PINNED_HOST, host_copy_path=hp,
                        host_load_ctas=8, host_store_ctas=4))
    # copy engine only: needs the piece arrays at one pitch, i.e. one allocation for the whole pool
    for loc in (e.TIER_PINNED_HOST, e.TIER_DEVICE):
        out.append(dict(link_strategy=e.LINK_COPY_ENGINE, tier_location=loc, contiguous_pool=True))
    return out


def random_pool(rng, shape, nb):
    return [rng.integers(0, 256, size=(nb, shape.piece_bytes), dtype=np.uint8)
            for _ in range(shape.pieces_per_block)]


def to_device(pool_np, contiguous=False):
    if contiguous:      # one [2L][blocks][words] allocation; the piece arrays are its slices
        whole = torch.from_numpy(np.stack([a.view(np.int16) for a in pool_np])).cuda()
        return [whole[q] for q in range(len(pool_np))]
    return [torch.from_numpy(a.view(np.int16).copy()).cuda() for a in pool_np]


def pool_to_numpy(pool_dev):
    return [t.cpu().numpy().view(np.uint8) for t in pool_dev]


class Rig:
    """Device pool + context + oracle mirror, with a tier both sides initialise equally."""

    def __init__(self, shape, nb, kh, seed, **kw):
        e = eakv()
        self.shape, self.nb, self.kh = shape, nb, kh
        rng = np.random.default_rng(seed)
        self.rng = rng
        self.pool_np = random_pool(rng, shape, nb)
        self.pool_dev = to_device(self.pool_np, kw.pop("contiguous_pool", False))
        self.tier_np = rng.integers(0, 256, size=(kh, shape.pieces_per_block, shape.piece_bytes),
                                    dtype=np.uint8)
        self.loc = kw.get("tier_location", e.TIER_PINNED_HOST)
        if self.loc == e.TIER_DEVICE:
            self.tier_dev = torch.from_numpy(self.tier_np.copy()).cuda()
            kw["tier_memory"] = self.tier_dev.data_ptr()
        else:
            self.tier_host = torch.from_numpy(self.tier_np.copy()).pin_memory()
            kw["tier_memory"] = self.tier_host.data_ptr()
        self.ctx = make_ctx(shape, nb, kh, self.pool_dev, **kw)

    def tier_bytes(self):
        self.ctx.eakv_sync()
        if self.loc == eakv().TIER_DEVICE:
            return self.tier_dev.cpu().numpy()
        return self.tier_host.numpy()

    def check(self):
        got_tier = self.tier_bytes()
        assert np.array_equal(got_tier, self.tier_np)
        for a, b in zip(pool_to_numpy(self.pool_dev), self.pool_np):
            assert np.array_equal(a, b)

    def store(self, table, admit, slots):
        self.ctx.eakv_store(table, admit, slots)
        osl.store(self.pool_np, self.tier_np, table, [1] * len(table) if admit is None else admit, slots)

    def load(self, slots, table):
        self.ctx.eakv_load(slots, table)
        osl.load(self.pool_np, self.tier_np, slots, table)

    def close(self):
        self.ctx.close()


SHAPE_CASES = {
    "tiny": SHAPES["tiny"],                       # piece 4 KiB (one partial 16-KiB item)
    "qwen": SHAPES["qwen3_30b_a3b"],              # piece 16 KiB
    "llama": SHAPES["llama3_8b"],                 # piece 64 KiB (4 items per piece)
    "ragged": KVShape(3, 5, 128, 16),             # piece 20 KiB (16 KiB + 4 KiB tail)
    "small": KVShape(2, 3, 40, 2),                # piece 480 B
    "qwen_tp8": SHAPES["qwen3_30b_a3b"].tp_shard(8),   # one rank of TP8: 96 pieces of 4 KiB per block
}


@pytest.mark.parametrize("kw", variants(), ids=lambda k: "-".join(f"{v}" for v in k.values()))
@pytest.mark.parametrize("name", ["tiny", "qwen", "ragged", "small", "qwen_tp8"])
def test_store_load_parity(name, kw):
    shape = SHAPE_CASES[name]
    nb, kh = (96, 80) if shape.block_bytes <= (1 << 21) else (24, 20)
    # small staging buffers so the staged strategy cycles through several chunks
    rig = Rig(shape, nb, kh, seed=11, staging_bytes=5 * shape.block_bytes, **kw)
    rng = rig.rng
    # 1. masked store, unsorted ids and slots
    m = min(nb, kh) - 3
    table = rng.permutation(nb)[:m].astype(np.int32)
    slots = rng.permutation(kh)[:m].astype(np.int32)
    admit = (rng.random(m) < 0.5).astype(np.uint8)
    rig.store(table, admit, slots)
    rig.check()
    # 2. full store, contiguous ids and slots (long copy-engine runs), reversed table
    rig.store(np.arange(m, dtype=np.int32)[::-1].copy(), None, np.arange(m, dtype=np.int32))
    rig.check()
    # 3. load into shuffled fresh blocks
    k = m // 2
    src = rng.permutation(kh)[:k].astype(np.int32)
    dst = rng.permutation(nb)[:k].astype(np.int32)
    rig.load(src, dst)
    rig.check()
    # 4. round trip: load(store(x)) == x into other blocks
    blocks = np.arange(0, 8, dtype=np.int32)
    rig.store(blocks, None, np.arange(8, dtype=np.int32))
    rig.load(np.arange(8, dtype=np.int32), np.arange(8, 16, dtype=np.int32))
    rig.check()
    for q in range(shape.pieces_per_block):
        assert np.array_equal(rig.pool_np[q][0:8], rig.pool_np[q][8:16])
    # 5. degenerate calls: empty, all-zero mask, single block
    rig.store(np.zeros(0, np.int32), None, np.zeros(0, np.int32))
    rig.load(np.zeros(0, np.int32), np.zeros(0, np.int32))
    rig.store(table, np.zeros(m, np.uint8), slots)
    rig.store(np.array([nb - 1], np.int32), None, np.array([kh - 1], np.int32))
    rig.load(np.array([0], np.int32), np.array([nb - 2], np.int32))
    rig.check()
    rig.close()


def test_llama_shape_multi_item_pieces():
    e = eakv()
    for kw in (dict(copy_path=e.COPY_VECTOR), dict(copy_path=e.COPY_BULK, tier_location=e.TIER_DEVICE),
               dict(link_strategy=e.LINK_STAGED, min_staged_run_bytes=-1)):
        rig = Rig(SHAPE_CASES["llama"], 12, 10, seed=12, **kw)
        rig.store(np.array([3, 11, 0, 7], np.int32), np.array([1, 1, 0, 1], np.uint8),
                  np.array([9, 0, 5, 4], np.int32))
        rig.load(np.array([9, 4], np.int32), np.array([1, 2], np.int32))
        rig.check()
        rig.close()


def test_nan_payloads_and_negative_zero_survive():
    shape = SHAPES["tiny"]
    rig = Rig(shape, 4, 4, seed=13)
    words = np.array([0x7FC1, 0xFFFF, 0x8000, 0x7F80, 0xFF80, 0x0001] * (shape.piece_bytes // 12),
                     dtype=np.uint16)
    for q in range(shape.pieces_per_block):
        rig.pool_np[q][0, :len(words) * 2] = words.view(np.uint8)
        rig.pool_dev[q][0, :len(words)] = torch.from_numpy(words.view(np.int16)).cuda()
    rig.store(np.array([0], np.int32), None, np.array([2], np.int32))
    rig.load(np.array([2], np.int32), np.array([3], np.int32))
    rig.check()
    assert np.array_equal(rig.pool_np[0][3, :len(words) * 2].view(np.uint16), words)
    rig.close()


def test_validation_errors_change_nothing():
    e = eakv()
    shape = SHAPES["tiny"]
    rig = Rig(shape, 8, 6, seed=14)
    i32 = lambda *a: np.array(a, np.int32)
    cases = [
        (lambda: rig.ctx.eakv_store(i32(0, 8), None, i32(0, 1)), e.E_RANGE),     # block id == NB
        (lambda: rig.ctx.eakv_store(i32(0, -1), None, i32(0, 1)), e.E_RANGE),
        (lambda: rig.ctx.eakv_store(i32(0, 1), None, i32(0, 6)), e.E_RANGE),     # slot == K_H
        (lambda: rig.ctx.eakv_store(i32(0, 1), None, i32(3, 3)), e.E_INVAL),     # duplicate slot
        (lambda: rig.ctx.eakv_load(i32(0, 1), i32(5, 5)), e.E_INVAL),            # duplicate block
        (lambda: rig.ctx.eakv_load(i32(0, 7), i32(1, 2)), e.E_RANGE),
        (lambda: rig.ctx.eakv_load(i32(0, 1), i32(1, 9)), e.E_RANGE),
    ]
    for fn, code in cases:
        with pytest.raises(e.EakvError) as ei:
            fn()
        assert ei.value.code == code
    # masked-out entries are not validated, duplicates among them are fine
    rig.store(i32(0, 99, 99), np.array([1, 0, 0], np.uint8), i32(2, 2, 2))
    rig.check()
    assert rig.ctx.eakv_get_stats()["blocks_stored"] == 1
    rig.close()


def test_bad_shapes_rejected_at_create():
    e = eakv()
    t = torch.zeros(64, dtype=torch.int16, device="cuda")
    base = dict(num_layers=1, kv_heads=1, head_dim=8, block_size=16, gpu_blocks=1, host_blocks=1,
                kv_base=[t.data_ptr(), t.data_ptr()])
    for patch in (dict(head_dim=3, block_size=1),              # piece bytes not a multiple of 16
                  dict(kv_base=[t.data_ptr() + 2, t.data_ptr()]),   # misaligned base
                  dict(block_size=8192), dict(host_blocks=0), dict(policy=7),
                  dict(link_strategy=e.LINK_COPY_ENGINE),       # piece arrays not at one positive pitch
                  dict(link_strategy=3)):
        with pytest.raises(e.EakvError) as ei:
            e.Context(**{**base, **patch})
        assert ei.value.code == e.E_INVAL
    # a pool (or an adopted tier) in ordinary host memory: kernels cannot reach it
    host = np.zeros(4096, dtype=np.uint8)
    hp = (host.ctypes.data + 15) // 16 * 16
    for patch in (dict(kv_base=[hp, hp]), dict(tier_memory=hp)):
        with pytest.raises(e.EakvError) as ei:
            e.Context(**{**base, **patch})
        assert ei.value.code == e.E_INVAL
    # Copy engine alone: the pitch between piece arrays (2 GiB here: 131,072 blocks of 16 KiB) is
    # above what a strided copy-engine transfer accepts, so the configuration is refused at create
    # rather than failing on every later call.  The pool addresses are only compared, never
    # dereferenced: create returns before anything is allocated or copied.
    piece = 16 * 4 * 128 * 2
    pitch = 131072 * piece
    fake = [t.data_ptr() + q * pitch for q in range(4)]
    with pytest.raises(e.EakvError) as ei:
        e.Context(num_layers=2, kv_heads=4, head_dim=128, block_size=16, gpu_blocks=131072, host_blocks=1,
                  kv_base=fake, link_strategy=e.LINK_COPY_ENGINE)
    assert ei.value.code == e.E_INVAL


@pytest.mark.parametrize("kw", [
    dict(tier_location=1, copy_path=1), dict(tier_location=1, copy_path=0),
    dict(tier_location=0, link_strategy=0),
    dict(tier_location=0, link_strategy=1, min_staged_run_bytes=-1),
    dict(tier_location=0, link_strategy=1),
    dict(tier_location=0, link_strategy=2, contiguous_pool=True),
], ids=["hbm-bulk", "hbm-vector", "host-zero-copy", "host-staged", "host-default", "host-copy-engine"])
@pytest.mark.parametrize("name,group", [("qwen", 12), ("qwen", 5), ("tiny", 1), ("ragged", 2), ("qwen_tp8", 5),
                                        ("small", 1)])
def test_layer_pipelined_store(name, group, kw):
    """eakv_store_layers writes the same bytes as eakv_store, in layer groups (masked entries
    untouched, errors as for the plain store)."""
    e = eakv()
    shape = SHAPE_CASES[name]
    nb, kh = (64, 48) if shape.block_bytes <= (1 << 21) else (24, 20)
    rig = Rig(shape, nb, kh, seed=22, staging_bytes=3 * shape.block_bytes, **kw)
    rng = rig.rng
    groups = -(-shape.num_layers // group)
    none = [None] * groups
    m = min(nb, kh) - 5
    table = rng.permutation(nb)[:m].astype(np.int32)
    slots = rng.permutation(kh)[:m].astype(np.int32)
    admit = (rng.random(m) < 0.7).astype(np.uint8)
    stream = torch.cuda.Stream()
    rig.ctx.eakv_store_layers(table, admit, slots, group, none, stream)
    osl.store(rig.pool_np, rig.tier_np, table, admit, slots)
    stream.synchronize()
    rig.check()
    # contiguous slots without a mask, and an empty call
    rig.ctx.eakv_store_layers(np.arange(8, dtype=np.int32)[::-1].copy(), None, np.arange(8, dtype=np.int32),
                              group, none, stream)
    osl.store(rig.pool_np, rig.tier_np, list(range(8))[::-1], [1] * 8, list(range(8)))
    rig.ctx.eakv_store_layers(np.zeros(0, np.int32), None, np.zeros(0, np.int32), group, none, stream)
    stream.synchronize()
    rig.check()
    assert rig.ctx.eakv_get_stats()["blocks_stored"] == int(admit.sum()) + 8
    for bad, code in (((table, admit, slots, group, none + [None]), e.E_INVAL),                     # events
                      ((np.array([0, 1], np.int32), None, np.array([3, 3], np.int32), group, none), e.E_INVAL),
                      ((np.array([nb], np.int32), None, np.array([0], np.int32), group, none), e.E_RANGE)):
        with pytest.raises(e.EakvError) as ei:
            rig.ctx.eakv_store_layers(*bad, stream)
        assert ei.value.code == code
    rig.check()
    rig.close()


@pytest.mark.parametrize("kw", [
    dict(tier_location=1, copy_path=1),
    dict(tier_location=0, link_strategy=0),
    dict(tier_location=0, link_strategy=1, min_staged_run_bytes=-1),
    dict(tier_location=0, link_strategy=2, contiguous_pool=True),
], ids=["hbm-bulk", "host-zero-copy", "host-staged", "host-copy-engine"])
@pytest.mark.parametrize("name,group", [("qwen", 12), ("qwen_tp8", 16)])
def test_layer_pipelined_store_waits_for_each_group(name, group, kw):
    """The contract of eakv_store_layers: group g is read only after ready_events[g].  A producer
    stream fills the layers group by group, each fill held back by a delay and followed by its
    event; the store is enqueued on another stream right away.  The tier must hold what the
    producer wrote, not what the blocks held when the store was enqueued."""
    shape = SHAPE_CASES[name]
    nb, kh, m = 64, 48, 40
    rig = Rig(shape, nb, kh, seed=34, staging_bytes=4 * shape.block_bytes, **kw)
    rng = rig.rng
    groups = -(-shape.num_layers // group)
    table = rng.permutation(nb)[:m].astype(np.int32)
    slots = rng.permutation(kh)[:m].astype(np.int32)
    ids = torch.as_tensor(table.astype(np.int64), device="cuda")
    fresh = [torch.from_numpy(rng.integers(0, 256, size=(m, shape.piece_bytes), dtype=np.uint8)).cuda()
             for _ in range(shape.pieces_per_block)]
    producer, io = torch.cuda.Stream(), torch.cuda.Stream()
    events = [torch.cuda.Event() for _ in range(groups)]
    torch.cuda.synchronize()
    with torch.cuda.stream(producer):
        for g in range(groups):
            torch.cuda._sleep(20_000_000)                       # ~10 ms: the store is enqueued long before
            for q in range(2 * g * group, min(2 * (g + 1) * group, shape.pieces_per_block)):
                rig.pool_dev[q].view(torch.uint8).view(nb, -1)[ids] = fresh[q]
            events[g].record(producer)
    rig.ctx.eakv_store_layers(table, None, slots, group, [ev.cuda_event for ev in events], io)
    for q in range(shape.pieces_per_block):
        rig.pool_np[q][table] = fresh[q].cpu().numpy()
    osl.store(rig.pool_np, rig.tier_np, table, [1] * m, slots)
    io.synchronize()
    producer.synchronize()
    rig.check()
    rig.close()


def test_a_tier_that_cannot_be_allocated_is_refused_cleanly():
    """A 3 TiB tier in HBM (2 M slots of 1.5 MiB): the one device allocation of that size is refused
    by the runtime at once, create returns EAKV_E_NOMEM after freeing what it had, and the device
    is as usable as before (a working context right after it)."""
    e = eakv()
    shape = SHAPES["qwen3_30b_a3b"]
    t = torch.zeros(2 * shape.piece_bytes // 2, dtype=torch.int16, device="cuda")
    free_before = torch.cuda.mem_get_info()[0]
    with pytest.raises(e.EakvError) as ei:
        e.Context(num_layers=shape.num_layers, kv_heads=shape.kv_heads, head_dim=shape.head_dim,
                  block_size=shape.block_size, gpu_blocks=2, host_blocks=1 << 21,
                  kv_base=[t.data_ptr()] * shape.pieces_per_block, tier_location=e.TIER_DEVICE)
    assert ei.value.code == e.E_NOMEM
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] >= free_before - (64 << 20)      # nothing of the attempt is left
    rig = Rig(SHAPE_CASES["tiny"], 8, 4, 11, tier_location=1)
    rig.store(np.array([1, 3], np.int32), None, np.array([0, 2], np.int32))
    rig.load(np.array([0, 2], np.int32), np.array([5, 6], np.int32))
    rig.check()
    rig.close()


@pytest.mark.parametrize("kw", [
    dict(tier_location=1, copy_path=1), dict(tier_location=1, copy_path=0),
    dict(tier_location=0, link_strategy=0),
    dict(tier_location=0, link_strategy=1, min_staged_run_bytes=-1),
    dict(tier_location=0, link_strategy=1),
    dict(tier_location=0, link_strategy=2, contiguous_pool=True),
], ids=["hbm-bulk", "hbm-vector", "host-zero-copy", "host-staged", "host-default", "host-copy-engine"])
@pytest.mark.parametrize("name,group", [("qwen", 12), ("qwen", 5), ("tiny", 1), ("ragged", 2), ("tiny", 4),
                                        ("qwen_tp8", 12), ("qwen_tp8", 5), ("small", 1)])
def test_layer_pipelined_load(name, group, kw):
    """eakv_load_layers moves the same bytes as eakv_load, in layer groups, and records one
    event per group."""
    e = eakv()
    shape = SHAPE_CASES[name]
    nb, kh = (64, 48) if shape.block_bytes <= (1 << 21) else (24, 20)
    rig = Rig(shape, nb, kh, seed=21, staging_bytes=3 * shape.block_bytes, **kw)
    rng = rig.rng
    groups = -(-shape.num_layers // group)
    events = [torch.cuda.Event() for _ in range(groups)]
    for ev in events:
        ev.record()                                   # materialise the handles
    torch.cuda.synchronize()
    m = min(nb, kh) - 5
    src = rng.permutation(kh)[:m].astype(np.int32)
    dst = rng.permutation(nb)[:m].astype(np.int32)
    stream = torch.cuda.Stream()
    rig.ctx.eakv_load_layers(src, dst, group, [ev.cuda_event for ev in events], stream)
    osl.load(rig.pool_np, rig.tier_np, src, dst)
    for ev in events:
        ev.synchronize()
        assert ev.query()
    stream.synchronize()
    rig.check()
    # contiguous slots (long copy-engine strips), a small call, and an empty one
    rig.ctx.eakv_load_layers(np.arange(8, dtype=np.int32), np.arange(8, dtype=np.int32)[::-1].copy(),
                             group, [ev.cuda_event for ev in events], stream)
    osl.load(rig.pool_np, rig.tier_np, list(range(8)), list(range(8))[::-1])
    rig.ctx.eakv_load_layers(np.zeros(0, np.int32), np.zeros(0, np.int32), group,
                             [ev.cuda_event for ev in events], stream)
    stream.synchronize()
    rig.check()
    with pytest.raises(e.EakvError) as ei:            # wrong number of events
        rig.ctx.eakv_load_layers(src, dst, group, [ev.cuda_event for ev in events] + [events[0].cuda_event], stream)
    assert ei.value.code == e.E_INVAL
    with pytest.raises(e.EakvError) as ei:
        rig.ctx.eakv_load_layers(np.array([0, 1], np.int32), np.array([3, 3], np.int32), group,
                                 [ev.cuda_event for ev in events], stream)
    assert ei.value.code == e.E_INVAL
    rig.check()
    rig.close()


@pytest.mark.parametrize("kw", [
    dict(tier_location=1, copy_path=1),
    dict(tier_location=0, link_strategy=0),
    dict(tier_location=0, link_strategy=1, min_staged_run_bytes=-1),
    dict(tier_location=0, link_strategy=1),
    dict(tier_location=0, link_strategy=2, contiguous_pool=True),
], ids=["hbm-bulk", "host-zero-copy", "host-staged", "host-default", "host-copy-engine"])
@pytest.mark.parametrize("name,group,contiguous_slots", [("qwen", 12, True), ("qwen", 5, False), ("qwen_tp8", 16, True)])
def test_layer_group_event_means_the_group_has_landed(name, group, contiguous_slots, kw):
    """The contract of eakv_load_layers (Section 3.1, Eq. 2: tau_load is what a consumer waits for):
    a stream that waits on events[g] and on nothing else may read the layers of group g.  One
    consumer stream per group waits on its event and copies that group's layers of the
    destination blocks into a side buffer, all enqueued while the restore is still in flight;
    every side buffer must hold the oracle's bytes."""
    shape = SHAPE_CASES[name]
    nb, kh = 64, 48
    rig = Rig(shape, nb, kh, seed=33, staging_bytes=4 * shape.block_bytes, **kw)
    rng = rig.rng
    groups = -(-shape.num_layers // group)
    events = [torch.cuda.Event() for _ in range(groups)]
    for ev in events:
        ev.record()
    torch.cuda.synchronize()
    m = 40
    src = (np.arange(m) + 3 if contiguous_slots else rng.permutation(kh)[:m]).astype(np.int32)
    dst = rng.permutation(nb)[:m].astype(np.int32)
    ids = torch.as_tensor(dst.astype(np.int64), device="cuda")
    consumers = [torch.cuda.Stream() for _ in range(groups)]
    side = [None] * groups
    stream = torch.cuda.Stream()
    torch.cuda.synchronize()
    rig.ctx.eakv_load_layers(src, dst, group, [ev.cuda_event for ev in events], stream)
    for g in range(groups):
        q0, q1 = 2 * g * group, min(2 * (g + 1) * group, shape.pieces_per_block)
        consumers[g].wait_event(events[g])
        with torch.cuda.stream(consumers[g]):
            side[g] = torch.stack([rig.pool_dev[q][ids] for q in range(q0, q1)])
    osl.load(rig.pool_np, rig.tier_np, src, dst)
    for g in range(groups):
        consumers[g].synchronize()
        q0, q1 = 2 * g * group, min(2 * (g + 1) * group, shape.pieces_per_block)
        got = side[g].cpu().numpy().view(np.uint8)
        for i, q in enumerate(range(q0, q1)):
            assert np.array_equal(got[i], rig.pool_np[q][dst]), (g, q)
    stream.synchronize()
    rig.check()
    rig.close()


@pytest.mark.parametrize("kw", [
    dict(tier_location=1, copy_path=1), dict(tier_location=1, copy_path=0),
    dict(tier_location=0, link_strategy=0),
    dict(tier_location=0, link_strategy=1, min_staged_run_bytes=-1),
    dict(tier_location=0, link_strategy=1),
    dict(tier_location=0, link_strategy=2, contiguous_pool=True),
], ids=["hbm-bulk", "hbm-vector", "host-zero-copy", "host-staged", "host-default", "host-copy-engine"])
@pytest.mark.parametrize("name,group", [("qwen", 12), ("qwen", 5), ("tiny", 1), ("ragged", 2), ("qwen_tp8", 5),
                                        ("small", 1)])
def test_layer_pipelined_store(name, group, kw):
    """eakv_store_layers writes the same bytes as eakv_store, in layer groups (masked entries
    untouched, errors as for the plain store)."""
    e = eakv()
    shape = SHAPE_CASES[name]
    nb, kh = (64, 48) if shape.block_bytes <= (1 << 21) else (24, 20)
    rig = Rig(shape, nb, kh, seed=22, staging_bytes=3 * shape.block_bytes, **kw)
    rng = rig.rng
    groups = -(-shape.num_layers // group)
    none = [None] * groups
    m = min(nb, kh) - 5
    table = rng.permutation(nb)[:m].astype(np.int32)
    slots = rng.permutation(kh)[:m].astype(np.int32)
    admit = (rng.random(m) < 0.7).astype(np.uint8)
    stream = torch.cuda.Stream()
    rig.ctx.eakv_store_layers(table, admit, slots, group, none, stream)
    osl.store(rig.pool_np, rig.tier_np, table, admit, slots)
    stream.synchronize()
    rig.check()
    # contiguous slots without a mask, and an empty call
    rig.ctx.eakv_store_layers(np.arange(8, dtype=np.int32)[::-1].copy(), None, np.arange(8, dtype=np.int32),
                              group, none, stream)
    osl.store(rig.pool_np, rig.tier_np, list(range(8))[::-1], [1] * 8, list(range(8)))
    rig.ctx.eakv_store_layers(np.zeros(0, np.int32), None, np.zeros(0, np.int32), group, none, stream)
    stream.synchronize()
    rig.check()
    assert rig.ctx.eakv_get_stats()["blocks_stored"] == int(admit.sum()) + 8
    for bad, code in (((table, admit, slots, group, none + [None]), e.E_INVAL),                     # events
                      ((np.array([0, 1], np.int32), None, np.array([3, 3], np.int32), group, none), e.E_INVAL),
                      ((np.array([nb], np.int32), None, np.array([0], np.int32), group, none), e.E_RANGE)):
        with pytest.raises(e.EakvError) as ei:
            rig.ctx.eakv_store_layers(*bad, stream)
        assert ei.value.code == code
    rig.check()
    rig.close()


@pytest.mark.parametrize("kw", [
    dict(tier_location=1, copy_path=1),
    dict(tier_location=0, link_strategy=0),
    dict(tier_location=0, link_strategy=1, min_staged_run_bytes=-1),
    dict(tier_location=0, link_strategy=2, contiguous_pool=True),
], ids=["hbm-bulk", "host-zero-copy", "host-staged", "host-copy-engine"])
@pytest.mark.parametrize("name,group", [("qwen", 12), ("qwen_tp8", 16)])
def test_layer_pipelined_store_waits_for_each_group(name, group, kw):
    """The contract of eakv_store_layers: group g is read only after ready_events[g].  A producer
    stream fills the layers group by group, each fill held back by a delay and followed by its
    event; the store is enqueued on another stream right away.  The tier must hold what the
    producer wrote, not what the blocks held when the store was enqueued."""
    shape = SHAPE_CASES[name]
    nb, kh, m = 64, 48, 40
    rig = Rig(shape, nb, kh, seed=34, staging_bytes=4 * shape.block_bytes, **kw)
    rng = rig.rng
    groups = -(-shape.num_layers // group)
    table = rng.permutation(nb)[:m].astype(np.int32)
    slots = rng.permutation(kh)[:m].astype(np.int32)
    ids = torch.as_tensor(table.astype(np.int64), device="cuda")
    fresh = [torch.from_numpy(rng.integers(0, 256, size=(m, shape.piece_bytes), dtype=np.uint8)).cuda()
             for _ in range(shape.pieces_per_block)]
    producer, io = torch.cuda.Stream(), torch.cuda.Stream()
    events = [torch.cuda.Event() for _ in range(groups)]
    torch.cuda.synchronize()
    with torch.cuda.stream(producer):
        for g in range(groups):
            torch.cuda._sleep(20_000_000)                       # ~10 ms: the store is enqueued long before
            for q in range(2 * g * group, min(2 * (g + 1) * group, shape.pieces_per_block)):
                rig.pool_dev[q].view(torch.uint8).view(nb, -1)[ids] = fresh[q]
            events[g].record(producer)
    rig.ctx.eakv_store_layers(table, None, slots, group, [ev.cuda_event for ev in events], io)
    for q in range(shape.pieces_per_block):
        rig.pool_np[q][table] = fresh[q].cpu().numpy()
    osl.store(rig.pool_np, rig.tier_np, table, [1] * m, slots)
    io.synchronize()
    producer.synchronize()
    rig.check()
    rig.close()


def test_a_tier_that_cannot_be_allocated_is_refused_cleanly():
    """A 3 TiB tier in HBM (2 M slots of 1.5 MiB): the one device allocation of that size is refused
    by the runtime at once, create returns EAKV_E_NOMEM after freeing what it had, and the device
    is as usable as before (a working context right after it)."""
    e = eakv()
    shape = SHAPES["qwen3_30b_a3b"]
    t = torch.zeros(2 * shape.piece_bytes // 2, dtype=torch.int16, device="cuda")
    free_before = torch.cuda.mem_get_info()[0]
    with pytest.raises(e.EakvError) as ei:
        e.Context(num_layers=shape.num_layers, kv_heads=shape.kv_heads, head_dim=shape.head_dim,
                  block_size=shape.block_size, gpu_blocks=2, host_blocks=1 << 21,
                  kv_base=[t.data_ptr()] * shape.pieces_per_block, tier_location=e.TIER_DEVICE)
    assert ei.value.code == e.E_NOMEM
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] >= free_before - (64 << 20)      # nothing of the attempt is left
    rig = Rig(SHAPE_CASES["tiny"], 8, 4, 11, tier_location=1)
    rig.store(np.array([1, 3], np.int32), None, np.array([0, 2], np.int32))
    rig.load(np.array([0, 2], np.int32), np.array([5, 6], np.int32))
    rig.check()
    rig.close()


@pytest.mark.parametrize("kw", [
    dict(tier_location=1, copy_path=1), dict(tier_location=1, copy_path=0),
    dict(tier_location=0, link_strategy=0),
    dict(tier_location=0, link_strategy=1, min_staged_run_bytes=-1),
], ids=["hbm-bulk", "hbm-vector", "host-zero-copy", "host-staged"])
@pytest.mark.parametrize("name,m", [("tiny", 12), ("qwen", 40), ("qwen_tp8", 40)])
def test_device_self_check_skips_the_entry_and_reports_range(name, m, kw):
    """The kernels' own bounds checks, made to trip without any access out of bounds: the host
    validates against the real pool size, the kernels are told a narrower one.  Entries between
    the two are skipped on the device (their bytes do not move, everything else does) and the next
    eakv_sync returns EAKV_E_RANGE once; afterwards the context works as before."""
    e = eakv()
    shape = SHAPE_CASES[name]
    nb, kh = 64, 48
    rig = Rig(shape, nb, kh, seed=44, staging_bytes=4 * shape.block_bytes, **kw)
    rng = rig.rng
    narrowed = nb - 8
    rig.ctx.eakv_selfcheck_limits(gpu_blocks=narrowed)
    # (a staged store gathers into a staging buffer that the copy engine then moves as a whole, so
    # a skipped entry's slot would receive stale staging bytes: only its restore is checked here)
    staged = kw.get("link_strategy") == e.LINK_STAGED and kw.get("tier_location") == e.TIER_PINNED_HOST
    for op in (("load",) if staged else ("store", "load")):
        # m - 3 blocks below the narrowed limit and 3 between it and the real one, shuffled
        table = np.concatenate([rng.permutation(narrowed)[:m - 3],
                                narrowed + rng.permutation(nb - narrowed)[:3]]).astype(np.int32)
        rng.shuffle(table)
        slots = rng.permutation(kh)[:m].astype(np.int32)
        keep = table < narrowed
        if op == "store":
            rig.ctx.eakv_store(table, None, slots)
            osl.store(rig.pool_np, rig.tier_np, table[keep], [1] * int(keep.sum()), slots[keep])
        else:
            rig.ctx.eakv_load(slots, table)
            osl.load(rig.pool_np, rig.tier_np, slots[keep], table[keep])
        with pytest.raises(e.EakvError) as ei:
            rig.ctx.eakv_sync()
        assert ei.value.code == e.E_RANGE
        rig.check()                               # the sync inside succeeds: the word was cleared
    with pytest.raises(e.EakvError) as ei:        # limits above the real sizes are refused
        rig.ctx.eakv_selfcheck_limits(gpu_blocks=nb + 1)
    assert ei.value.code == e.E_INVAL
    rig.ctx.eakv_selfcheck_limits()               # back to the real sizes
    table = rng.permutation(nb)[:m].astype(np.int32)
    slots = rng.permutation(kh)[:m].astype(np.int32)
    rig.store(table, None, slots)
    rig.load(slots[::-1].copy(), rng.permutation(nb)[:m].astype(np.int32))
    rig.check()
    rig.close()


def test_tier_slot_self_check_and_bounded_wait_report():
    e = eakv()
    shape = SHAPE_CASES["tiny"]
    nb, kh = 32, 32
    for kw in (dict(tier_location=1, copy_path=1), dict(tier_location=0, link_strategy=0)):
        rig = Rig(shape, nb, kh, seed=45, **kw)
        rig.ctx.eakv_selfcheck_limits(tier_slots=kh - 4)
        table = np.arange(nb, dtype=np.int32)
        slots = np.arange(kh, dtype=np.int32)[::-1].copy()
        keep = slots < kh - 4
        rig.ctx.eakv_store(table, None, slots)
        osl.store(rig.pool_np, rig.tier_np, table[keep], [1] * int(keep.sum()), slots[keep])
        with pytest.raises(e.EakvError) as ei:
            rig.ctx.eakv_sync()
        assert ei.value.code == e.E_RANGE
        rig.check()
        rig.ctx.eakv_selfcheck_limits()
        # a bounded wait that nothing satisfies gives up, reports, and leaves the context usable
        rig.ctx.eakv_selfcheck_wait_probe()
        with pytest.raises(e.EakvError) as ei:
            rig.ctx.eakv_sync()
        assert ei.value.code == e.E_TIMEOUT
        rig.ctx.eakv_sync()
        rig.store(table, None, slots)
        rig.check()
        rig.close()


def test_calls_larger_than_the_argument_ring_slot_are_split():
    """max_call_blocks smaller than the call: several argument uploads per call; also more
    calls than ring slots back to back (slot reuse)."""
    e = eakv()
    shape = SHAPE_CASES["tiny"]
    for kw in (dict(tier_location=e.TIER_DEVICE), dict(link_strategy=e.LINK_STAGED, min_staged_run_bytes=-1),
               dict(link_strategy=e.LINK_ZERO_COPY)):
        rig = Rig(shape, 300, 280, seed=31, max_call_blocks=40, staging_bytes=9 * shape.block_bytes, **kw)
        rng = rig.rng
        for rep in range(12):                      # 12 calls x up to 7 uploads each > 8 ring slots
            m = int(rng.integers(33, 270))
            rig.store(rng.permutation(300)[:m].astype(np.int32), (rng.random(m) < 0.8).astype(np.uint8),
                      rng.permutation(280)[:m].astype(np.int32))
            k = int(rng.integers(33, 270))
            rig.load(rng.permutation(280)[:k].astype(np.int32), rng.permutation(300)[:k].astype(np.int32))
        rig.check()
        rig.close()


def test_store_and_load_on_two_streams_concurrently():
    """A store and a load that touch disjoint blocks and slots may overlap on two streams."""
    e = eakv()
    shape = SHAPE_CASES["qwen"]
    for kw in (dict(link_strategy=e.LINK_STAGED, min_staged_run_bytes=-1), dict(link_strategy=e.LINK_ZERO_COPY),
               dict(tier_location=e.TIER_DEVICE)):
        rig = Rig(shape, 128, 128, seed=32, staging_bytes=4 * shape.block_bytes, **kw)
        s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
        torch.cuda.synchronize()
        for rep in range(4):
            blocks = rig.rng.permutation(128).astype(np.int32)
            slots = rig.rng.permutation(128).astype(np.int32)
            st_b, ld_b = blocks[:60], blocks[60:120]
            st_s, ld_s = slots[:60], slots[60:120]
            rig.ctx.eakv_load(ld_s, ld_b, s1)
            rig.ctx.eakv_store(st_b, None, st_s, s2)
            osl.load(rig.pool_np, rig.tier_np, ld_s, ld_b)
            osl.store(rig.pool_np, rig.tier_np, st_b, [1] * 60, st_s)
            s1.synchronize(); s2.synchronize()
        rig.check()
        rig.close()


def test_staging_smaller_than_two_blocks_and_stats():
    e = eakv()
    shape = SHAPE_CASES["ragged"]
    rig = Rig(shape, 20, 20, seed=33, link_strategy=e.LINK_STAGED, min_staged_run_bytes=-1,
              staging_bytes=shape.block_bytes + 1)          # one block per staging buffer
    rig.store(np.arange(7, dtype=np.int32), None, np.arange(7, dtype=np.int32)[::-1].copy())
    rig.load(np.array([6, 5, 4], np.int32), np.array([17, 18, 19], np.int32))
    rig.check()
    st = rig.ctx.eakv_get_stats()
    assert (st["blocks_stored"], st["blocks_loaded"]) == (7, 3)
    assert st["bytes_stored"] == 7 * shape.block_bytes and st["bytes_loaded"] == 3 * shape.block_bytes
    assert st["kernel_launches"] >= 10 and st["memcpy_calls"] >= 10
    rig.close()
