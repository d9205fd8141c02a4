"""Pins for the CPU oracle: every check here compares the oracle with something
that is not the oracle — a label-assembled brute force, numpy array indexing,
closed forms, invariants, and counts the paper prints."""
import itertools
import os

import numpy as np
import pytest

import oracle
from paper_2605_03375_b200 import workload as wl
from tests import hostcase as hc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# --------------------------------------------------------------------------
# (i) brute force on tiny pools: the store is *assembled* from labelled pieces
# in the order the layout prescribes (nested loops, no offset arithmetic), the
# expected pool is read off the labels.
# --------------------------------------------------------------------------

def _label(slot, layer, kv, tok):
    return np.array([slot + 1, layer + 1, kv + 1, tok + 1], dtype=np.uint8)


def _assemble_store(n_layers, n_slots, n_dev, obj_tokens, layout):
    """Per device, concatenate object halves in storage order.
    FILE_MAJOR: a file (= one slot) holds layer 0 K, layer 0 V, layer 1 K, ... and files
    follow one another.  LAYER_MAJOR: all slots' objects of layer 0, then layer 1, ...
    Slot s lives on device s mod n_dev as that device's (s div n_dev)-th file."""
    n_local = (n_slots + n_dev - 1) // n_dev
    devs = []
    for d in range(n_dev):
        pieces = []
        slots = [d + i * n_dev for i in range(n_local)]
        if layout == oracle.FILE_MAJOR:
            order = [(s, l) for s in slots for l in range(n_layers)]
        else:
            order = [(s, l) for l in range(n_layers) for s in slots]
        for s, l in order:
            for kv in (0, 1):
                for tok in range(obj_tokens):
                    pieces.append(_label(s, l, kv, tok))
        devs.append(np.concatenate(pieces))
    return devs


@pytest.mark.parametrize("layout", [oracle.FILE_MAJOR, oracle.LAYER_MAJOR])
@pytest.mark.parametrize("n_dev", [1, 2])
@pytest.mark.parametrize("obj_blocks", [1, 2])
def test_bruteforce_tiny_pools(layout, n_dev, obj_blocks):
    bt, n_layers, n_pool = 2, 2, 5
    obj_tokens = obj_blocks * bt
    n_slots = 4
    g = oracle.geom(n_layers, 1, 2, 2, bt, obj_tokens, n_dev, layout, n_slots)   # 4-byte tokens
    lo = oracle.obj_layout(g)
    assert lo.token_bytes == 4
    store = _assemble_store(n_layers, n_slots, n_dev, obj_tokens, layout)
    assert all(s.nbytes == lo.dev_bytes for s in store)
    n_cases = 0
    for n_blk in (1, 2, 3):
        hit = n_blk * bt
        n_obj = (hit + obj_tokens - 1) // obj_tokens
        for ids in itertools.permutations(range(n_pool), n_blk):
            for slots in itertools.permutations(range(n_slots), n_obj):
                if n_cases % 7 != 0 and n_blk == 3:      # thin the largest family
                    n_cases += 1
                    continue
                n_cases += 1
                batch = ([hit], [0, n_obj], list(slots), [0, n_blk], list(ids))
                for layer in range(n_layers):
                    pool = np.zeros(2 * n_pool * bt * 4, dtype=np.uint8)
                    rc = oracle.restore_layer(g, layer, batch, store, pool, 0, n_pool * bt * 4,
                                              bt * 4, n_pool)
                    assert rc == oracle.OK
                    exp = np.zeros((2, n_pool, bt, 4), dtype=np.uint8)
                    for t in range(hit):
                        for kv in (0, 1):
                            exp[kv, ids[t // bt], t % bt] = _label(slots[t // obj_tokens], layer,
                                                                   kv, t % obj_tokens)
                    assert np.array_equal(pool.reshape(2, n_pool, bt, 4), exp)
                    # save: pool labelled by (block, row), store must receive those labels
                    pool2 = np.zeros((2, n_pool, bt, 4), dtype=np.uint8)
                    for kv in (0, 1):
                        for b in range(n_pool):
                            for row in range(bt):
                                pool2[kv, b, row] = [200 + kv, b + 1, row + 1, 77]
                    st2 = [s.copy() for s in store]
                    rc = oracle.save_layer(g, layer, batch, st2, pool2.reshape(-1), 0,
                                           n_pool * bt * 4, bt * 4, n_pool)
                    assert rc == oracle.OK
                    # walk the store in assembly order and predict every 4-byte token cell
                    where = {}
                    for t in range(hit):
                        for kv in (0, 1):
                            where[(slots[t // obj_tokens], layer, kv, t % obj_tokens)] = \
                                (kv, ids[t // bt], t % bt)
                    for d in range(n_dev):
                        cells = st2[d].reshape(-1, 4)
                        orig = store[d].reshape(-1, 4)
                        for i in range(cells.shape[0]):
                            s, l, kv, tok = (int(v) - 1 for v in orig[i])
                            key = (s, l, kv, tok)
                            if key in where:
                                a, b, c = where[key]
                                assert np.array_equal(cells[i], pool2[a, b, c])
                            else:
                                assert np.array_equal(cells[i], orig[i])
    assert n_cases > 100


# --------------------------------------------------------------------------
# (ii) array-shaped restatement at medium size: the store viewed as an ndarray
# whose *shape* is the layout, the pool as [2][N][bt][token_bytes]; restore is
# one advanced-indexing assignment.
# --------------------------------------------------------------------------

def _store_nd(store, w, lo, d):
    n_local = int(lo.n_slots_local)
    tb = int(lo.token_bytes)
    if w.layout == wl.LAYOUT_FILE_MAJOR:
        return store[d].reshape(n_local, w.n_layers, 2, w.obj_tokens, tb), "file"
    return store[d].reshape(w.n_layers, n_local, 2, w.obj_tokens, tb), "layer"


def _expected_pool_numpy(w, lo, store, pool_before, layer):
    tb = int(lo.token_bytes)
    exp = pool_before.copy()
    if w.pool_hnd:
        # a block is [head][token][row]: present it as [token][head * row] through a view
        row = w.head_dim * w.elem_bytes
        if w.pool_interleaved:
            nd = exp.reshape(w.n_pool_blocks, 2, w.n_kv_heads, w.block_tokens, row)
            nd = nd.transpose(1, 0, 3, 2, 4)
        else:
            nd = exp.reshape(2, w.n_pool_blocks, w.n_kv_heads, w.block_tokens, row)
            nd = nd.transpose(0, 1, 3, 2, 4)
        # nd is now [kv][block][token][head][row]
    elif w.pool_pad_bytes:
        # every block is followed by unused bytes: a strided view that steps over them
        assert not w.pool_interleaved
        step = w.block_tokens * tb + w.pool_pad_bytes
        nd = np.lib.stride_tricks.as_strided(
            exp, shape=(2, w.n_pool_blocks, w.block_tokens, tb),
            strides=(w.n_pool_blocks * step, step, tb, 1))
    elif w.pool_interleaved:
        nd = exp.reshape(w.n_pool_blocks, 2, w.block_tokens, tb).transpose(1, 0, 2, 3)
    else:
        nd = exp.reshape(2, w.n_pool_blocks, w.block_tokens, tb)
    for r in range(w.n_req):
        hit = int(w.hit_tokens[r])
        t = np.arange(hit)
        blk = w.block_ids[w.blk_start[r] + t // w.block_tokens]
        slot = w.obj_slot[w.obj_start[r] + t // w.obj_tokens].astype(np.int64)
        for d in range(w.n_devices):
            sel = (slot % w.n_devices) == d
            if not sel.any():
                continue
            snd, kind = _store_nd(store, w, lo, d)
            loc = slot[sel] // w.n_devices
            for kv in (0, 1):
                if kind == "file":
                    src = snd[loc, layer, kv, t[sel] % w.obj_tokens]
                else:
                    src = snd[layer, loc, kv, t[sel] % w.obj_tokens]
                if w.pool_hnd:
                    src = src.reshape(src.shape[0], w.n_kv_heads, -1)
                nd[kv, blk[sel], t[sel] % w.block_tokens] = src
    return exp


CASES = [
    dict(index=2, scale=0.03),
    dict(index=2, scale=0.03, layout=wl.LAYOUT_FILE_MAJOR, n_layers=3),
    dict(index=2, scale=0.03, n_devices=2, pool_interleaved=True, n_layers=2),
    dict(index=4, scale=0.02, n_layers=2),
    dict(index=4, scale=0.02, n_layers=2, n_devices=3, layout=wl.LAYOUT_FILE_MAJOR),
    dict(index=3, scale=0.02, n_layers=2),
    dict(index=1),
    dict(index=2, scale=0.03, n_layers=2, pool_hnd=True),
    dict(index=2, scale=0.03, n_layers=2, pool_pad_bytes=64),
    dict(index=4, scale=0.02, n_layers=2, pool_hnd=True, pool_interleaved=True, n_kv_heads=4,
         head_dim=32, block_tokens=4, obj_tokens=32),
]


def _mk(case):
    case = dict(case)
    idx = case.pop("index")
    scale = case.pop("scale", 1.0)
    w = wl.config(idx, scale, **case)
    g = oracle.geom_of(w)
    lo = oracle.obj_layout(g)
    return w, g, lo


@pytest.mark.parametrize("case", CASES, ids=lambda c: "-".join(f"{k}{v}" for k, v in c.items()))
def test_restore_equals_numpy_indexing(case):
    w, g, lo = _mk(case)
    store = hc.make_store(w, lo)
    nbytes, k_off, v_off, stride = hc.pool_geometry(w, lo)
    for layer in sorted({0, w.n_layers - 1}):
        pool0 = hc.make_pool_layer(w, lo, layer)
        pool = pool0.copy()
        rc = oracle.restore_layer(g, layer, hc.batch_of(w), store, pool, k_off, v_off, stride,
                                  w.n_pool_blocks, w.pool_hnd)
        assert rc == oracle.OK
        exp = _expected_pool_numpy(w, lo, store, pool0, layer)
        assert np.array_equal(pool, exp)
        # the block-granular multi-threaded form (the all-cores baseline) gives the same bytes,
        # and its save equals the plain save
        pool_mt = pool0.copy()
        assert oracle.move_layer_blocks_mt(g, layer, hc.batch_of(w), store, pool_mt, k_off, v_off,
                                           stride, w.n_pool_blocks, True, 7, w.pool_hnd) == 0
        assert np.array_equal(pool_mt, exp)
        st_a = [np.zeros_like(x) for x in store]
        st_b = [np.zeros_like(x) for x in store]
        assert oracle.save_layer(g, layer, hc.batch_of(w), st_a, exp, k_off, v_off, stride,
                                 w.n_pool_blocks, w.pool_hnd) == 0
        assert oracle.move_layer_blocks_mt(g, layer, hc.batch_of(w), st_b, exp, k_off, v_off,
                                           stride, w.n_pool_blocks, False, 7, w.pool_hnd) == 0
        assert all(np.array_equal(a, b) for a, b in zip(st_a, st_b))
        # blocks not in the block table are byte-unchanged (canary / background)
        touched = np.zeros(w.n_pool_blocks, dtype=bool)
        touched[w.block_ids] = True
        bb = int(lo.block_bytes)
        for plane in (k_off, v_off):
            for b in np.nonzero(~touched)[0][:200]:
                o = plane + int(b) * stride
                assert np.array_equal(pool[o:o + bb], pool0[o:o + bb])
        assert not np.array_equal(pool, pool0)


def test_identity_table_is_memcpy():
    """Identity block table + consecutive slots: restore is one contiguous copy per plane."""
    w = wl.make_workload("ident", seed=7, n_layers=2, hit_tokens=[1024], block_tokens=16,
                         obj_tokens=256, n_pool_blocks=64, consecutive_slots=True)
    w.block_ids[:] = np.arange(64, dtype=np.int32)
    g = oracle.geom_of(w)
    lo = oracle.obj_layout(g)
    store = hc.make_store(w, lo)
    nbytes, k_off, v_off, stride = hc.pool_geometry(w, lo)
    layer = 1
    pool = np.zeros(nbytes, dtype=np.uint8)
    assert oracle.restore_layer(g, layer, hc.batch_of(w), store, pool, k_off, v_off, stride,
                                w.n_pool_blocks) == 0
    lay = store[0].reshape(w.n_layers, -1)[layer]           # LAYER_MAJOR: one layer contiguous
    objs = lay.reshape(4, 2, -1)                             # 4 objects, K half / V half
    assert np.array_equal(pool[k_off:k_off + 64 * stride], objs[:, 0].reshape(-1))
    assert np.array_equal(pool[v_off:v_off + 64 * stride], objs[:, 1].reshape(-1))


# --------------------------------------------------------------------------
# invariants: round trip, untouched bytes, exec(build) == restore
# --------------------------------------------------------------------------

@pytest.mark.parametrize("case", CASES[:5] + CASES[7:],
                         ids=lambda c: "-".join(f"{k}{v}" for k, v in c.items()))
def test_round_trip_and_untouched(case):
    w, g, lo = _mk(case)
    store = hc.make_store(w, lo)
    nbytes, k_off, v_off, stride = hc.pool_geometry(w, lo)
    layer = w.n_layers - 1
    batch = hc.batch_of(w)
    pool = hc.make_pool_layer(w, lo, layer)
    assert oracle.restore_layer(g, layer, batch, store, pool, k_off, v_off, stride,
                                w.n_pool_blocks, w.pool_hnd) == 0
    # save into a zeroed store: covered ranges reproduce the original store, rest stays zero
    st2 = [np.zeros_like(s) for s in store]
    assert oracle.save_layer(g, layer, batch, st2, pool, k_off, v_off, stride,
                             w.n_pool_blocks, w.pool_hnd) == 0
    covered = [np.zeros(s.nbytes, dtype=bool) for s in store]
    tb = int(lo.token_bytes)
    for r in range(w.n_req):
        hit = int(w.hit_tokens[r])
        for t in list(range(0, hit, max(1, hit // 37))) + [hit - 1]:
            for kv in (0, 1):
                d, so, blk, ro = oracle.token_location(g, layer, batch, r, t, kv)
                assert np.array_equal(st2[d][so:so + tb], store[d][so:so + tb])
    total = sum(int(s.astype(bool).sum()) for s in st2)
    payload = w.total_tokens * 2 * tb
    assert total <= payload                      # nothing outside the covered ranges was written
    assert total > 0.9 * payload                 # N(0,1) bf16 bytes are rarely zero
    # restore the saved store through a different block table: same logical content
    w2 = wl.make_workload("alt", seed=w.seed + 99, n_layers=w.n_layers,
                          hit_tokens=w.hit_tokens, block_tokens=w.block_tokens,
                          obj_tokens=w.obj_tokens, n_devices=w.n_devices, layout=w.layout,
                          n_pool_blocks=w.n_pool_blocks, pool_interleaved=w.pool_interleaved)
    batch2 = (w.hit_tokens, w.obj_start, w.obj_slot, w2.blk_start, w2.block_ids)
    pool2 = np.zeros(nbytes, dtype=np.uint8)
    assert oracle.restore_layer(g, layer, batch2, st2, pool2, k_off, v_off, stride,
                                w.n_pool_blocks, w.pool_hnd) == 0
    bb = int(lo.block_bytes)
    for plane in (k_off, v_off):
        for i in range(0, len(w.block_ids), max(1, len(w.block_ids) // 64)):
            a = plane + int(w.block_ids[i]) * stride
            b = plane + int(w2.block_ids[i]) * stride
            assert np.array_equal(pool[a:a + bb], pool2[b:b + bb])


@pytest.mark.parametrize("case", CASES, ids=lambda c: "-".join(f"{k}{v}" for k, v in c.items()))
@pytest.mark.parametrize("capacity", [2048, 3])
def test_descriptors(case, capacity):
    w, g, lo = _mk(case)
    nbytes, k_off, v_off, stride = hc.pool_geometry(w, lo)
    base = 0x7F0000000000
    layer = w.n_layers - 1
    batch = hc.batch_of(w)
    flag = oracle.OP_HND if w.pool_hnd else 0
    rowb = w.head_dim * w.elem_bytes
    rc, sqes, sgl, num = oracle.build_descriptors(g, layer, oracle.OP_READ | flag, batch,
                                                  base + k_off, base + v_off, stride, capacity)
    assert rc == 0
    assert np.all(sqes["opcode"] == (oracle.OP_READ | flag))
    tb, bb = int(lo.token_bytes), int(lo.block_bytes)
    payload = w.total_tokens * 2 * tb
    # total length = payload; sgl_first = exclusive prefix sum of sgl_count
    assert int(sqes["len"].sum()) == payload
    assert np.array_equal(sqes["sgl_first"], np.cumsum(sqes["sgl_count"]) - sqes["sgl_count"])
    assert int(sqes["sgl_count"].sum()) == len(sgl) == 2 * len(w.block_ids)
    assert np.all(sqes["len"] == sqes["sgl_count"].astype(np.uint64) * bb)
    assert np.all(sgl["len"] == bb)
    # strictly increasing (dev, offset), runs disjoint and never exactly adjacent
    key = [(int(s["dev"]), int(s["src_off"])) for s in sqes]
    assert key == sorted(key) and len(set(key)) == len(key)
    for a, b in zip(sqes[:-1], sqes[1:]):
        if a["dev"] == b["dev"]:
            assert int(a["src_off"]) + int(a["len"]) < int(b["src_off"])
    # every (request, token-block, kv) destination appears exactly once
    want = set()
    for kv, off in ((0, k_off), (1, v_off)):
        for b in w.block_ids:
            want.add(base + off + int(b) * stride)
    got = [int(a) for a in sgl["addr"]]
    assert len(got) == len(set(got)) and set(got) == want
    # bounds on the number of contexts
    n_items = 2 * int(((w.hit_tokens.astype(np.int64) + w.obj_tokens - 1) // w.obj_tokens).sum())
    assert len(set(int(s["dev"]) for s in sqes)) <= len(sqes) <= n_items
    # IOCB packing
    assert len(num) == max(1, -(-len(sqes) // capacity))
    assert int(num.sum()) == len(sqes) and np.all(num[:-1] == capacity)
    # executing the descriptors reproduces the plain restore, byte for byte
    store = hc.make_store(w, lo)
    pool_a = hc.make_pool_layer(w, lo, layer)
    pool_b = pool_a.copy()
    assert oracle.restore_layer(g, layer, batch, store, pool_a, k_off, v_off, stride,
                                w.n_pool_blocks, w.pool_hnd) == 0
    assert oracle.exec_descriptors(sqes, sgl, store, pool_b, base, w.n_kv_heads, rowb) == 0
    assert np.array_equal(pool_a, pool_b)
    # and the WRITE direction reproduces the plain save
    rc, sq_w, sgl_w, _ = oracle.build_descriptors(g, layer, oracle.OP_WRITE | flag, batch,
                                                  base + k_off, base + v_off, stride, capacity)
    assert rc == 0 and np.all(sq_w["opcode"] == (oracle.OP_WRITE | flag))
    st_a = [np.zeros_like(s) for s in store]
    st_b = [np.zeros_like(s) for s in store]
    assert oracle.save_layer(g, layer, batch, st_a, pool_a, k_off, v_off, stride,
                             w.n_pool_blocks, w.pool_hnd) == 0
    assert oracle.exec_descriptors(sq_w, sgl_w, st_b, pool_a, base, w.n_kv_heads, rowb) == 0
    for a, b in zip(st_a, st_b):
        assert np.array_equal(a, b)


SHARED = [
    dict(index=2, scale=0.05, n_layers=2, shared_prefix_frac=0.75),
    dict(index=2, scale=0.05, n_layers=2, shared_prefix_frac=1.0, n_devices=2,
         layout=wl.LAYOUT_FILE_MAJOR),
    dict(index=4, scale=0.04, n_layers=2, shared_prefix_frac=1.0),
    dict(index=2, scale=0.05, n_layers=2, shared_prefix_frac=0.75, pool_hnd=True),
]


@pytest.mark.parametrize("case", SHARED, ids=lambda c: "-".join(f"{k}{v}" for k, v in c.items()))
@pytest.mark.parametrize("capacity", [2048, 3])
def test_descriptors_of_requests_with_a_shared_prefix(case, capacity):
    """Several requests of a batch hit the same stored objects: each distinct source is named
    once, every destination still appears exactly once, and executing the descriptors is the
    plain restore."""
    w, g, lo = _mk(case)
    nbytes, k_off, v_off, stride = hc.pool_geometry(w, lo)
    base = 0x7F0000000000
    layer = w.n_layers - 1
    batch = hc.batch_of(w)
    flag = oracle.OP_HND if w.pool_hnd else 0
    rowb = w.head_dim * w.elem_bytes
    rc, sqes, sgl, num = oracle.build_descriptors(g, layer, oracle.OP_READ | flag, batch,
                                                  base + k_off, base + v_off, stride, capacity)
    assert rc == 0
    tb, bb = int(lo.token_bytes), int(lo.block_bytes)
    # distinct sources, counted from the inputs alone: (slot, tokens of it that are hit)
    distinct = set()
    for r in range(w.n_req):
        hit = int(w.hit_tokens[r])
        for c in range(-(-hit // w.obj_tokens)):
            distinct.add((int(w.obj_slot[int(w.obj_start[r]) + c]), min(w.obj_tokens, hit - c * w.obj_tokens)))
    unique_bytes = sum(2 * v * tb for _, v in distinct)
    payload = w.total_tokens * 2 * tb
    assert unique_bytes < payload                               # the batch does share objects
    assert int(sqes["len"].sum()) == unique_bytes
    assert len(sgl) == 2 * len(w.block_ids) == int(sqes["sgl_count"].sum())
    dup = (sgl["id"] & oracle.SGL_DUP) != 0
    assert int((~dup).sum()) * bb == unique_bytes and int(dup.sum()) * bb == payload - unique_bytes
    assert np.array_equal(sqes["sgl_first"], np.cumsum(sqes["sgl_count"]) - sqes["sgl_count"])
    for s_ in sqes:
        e0, e1 = int(s_["sgl_first"]), int(s_["sgl_first"]) + int(s_["sgl_count"])
        assert not dup[e0]                                      # a context never opens with a repeat
        assert int((~dup[e0:e1]).sum()) * bb == int(s_["len"])
    # contexts in (device, offset) order, a context never starts exactly where its predecessor
    # ends (they would have merged); contexts overlap only where prefixes of different length of
    # one object are hit (1-token pages with ragged hits)
    for a, b in zip(sqes[:-1], sqes[1:]):
        assert (int(a["dev"]), int(a["src_off"])) <= (int(b["dev"]), int(b["src_off"]))
        if a["dev"] == b["dev"]:
            assert int(a["src_off"]) + int(a["len"]) != int(b["src_off"])
    # every destination block (K and V of every request's table) exactly once
    want = {base + off + int(b) * stride for off in (k_off, v_off) for b in w.block_ids}
    got = [int(a) for a in sgl["addr"]]
    assert len(got) == len(set(got)) and set(got) == want
    assert np.array_equal(sgl["id"] & 0x7FFFFFFF,
                          ((sgl["addr"] - np.uint64(base)) % np.uint64(v_off if v_off > stride else stride)
                           // np.uint64(stride)).astype(np.uint32)) or w.pool_interleaved
    assert int(num.sum()) == len(sqes) and len(num) == max(1, -(-len(sqes) // capacity))
    # executing the descriptors reproduces the plain restore, byte for byte
    store = hc.make_store(w, lo)
    pool_a = hc.make_pool_layer(w, lo, layer)
    pool_b = pool_a.copy()
    assert oracle.restore_layer(g, layer, batch, store, pool_a, k_off, v_off, stride,
                                w.n_pool_blocks, w.pool_hnd) == 0
    assert oracle.exec_descriptors(sqes, sgl, store, pool_b, base, w.n_kv_heads, rowb) == 0
    assert np.array_equal(pool_a, pool_b)
    assert not np.array_equal(pool_a, hc.make_pool_layer(w, lo, layer))


def test_iocbs_cut_by_entries_hand_worked():
    """IOCBs of equal work: boundaries every `per` scatter-gather entries, moved back so that a
    repeat stays with the bytes it repeats; a context crossing a boundary is cut in two."""
    g = oracle.geom(2, 8, 128, 2, 16, 256, 1, oracle.LAYER_MAJOR, 8)
    lo = oracle.obj_layout(g)
    bb = int(lo.block_bytes)
    # one request, 512 tokens in the consecutive slots 3 and 4: one context of 64 entries
    batch = ([512], [0, 2], [3, 4], [0, 32], list(range(32)))
    rc, sqes, sgl, num = oracle.build_descriptors(g, 1, 0, batch, 0, 1 << 30, bb, 2048, 24)
    assert rc == 0 and len(sgl) == 64
    base = int(lo.stride_layer) + 3 * int(lo.obj_bytes)
    assert [(int(s["src_off"]) - base, int(s["len"]), int(s["sgl_first"]), int(s["sgl_count"]))
            for s in sqes] == [(0, 24 * bb, 0, 24), (24 * bb, 24 * bb, 24, 24), (48 * bb, 16 * bb, 48, 16)]
    assert list(num) == [1, 1, 1]
    # a budget that covers everything: one IOCB, the context as it is
    rc, sq1, sg1, num1 = oracle.build_descriptors(g, 1, 0, batch, 0, 1 << 30, bb, 2048, 1000)
    rc, sq0, sg0, num0 = oracle.build_descriptors(g, 1, 0, batch, 0, 1 << 30, bb, 2048)
    assert sq1.tobytes() == sq0.tobytes() and sg1.tobytes() == sg0.tobytes() and list(num1) == [1]
    # two requests sharing slot 5: entries go (block j of request 0, its repeat for request 1);
    # with 5 entries per IOCB the odd boundaries 5, 15, ... fall on repeats and move back by one
    batch = ([256, 256], [0, 1, 2], [5, 5], [0, 16, 32], list(range(32)))
    rc, sqes, sgl, num = oracle.build_descriptors(g, 0, 0, batch, 0, 1 << 30, bb, 2048, 5)
    assert rc == 0 and len(sgl) == 64
    firsts = [int(s["sgl_first"]) for s in sqes]
    assert firsts == [0, 4, 10, 14, 20, 24, 30, 34, 40, 44, 50, 54, 60]
    assert list(num) == [1] * 13
    assert [int(s["sgl_count"]) for s in sqes] == [4, 6, 4, 6, 4, 6, 4, 6, 4, 6, 4, 6, 4]
    # the bytes are named once: 2, 3, 2, 3, ... source blocks per piece, back to back
    assert [int(s["len"]) // bb for s in sqes] == [2, 3] * 6 + [2]
    off5 = 5 * int(lo.obj_bytes)
    assert [int(s["src_off"]) - off5 for s in sqes] == [bb * x for x in (0, 2, 5, 7, 10, 12, 15, 17, 20, 22, 25, 27, 30)]


@pytest.mark.parametrize("case", [CASES[0], CASES[2], CASES[3]] + SHARED,
                         ids=lambda c: "-".join(f"{k}{v}" for k, v in c.items()))
@pytest.mark.parametrize("per", [7, 64, 1000])
def test_iocbs_cut_by_entries_invariants(case, per):
    w, g, lo = _mk(case)
    nbytes, k_off, v_off, stride = hc.pool_geometry(w, lo)
    base = 0x7F0000000000
    layer = w.n_layers - 1
    batch = hc.batch_of(w)
    flag = oracle.OP_HND if w.pool_hnd else 0
    rowb = w.head_dim * w.elem_bytes
    bb = int(lo.block_bytes)
    rc, sq0, sg0, num0 = oracle.build_descriptors(g, layer, oracle.OP_READ | flag, batch,
                                                  base + k_off, base + v_off, stride, 1 << 20)
    rc, sqes, sgl, num = oracle.build_descriptors(g, layer, oracle.OP_READ | flag, batch,
                                                  base + k_off, base + v_off, stride, 1 << 20, per)
    assert rc == 0
    assert sgl.tobytes() == sg0.tobytes()                       # the entries do not change
    ne = len(sgl)
    assert len(num) == max(1, -(-ne // per)) and int(num.sum()) == len(sqes)
    dup = (sgl["id"] & oracle.SGL_DUP) != 0
    # the contexts, IOCB by IOCB, partition the entries in order
    assert int(sqes["sgl_first"][0]) == 0
    ends = sqes["sgl_first"].astype(np.int64) + sqes["sgl_count"].astype(np.int64)
    assert np.array_equal(ends[:-1], sqes["sgl_first"][1:]) and int(ends[-1]) == ne
    at = 0
    for k, n in enumerate(num):
        first = int(sqes["sgl_first"][at]) if n else None
        last = int(ends[at + n - 1]) if n else None
        if n:
            # an IOCB starts at its boundary moved back over repeats, and holds at most `per`
            # entries more than that
            want = min(k * per, ne)
            while 0 < want < ne and dup[want]:
                want -= 1
            assert first == want and last - first <= per + (k * per - want)
            assert not dup[first]
        at += n
    for s_ in sqes:
        e0, e1 = int(s_["sgl_first"]), int(s_["sgl_first"]) + int(s_["sgl_count"])
        assert not dup[e0] and int((~dup[e0:e1]).sum()) * bb == int(s_["len"])
    assert int(sqes["len"].sum()) == int(sq0["len"].sum())       # the same bytes are named
    # executing the cut contexts is the plain restore
    store = hc.make_store(w, lo)
    pool_a = hc.make_pool_layer(w, lo, layer)
    pool_b = pool_a.copy()
    assert oracle.restore_layer(g, layer, batch, store, pool_a, k_off, v_off, stride,
                                w.n_pool_blocks, w.pool_hnd) == 0
    assert oracle.exec_descriptors(sqes, sgl, store, pool_b, base, w.n_kv_heads, rowb) == 0
    assert np.array_equal(pool_a, pool_b)


def test_config1_closed_form_counts():
    """Config 1: 16 items, 256 SGL entries; consecutive slots give one 8 MiB context,
    pairwise non-adjacent slots give eight 1 MiB contexts (K and V halves always merge)."""
    w = wl.config(1)
    g = oracle.geom_of(w)
    lo = oracle.obj_layout(g)
    assert (lo.token_bytes, lo.block_bytes, lo.obj_kv_bytes, lo.obj_bytes) == \
        (2048, 32768, 512 * 1024, 1024 * 1024)
    nbytes, k_off, v_off, stride = hc.pool_geometry(w, lo)
    rc, sqes, sgl, num = oracle.build_descriptors(g, 0, 0, hc.batch_of(w), k_off, v_off, stride,
                                                  2048)
    assert rc == 0 and len(sgl) == 256 and len(sqes) == 1 and int(sqes["len"][0]) == 8 << 20
    assert list(num) == [1]
    w.obj_slot[:] = np.array([0, 2, 4, 6, 8, 10, 12, 14], dtype=np.uint32)[::-1]
    w.n_slots = 16
    g = oracle.geom_of(w)
    rc, sqes, sgl, num = oracle.build_descriptors(g, 0, 0, hc.batch_of(w), k_off, v_off, stride,
                                                  2048)
    assert rc == 0 and len(sqes) == 8 and np.all(sqes["len"] == 1 << 20)
    assert np.array_equal(sqes["sgl_first"], 32 * np.arange(8))
    # sorted by offset: the chunk order is reversed, so the first context carries the
    # blocks of the last chunk, K blocks before V blocks
    first = sgl[:32]
    assert np.array_equal(first["id"][:16], w.block_ids[7 * 16:8 * 16].astype(np.uint32))
    assert np.array_equal(first["id"][16:], w.block_ids[7 * 16:8 * 16].astype(np.uint32))
    assert np.all(first["addr"][:16] < v_off) and np.all(first["addr"][16:] >= v_off)


def test_partial_last_object_and_duplicates():
    """A prefix that ends inside an object: its K and V halves are not adjacent, so they stay
    separate contexts.  The same object hit by two requests is read once (one source, two
    destinations per block)."""
    g = oracle.geom(2, 8, 128, 2, 16, 256, 1, oracle.LAYER_MAJOR, 8)
    batch = ([256 + 64], [0, 2], [3, 4], [0, 20], list(range(20)))
    rc, sqes, sgl, num = oracle.build_descriptors(g, 1, 0, batch, 0, 1 << 30, 32768, 2048)
    assert rc == 0
    lo = oracle.obj_layout(g)
    base = lo.stride_layer + 3 * lo.obj_bytes
    assert [(int(s["src_off"]), int(s["len"])) for s in sqes] == [
        (base, lo.obj_bytes + 64 * 2048), (base + lo.obj_bytes + lo.obj_kv_bytes, 64 * 2048)]
    assert list(sqes["sgl_count"]) == [36, 4]
    # the same object hit by two requests is one source, read once: sorted items K(req 0),
    # K(req 1), V(req 0), V(req 1) are two groups of two; K and V are byte-adjacent, so one
    # context names the object's bytes once and lists, block by block, both destinations
    batch = ([256, 256], [0, 1, 2], [5, 5], [0, 16, 32], list(range(32)))
    rc, sqes, sgl, num = oracle.build_descriptors(g, 0, 0, batch, 0, 1 << 30, 32768, 2048)
    assert rc == 0
    kvb = int(lo.obj_kv_bytes)
    assert [(int(s["src_off"]) - 5 * lo.obj_bytes, int(s["len"]), int(s["sgl_count"]))
            for s in sqes] == [(0, 2 * kvb, 64)]
    D = oracle.SGL_DUP
    want_ids = [x for j in range(16) for x in (j, (16 + j) | D)]
    assert list(sgl["id"][:32]) == want_ids and list(sgl["id"][32:]) == want_ids
    assert np.all(sgl["addr"][:32] < 1 << 30) and np.all(sgl["addr"][32:] >= 1 << 30)
    assert [int(a) for a in sgl["addr"][:4]] == [0, 16 * 32768, 32768, 17 * 32768]
    # a partial hit of the same object is a different source (other length), read on its own.
    # Sorted by (offset, length): K of the 64-token hit [0, 128K), K of the full hit [0, 512K),
    # V of the 64-token hit [512K, 640K), V of the full hit [512K, 1M).  The full K ends where
    # the short V starts, so those two merge; the full V starts before its predecessor ends.
    batch = ([256, 64], [0, 1, 2], [5, 5], [0, 16, 20], list(range(20)))
    rc, sqes, sgl, num = oracle.build_descriptors(g, 0, 0, batch, 0, 1 << 30, 32768, 2048)
    assert rc == 0
    p64 = 64 * 2048
    assert [(int(s["src_off"]) - 5 * lo.obj_bytes, int(s["len"]), int(s["sgl_count"]))
            for s in sqes] == [(0, p64, 4), (0, kvb + p64, 20), (kvb, kvb, 16)]
    assert not np.any(sgl["id"] & D)
    assert list(sgl["id"]) == [16, 17, 18, 19] + list(range(16)) + [16, 17, 18, 19] + list(range(16))


def test_many_requests_on_one_object():
    """40 requests on one object: one source with 40 destinations per block.  Sorted items:
    K x 40, V x 40; K and V are byte-adjacent, so one context names the object once and lists
    40 entries per block, all but the first of each block flagged as repeats."""
    g = oracle.geom(1, 8, 128, 2, 16, 256, 1, oracle.LAYER_MAJOR, 8)
    lo = oracle.obj_layout(g)
    kvb, bb = int(lo.obj_kv_bytes), int(lo.block_bytes)
    n = 40
    batch = ([256] * n, list(range(n + 1)), [5] * n, [16 * r for r in range(n + 1)],
             list(range(16 * n)))
    rc, sqes, sgl, num = oracle.build_descriptors(g, 0, 0, batch, 0, 1 << 30, bb, 2048)
    assert rc == 0 and len(sgl) == 2 * 16 * n
    off5 = 5 * int(lo.obj_bytes)
    assert [(int(s["src_off"]) - off5, int(s["len"]), int(s["sgl_count"])) for s in sqes] == [
        (0, 2 * kvb, 2 * 16 * n)]
    D = oracle.SGL_DUP
    # block 0 of K: requests 0..39 side by side, only the first without the repeat flag
    assert list(sgl["id"][:n]) == [0] + [(16 * r) | D for r in range(1, n)]
    assert int(sgl["id"][n]) == 1 and int(sgl["id"][n + 1]) == 17 | D     # then block 1
    store = [np.arange(int(lo.dev_bytes), dtype=np.uint64).astype(np.uint8)]
    pool_a = np.zeros(2 * 16 * n * bb, dtype=np.uint8)
    pool_b = pool_a.copy()
    v_off = 16 * n * bb
    assert oracle.restore_layer(g, 0, batch, store, pool_a, 0, v_off, bb, 16 * n) == 0
    rc, sqes, sgl, num = oracle.build_descriptors(g, 0, 0, batch, 1 << 40, (1 << 40) + v_off, bb, 2048)
    assert oracle.exec_descriptors(sqes, sgl, store, pool_b, 1 << 40) == 0
    assert np.array_equal(pool_a, pool_b)


def test_empty_and_invalid():
    g = oracle.geom(2, 8, 128, 2, 16, 256, 1, oracle.LAYER_MAJOR, 8)
    rc, sqes, sgl, num = oracle.build_descriptors(g, 0, 0, ([0], [0, 0], [], [0, 0], []), 0, 0,
                                                  32768, 2048)
    assert rc == 0 and len(sqes) == 0 and len(sgl) == 0 and list(num) == [0]
    rc, *_ = oracle.build_descriptors(g, 0, 0, ([8], [0, 1], [0], [0, 1], [0]), 0, 0, 32768, 16)
    assert rc == oracle.EINVAL                  # hit not a multiple of the block size
    rc, *_ = oracle.build_descriptors(g, 2, 0, ([16], [0, 1], [0], [0, 1], [0]), 0, 0, 32768, 16)
    assert rc == oracle.EINVAL                  # layer out of range
    rc, *_ = oracle.build_descriptors(g, 0, 0, ([32], [0, 1], [0], [0, 1], [0]), 0, 0, 32768, 16)
    assert rc == oracle.EINVAL                  # block-table row too short
    with pytest.raises(ValueError):
        oracle.obj_layout(oracle.geom(2, 8, 128, 2, 16, 24, 1, 0, 8))


# --------------------------------------------------------------------------
# counts the paper prints (tests/golden/paper_counts.txt)
# --------------------------------------------------------------------------

def _golden():
    out = {}
    with open(os.path.join(GOLDEN, "paper_counts.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                k, v = line.split("=")
                out[k.strip()] = int(v)
    return out


def test_paper_counts():
    gold = _golden()
    # Section 2.2: 64 layers, block 64, 128K tokens, one object per block and per K/V
    n_tok = 128 * 1024
    w = wl.make_workload("q", seed=1, n_layers=64, hit_tokens=[n_tok], block_tokens=64,
                         obj_tokens=64, n_pool_blocks=4096, consecutive_slots=False,
                         slot_mean_run=1.0, slot_space_factor=2.0)
    g = oracle.geom_of(w)
    # make no two slots adjacent so no K|V pair merges with a neighbour
    w.obj_slot[:] = (2 * np.random.default_rng(0).permutation(len(w.obj_slot))).astype(np.uint32)
    g.n_slots = 2 * len(w.obj_slot)
    rc, sqes, sgl, num = oracle.build_descriptors(g, 0, 0, hc.batch_of(w), 0, 1 << 40, 65536 * 2,
                                                  2048)
    assert rc == 0
    per_layer_objects = len(sgl)                  # one K and one V object per block
    assert per_layer_objects * 64 == gold["qwen3_32b_128k_objects"]
    # Section 2.2: 256-token chunks, 128K tokens -> "more than 1,000" chunk accesses (K and V)
    w = wl.make_workload("c", seed=1, n_layers=1, hit_tokens=[n_tok], block_tokens=16,
                         obj_tokens=256, consecutive_slots=True)
    g = oracle.geom_of(w)
    lo = oracle.obj_layout(g)
    assert 2 * len(w.obj_slot) == gold["lmcache_128k_chunk_accesses"] > 1000
    # Section 3.1: 60 GB of KV at 64 KB per SGL entry -> 983,040 entries of 16 B = 15 MB
    entries = 60 * 1024 ** 3 // (64 * 1024)
    assert entries == gold["sgl_entries_60gb"]
    assert entries * oracle.SGL_DTYPE.itemsize == gold["sgl_bytes_60gb"] == 15 * 1024 ** 2
    assert 60 * 1024 ** 3 // 4096 == gold["prp_pages_60gb"]
    # Section 3.2: one IOCB holds 2048 contexts = 2 SMs x 64 warps x 32 threads / 2
    assert 2 * 64 * 32 // 2 == gold["ioctx_per_iocb"]


def test_head_major_block_by_enumeration():
    """Head-major pool block, tiny and explicit: the block is written down in pool order
    (for each head, for each token, one row) and compared with what restore leaves there."""
    H, D, bt = 3, 8, 4                                   # rows of 16 bytes
    g = oracle.geom(1, H, D, 2, bt, 2 * bt, 1, oracle.LAYER_MAJOR, 2)
    row = D * 2
    store = np.zeros(2 * 2 * 2 * bt * H * row, dtype=np.uint8)     # 2 slots x {K,V} x 8 tokens
    cells = store.reshape(2, 2, 2 * bt, H, row)                    # [slot][kv][token][head][row]
    for s in range(2):
        for kv in range(2):
            for t in range(2 * bt):
                for h in range(H):
                    cells[s, kv, t, h, :] = [s + 1, kv + 1, t + 1, h + 1] * (row // 4)
    n_pool = 5
    ids = [3, 0]                                          # token 0..3 -> block 3, 4..7 -> block 0
    batch = ([2 * bt], [0, 1], [1], [0, 2], ids)          # one request, object slot 1
    pool = np.zeros(2 * n_pool * bt * H * row, dtype=np.uint8)
    bb = bt * H * row
    assert oracle.restore_layer(g, 0, batch, [store], pool, 0, n_pool * bb, bb, n_pool, True) == 0
    for kv in range(2):
        for j, blk in enumerate(ids):
            want = []
            for h in range(H):                            # pool order: head, then token
                for tt in range(bt):
                    want += [2, kv + 1, j * bt + tt + 1, h + 1] * (row // 4)
            o = kv * n_pool * bb + blk * bb
            assert pool[o:o + bb].tolist() == want
    untouched = [b for b in range(n_pool) if b not in ids]
    for b in untouched:
        assert not pool[b * bb:(b + 1) * bb].any()
    # and back
    st2 = np.zeros_like(store)
    assert oracle.save_layer(g, 0, batch, [st2], pool, 0, n_pool * bb, bb, n_pool, True) == 0
    assert np.array_equal(st2.reshape(2, -1)[1], store.reshape(2, -1)[1]) and not st2.reshape(2, -1)[0].any()


def test_row_location_agrees_with_restore():
    """The single-row locator used for sampled checks at full size names exactly the bytes
    that restore moves, for both element orders of a pool block."""
    for hnd in (False, True):
        w = wl.config(2, 0.03, n_layers=2, pool_hnd=hnd)
        g = oracle.geom_of(w)
        lo = oracle.obj_layout(g)
        store = hc.make_store(w, lo)
        nbytes, k_off, v_off, stride = hc.pool_geometry(w, lo)
        pool = np.zeros(nbytes, dtype=np.uint8)
        batch = hc.batch_of(w)
        assert oracle.restore_layer(g, 1, batch, store, pool, k_off, v_off, stride,
                                    w.n_pool_blocks, hnd) == 0
        row = w.head_dim * w.elem_bytes
        rng = np.random.default_rng(0)
        for _ in range(300):
            r = int(rng.integers(0, w.n_req)); t = int(rng.integers(0, int(w.hit_tokens[r])))
            kv = int(rng.integers(0, 2)); hd = int(rng.integers(0, w.n_kv_heads))
            d, so, blk, bo = oracle.row_location(g, 1, batch, r, t, kv, hd, hnd)
            po = (v_off if kv else k_off) + blk * stride + bo
            assert np.array_equal(pool[po:po + row], store[d][so:so + row])
