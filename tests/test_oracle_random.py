"""Randomised small cases: the C oracle against a second implementation written as plain
Python loops over nested lists (no byte-offset arithmetic shared with the oracle: the store is
a dict keyed by (device, file index, layer, kv, token, head), the pool a dict keyed by
(kv, block, token, head))."""
import numpy as np
import pytest

import oracle


def _case(seed):
    rng = np.random.default_rng(seed)
    H = int(rng.choice([1, 2, 4]))
    row = int(rng.choice([4, 8, 16]))                  # bytes per head per token
    bt = int(rng.choice([1, 2, 4]))
    ot = bt * int(rng.choice([1, 2, 3]))
    L = int(rng.integers(1, 4))
    n_dev = int(rng.integers(1, 4))
    layout = int(rng.choice([oracle.FILE_MAJOR, oracle.LAYER_MAJOR]))
    n_req = int(rng.integers(1, 4))
    hits = [int(rng.integers(0, 9)) * bt for _ in range(n_req)]
    n_objs = [-(-h // ot) for h in hits]
    n_slots = max(sum(n_objs) + int(rng.integers(0, 4)), 1)
    slots = rng.permutation(n_slots)[:sum(n_objs)].tolist()
    # half of the multi-request cases share leading objects with request 0 (a common prefix
    # stored once): the same slot is then hit by several requests
    shared = False
    if n_req > 1 and rng.random() < 0.7:
        pos = np.concatenate([[0], np.cumsum(n_objs)]).tolist()
        for r in range(1, n_req):
            m = min(n_objs[0], n_objs[r])
            k = int(rng.integers(min(1, m), m + 1))
            slots[pos[r]:pos[r] + k] = slots[pos[0]:pos[0] + k]
            shared = shared or k > 0
    n_blks = [h // bt for h in hits]
    n_pool = sum(n_blks) + int(rng.integers(1, 5))
    blocks = rng.permutation(n_pool)[:sum(n_blks)].tolist()
    hnd = bool(rng.random() < 0.5)
    interleaved = bool(rng.random() < 0.5)
    pad = int(rng.choice([0, 0, 8]))
    return dict(H=H, row=row, bt=bt, ot=ot, L=L, n_dev=n_dev, layout=layout, hits=hits,
                n_objs=n_objs, n_slots=n_slots, slots=slots, n_blks=n_blks, n_pool=n_pool,
                blocks=blocks, hnd=hnd, interleaved=interleaved, pad=pad, rng=rng, shared=shared)


def _store_as_dict(c, store):
    """Walk every device region in storage order and name each row."""
    n_local = -(-c["n_slots"] // c["n_dev"])
    out = {}
    for d in range(c["n_dev"]):
        pos = 0
        files = range(n_local)
        order = ([(f, l) for f in files for l in range(c["L"])] if c["layout"] == oracle.FILE_MAJOR
                 else [(f, l) for l in range(c["L"]) for f in files])
        for f, l in order:
            for kv in (0, 1):
                for tok in range(c["ot"]):
                    for h in range(c["H"]):
                        out[(d, f, l, kv, tok, h)] = (d, pos)
                        pos += c["row"]
        assert pos == store[d].nbytes
    return out


def _pool_pos(c, kv, blk, tok, h):
    bb = c["bt"] * c["H"] * c["row"]
    step = bb + c["pad"]
    inner = (h * c["bt"] + tok) * c["row"] if c["hnd"] else (tok * c["H"] + h) * c["row"]
    if c["interleaved"]:
        return (blk * 2 + kv) * step + inner
    return (kv * c["n_pool"] + blk) * step + inner


@pytest.mark.parametrize("seed", range(60))
def test_restore_and_save_against_python_loops(seed):
    c = _case(seed)
    rng = c["rng"]
    g = oracle.geom(c["L"], c["H"], c["row"], 1, c["bt"], c["ot"], c["n_dev"], c["layout"], c["n_slots"])
    lo = oracle.obj_layout(g)
    store = [rng.integers(0, 256, int(lo.dev_bytes), dtype=np.uint8) for _ in range(c["n_dev"])]
    bb = c["bt"] * c["H"] * c["row"]
    step = bb + c["pad"]
    pool0 = rng.integers(0, 256, 2 * c["n_pool"] * step, dtype=np.uint8)
    os_ = np.concatenate([[0], np.cumsum(c["n_objs"])]).tolist()
    bs_ = np.concatenate([[0], np.cumsum(c["n_blks"])]).tolist()
    batch = (c["hits"], os_, c["slots"], bs_, c["blocks"])
    if c["interleaved"]:
        k_off, v_off, stride = 0, step, 2 * step
    else:
        k_off, v_off, stride = 0, c["n_pool"] * step, step
    names = _store_as_dict(c, store)
    layer = int(rng.integers(0, c["L"]))
    # expected restore, row by row
    exp = pool0.copy()
    moves = []
    for r, hit in enumerate(c["hits"]):
        for t in range(hit):
            slot = c["slots"][os_[r] + t // c["ot"]]
            blk = c["blocks"][bs_[r] + t // c["bt"]]
            for kv in (0, 1):
                for h in range(c["H"]):
                    d, spos = names[(slot % c["n_dev"], slot // c["n_dev"], layer, kv, t % c["ot"], h)]
                    ppos = _pool_pos(c, kv, blk, t % c["bt"], h)
                    exp[ppos:ppos + c["row"]] = store[d][spos:spos + c["row"]]
                    moves.append((d, spos, ppos))
    got = pool0.copy()
    assert oracle.restore_layer(g, layer, batch, store, got, k_off, v_off, stride, c["n_pool"],
                                c["hnd"]) == 0
    assert np.array_equal(got, exp)
    # the block-granular multi-threaded form restores the same bytes
    for n_thr in (1, 2, 3, 5):
        got_mt = pool0.copy()
        assert oracle.move_layer_blocks_mt(g, layer, batch, store, got_mt, k_off, v_off, stride,
                                           c["n_pool"], True, n_thr, c["hnd"]) == 0
        assert np.array_equal(got_mt, exp)
    # descriptors executed = plain restore (shared objects are named once, with repeat entries)
    flag = oracle.OP_HND if c["hnd"] else 0
    base = 1 << 32
    rc, sq, sg, num = oracle.build_descriptors(g, layer, oracle.OP_READ | flag, batch, base + k_off,
                                               base + v_off, stride, 3)
    assert rc == 0
    got2 = pool0.copy()
    assert oracle.exec_descriptors(sq, sg, store, got2, base, c["H"], c["row"]) == 0
    assert np.array_equal(got2, exp)
    n_dup = int(((sg["id"] & oracle.SGL_DUP) != 0).sum())
    distinct = {(c["slots"][os_[r] + t // c["ot"]], min(c["ot"], hit - (t // c["ot"]) * c["ot"]))
                for r, hit in enumerate(c["hits"]) for t in range(0, hit, c["ot"])}
    assert int(sq["len"].sum()) == sum(2 * v * c["H"] * c["row"] for _, v in distinct)
    assert (n_dup > 0) == (int(sq["len"].sum()) < 2 * sum(c["hits"]) * c["H"] * c["row"])
    if c["shared"]:
        return          # saving several requests' blocks into one object is the caller's error
    # expected save from a fresh random pool
    pool1 = rng.integers(0, 256, pool0.nbytes, dtype=np.uint8)
    st_exp = [s.copy() for s in store]
    for d, spos, ppos in moves:
        st_exp[d][spos:spos + c["row"]] = pool1[ppos:ppos + c["row"]]
    st_got = [s.copy() for s in store]
    assert oracle.save_layer(g, layer, batch, st_got, pool1, k_off, v_off, stride, c["n_pool"],
                             c["hnd"]) == 0
    for a, b in zip(st_got, st_exp):
        assert np.array_equal(a, b)
    # the block-granular, multi-threaded form used as the all-cores baseline: same bytes
    for n_thr in (1, 2, 3, 5):
        st_mt = [s.copy() for s in store]
        assert oracle.move_layer_blocks_mt(g, layer, batch, st_mt, pool1, k_off, v_off, stride,
                                           c["n_pool"], False, n_thr, c["hnd"]) == 0
        for a, b in zip(st_mt, st_exp):
            assert np.array_equal(a, b)
