"""The seeded input generators: host and device fills agree bit for bit, values look
like N(0,1), block tables and object maps have the promised structure."""
import numpy as np
import torch

from paper_2605_03375_b200 import workload as wl


def test_fill_numpy_matches_torch_and_is_random_access():
    a = wl.fill_u16_numpy(11, 3, 0, 4096)
    b = wl.fill_u16_torch(11, 3, 0, 4096, "cpu", chunk_words=300).numpy().view(np.uint16)
    assert np.array_equal(a, b)
    c = wl.fill_u16_numpy(11, 3, 1001, 777)
    assert np.array_equal(c, a[1001:1778])
    d = wl.fill_u16_torch(11, 3, 1000, 400, "cpu").numpy().view(np.uint16)
    assert np.array_equal(d, a[1000:1400])
    assert not np.array_equal(wl.fill_u16_numpy(11, 4, 0, 4096), a)
    assert not np.array_equal(wl.fill_u16_numpy(12, 3, 0, 4096), a)


def test_values_are_standard_normal_bf16():
    bits = wl.fill_u16_numpy(5, 0, 0, 1 << 18)
    f = (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    assert abs(f.mean()) < 0.01 and abs(f.std() - 1.0) < 0.01
    assert abs((np.abs(f) < 1.0).mean() - 0.6827) < 0.01


def test_config_shapes():
    w = wl.config(1)
    assert w.n_req == 1 and w.hit_tokens[0] == 2048 and len(w.block_ids) == 128
    assert w.n_pool_blocks == 1024 and len(set(w.block_ids.tolist())) == 128
    assert list(w.obj_slot) == list(range(8))
    w = wl.config(2)
    assert (w.n_layers, w.n_req, w.n_pool_blocks) == (32, 8, 40960)
    assert len(w.block_ids) == 16384 and len(w.obj_slot) == 1024
    assert len(w.occupied_blocks) == 24576                      # 60 % hold other data
    assert not set(w.block_ids.tolist()) & set(w.occupied_blocks.tolist())
    assert len(set(w.obj_slot.tolist())) == 1024 and w.obj_slot.max() < w.n_slots
    runs = 1 + int((np.diff(w.obj_slot.astype(np.int64)) != 1).sum())
    assert 60 < runs < 400                                      # runs of mean length ~8
    # fully fragmented: consecutive logical blocks are almost never neighbours
    assert (np.diff(w.block_ids) == 1).mean() < 0.01
    w = wl.config(3)
    assert (w.n_layers, w.n_req, w.obj_tokens, w.store_kind) == (80, 2, 1024, "host")
    assert len(w.block_ids) == 16384 and len(w.obj_slot) == 256
    w = wl.config(4)
    assert w.n_req == 64 and w.block_tokens == 1
    assert w.hit_tokens.min() >= 512 and w.hit_tokens.max() <= 16384
    assert len(w.block_ids) == w.total_tokens
    w2 = wl.config(4)
    assert np.array_equal(w.block_ids, w2.block_ids) and np.array_equal(w.obj_slot, w2.obj_slot)
