"""The score kernel's launch plan, built and checked on the host alone (no GPU): random ragged
batches, head counts and SM counts through cake_plan_check, which verifies tile coverage, the
order of every CTA's program, the wave span of merge groups and the table bounds."""
import ctypes

import numpy as np

from paper_2503_12491_b200 import binding


def check(n_q, n_kv, window, head_dim, seq_lens, n_sm, reserved):
    lib = binding.load_library()
    total = int(sum(seq_lens))
    cfg = binding.CakeConfig(4, n_q, n_kv, head_dim, window, 7, 0, 0, binding.CAKE_DTYPE_BF16, 1.0, 1.0,
                             1.0, 4 * window + 64, len(seq_lens), total, 0, 0, 0.0)
    cu = np.concatenate([[0], np.cumsum(seq_lens)]).astype(np.int64)
    info = (ctypes.c_int32 * 8)()
    rc = lib.cake_plan_check(ctypes.byref(cfg), n_sm, reserved, len(seq_lens),
                             cu.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)), info)
    return rc, list(info)


def test_benchmark_shapes():
    rc, info = check(32, 8, 32, 128, [131072], 148, 16)
    assert rc == 0 and info[0] == 128 and info[1] == 8 and info[2] == 1 and info[7] == 0
    rc, info = check(32, 32, 32, 128, [4096], 148, 16)
    assert rc == 0 and info[7] == 0 and info[2] in (1, 2, 4, 8, 16, 32)
    rc, info = check(32, 8, 32, 128, [32768], 148, 16)
    assert rc == 0 and info[7] == 0


def test_random_ragged_batches_and_sm_counts():
    rng = np.random.default_rng(20250312)
    shapes = [(32, 8, 32, 128), (8, 2, 16, 128), (4, 4, 32, 64), (16, 2, 16, 128), (8, 1, 8, 64), (3, 3, 96, 128)]
    seen_ways = set()
    for trial in range(300):
        n_q, n_kv, window, d = shapes[trial % len(shapes)]
        n_req = int(rng.integers(1, 9))
        kind = trial % 4
        if kind == 0:
            lens = rng.integers(window, 3000, size=n_req)
        elif kind == 1:
            lens = rng.integers(8192, 70000, size=n_req)
        elif kind == 2:                                   # pairs of ~10 to 11 MB: waves of two or three pairs
            lens = rng.integers(38000, 45000, size=n_req)
        else:
            lens = np.where(rng.random(n_req) < 0.5, rng.integers(window, 400, size=n_req),
                            rng.integers(20000, 140000, size=n_req))
        n_sm = int(rng.choice([8, 33, 74, 108, 132, 148]))
        reserved = int(rng.choice([0, 4, 16, 40, 74]))
        if reserved >= n_sm:
            reserved = n_sm // 2
        rc, info = check(n_q, n_kv, window, d, [int(x) for x in lens], n_sm, reserved)
        assert rc == 0, (trial, rc, info, lens.tolist(), n_sm, reserved)
        assert info[7] == 0 and 1 <= info[0] <= n_sm - reserved
        seen_ways.add(info[2])
    assert seen_ways >= {1, 4}                            # both merger modes were exercised


def test_shapes_of_the_simt_path_are_refused():
    rc, info = check(4, 4, 16, 64, [512], 148, 16)       # 16 rows: not a multiple of 32
    assert rc == binding.CAKE_ERR_ARG
