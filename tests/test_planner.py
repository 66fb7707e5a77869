"""Block planner: the oracle against the paper's Table 1 and against properties, and the C-ABI
planner (host code, no GPU needed) against the oracle."""
import ctypes
import math
import os

import numpy as np
import pytest

from oracle.planner import plan_blocks

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "table1_blocks.txt")


def _table1():
    rows = []
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        name, value, scaffold, blocks = line.split()
        rows.append((name, int(value), int(scaffold), int(blocks)))
    return rows[:-1], rows[-1]


def _template(sections, rng):
    """A token template with the given (value, scaffold) counts per section, scaffold and value
    positions interleaved at random (what the counts leave open)."""
    editable, ends = [], []
    for value, scaffold in sections:
        part = np.array([1] * value + [0] * scaffold, dtype=np.uint8)
        rng.shuffle(part)
        editable.extend(part.tolist())
        ends.append(len(editable))
    return np.array(editable, dtype=np.uint8), ends


def test_table1_block_counts():
    sections, total = _table1()
    rng = np.random.default_rng(0)
    editable, ends = _template([(v, s) for _, v, s, _ in sections], rng)
    assert len(editable) == total[1] + total[2] == 404
    blocks = plan_blocks(editable, ends, 32)
    per_section = [sum(1 for b in blocks if b[2] == s) for s in range(len(sections))]
    assert per_section == [b for *_, b in sections] == [1, 6, 1, 3]
    assert len(blocks) == total[3] == 11
    # only block sizes 24..34 give the trajectory section its three blocks, and 32 is the one in that
    # range that cuts the explanation section into six full blocks
    assert [d for d in range(8, 80) if math.ceil(70 / d) == 3] == list(range(24, 35))
    assert 192 % 32 == 0 and 192 // 32 == 6


def _check_partition(editable, ends, d, blocks):
    pos = 0
    for b, e, s in blocks:
        assert b == pos and e > b                       # contiguous, in order, non-empty
        lo = ends[s - 1] if s else 0
        assert lo <= b and e <= ends[s]                 # never across a section border
        assert int(np.sum(editable[b:e])) <= d
        pos = e
    assert pos == len(editable)
    lo = 0
    for s, hi in enumerate(ends):
        n_val = int(np.sum(editable[lo:hi]))
        n_blk = sum(1 for blk in blocks if blk[2] == s)
        assert n_blk == (math.ceil(n_val / d) if n_val else (1 if hi > lo else 0))
        full = [int(np.sum(editable[b:e])) for b, e, ss in blocks if ss == s]
        assert all(v == d for v in full[:-1])           # every block but the last is full
        lo = hi


def test_partition_properties_on_random_templates():
    rng = np.random.default_rng(1)
    for _ in range(50):
        sections = [(int(rng.integers(0, 60)), int(rng.integers(0, 30))) for _ in range(int(rng.integers(1, 6)))]
        editable, ends = _template(sections, rng)
        if len(editable) == 0:
            continue
        d = int(rng.integers(1, 40))
        _check_partition(editable, ends, d, plan_blocks(editable, ends, d))


def _c_plan(editable, ends, d, cap=64):
    from paper_2605_23163_b200 import fdd
    L = fdd.lib()
    L.fdd_plan_blocks.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                  ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int,
                                  ctypes.POINTER(ctypes.c_int)]
    L.fdd_plan_blocks.restype = ctypes.c_int
    ed = np.ascontiguousarray(editable, dtype=np.uint8)
    en = np.ascontiguousarray(ends, dtype=np.int32)
    bb, be, bs = (np.zeros(cap, dtype=np.int32) for _ in range(3))
    n = ctypes.c_int(-1)
    st = L.fdd_plan_blocks(ed.ctypes.data, en.ctypes.data, len(en), len(ed), d, bb.ctypes.data, be.ctypes.data,
                           bs.ctypes.data, cap, ctypes.byref(n))
    return st, [(int(bb[i]), int(be[i]), int(bs[i])) for i in range(max(n.value, 0))], n.value


def test_c_planner_matches_oracle():
    pytest.importorskip("paper_2605_23163_b200.fdd")
    from paper_2605_23163_b200 import fdd
    if not os.path.exists(fdd.LIB_PATH):
        pytest.skip("library not built")
    rng = np.random.default_rng(2)
    sections, _ = _table1()
    editable, ends = _template([(v, s) for _, v, s, _ in sections], rng)
    st, blocks, n = _c_plan(editable, ends, 32)
    assert st == 0 and blocks == plan_blocks(editable, ends, 32) and n == 11
    for _ in range(30):
        secs = [(int(rng.integers(0, 60)), int(rng.integers(0, 30))) for _ in range(int(rng.integers(1, 6)))]
        editable, ends = _template(secs, rng)
        if len(editable) == 0:
            continue
        d = int(rng.integers(1, 40))
        st, blocks, n = _c_plan(editable, ends, d, cap=256)
        assert st == 0 and blocks == plan_blocks(editable, ends, d)
    # errors: too little room, bad section ends
    st, _, n = _c_plan(editable, ends, 1, cap=1)
    assert st == fdd.FDD_ERR_CAPACITY or n <= 1
    st, _, _ = _c_plan(np.ones(4, dtype=np.uint8), [2, 3], 2)
    assert st == fdd.FDD_ERR_INVALID_ARG
