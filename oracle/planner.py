"""Section-aligned block planner (test infrastructure, CPU oracle).

Sec. 3.2 ("Scaffold Construction and Section-Aligned Blocks"): the output is a fixed template whose
structural tokens are frozen scaffold and whose value tokens are editable; block borders are
aligned with section borders, section s being cut into n_s = ceil(|E_s| / d) blocks (E_s = its
editable positions), and sections are decoded in their causal order.

Readings where the paper is silent: inside a section the blocks are filled from the left, every
block but the last taking exactly d editable positions; a block starts right after the previous
one ends, and ends right after its last editable position, except that the last block of a section
runs to the section's end (so scaffold tokens travel with the value tokens that follow them, and
trailing scaffold stays with the last block); a section without editable positions is one block
that needs no decoding.
"""
import math


def plan_blocks(editable, section_end, d):
    """editable: sequence of 0/1 per position; section_end: exclusive end of every section
    (increasing, the last one == len(editable)); d: editable positions per block.
    Returns a list of (begin, end, section)."""
    assert d >= 1 and len(section_end) >= 1 and section_end[-1] == len(editable)
    blocks = []
    begin_s = 0
    for s, end_s in enumerate(section_end):
        assert end_s >= begin_s
        values = [i for i in range(begin_s, end_s) if editable[i]]
        n_s = math.ceil(len(values) / d)
        if n_s == 0:
            if end_s > begin_s:
                blocks.append((begin_s, end_s, s))
        else:
            b = begin_s
            for j in range(n_s):
                last_value = values[min(len(values), (j + 1) * d) - 1]
                e = end_s if j == n_s - 1 else last_value + 1
                blocks.append((b, e, s))
                b = e
        begin_s = end_s
    return blocks
