"""Why the INT3 format costs nine operand registers per 32 codes and not eight.

The integer form of the decode kernel feeds masked code bytes to the 8-bit MMA as
they stand: an operand register is a 32-bit window of the packed stream (a word,
possibly shifted) AND a mask that leaves ONE whole 3-bit field in each of its four
byte lanes.  INT4 needs 8 such registers per 32 codes.  If 32 three-bit codes are
stored with every field whole (contiguous), the fields tile the 96 bits at
positions 0, 3, ..., 93 whatever the order of the codes, so the question "is there
a layout that unpacks with 8 registers" is: can 8 windows, four fields each, one
per byte lane, cover those 32 positions?  The search below is exhaustive, and more
generous than the kernel (a window may start at any bit, even across words), and
finds none; the shipped format therefore splits two codes of every 32 over spare
bits and uses a ninth register for them.
"""
import sys

def _covers(max_windows, width):
    """1 if 32 whole `width`-bit fields at 0, width, 2 width, ... can be covered by `max_windows` full windows, else 0."""
    fields = [width * j for j in range(32)]
    total_bits = 32 * width
    found = 0
    windows = []                                   # (start bit, [field position or None] * 4)

    def place(i):
        nonlocal found
        if found:
            return
        if i == len(fields):
            found += 1
            return
        p = fields[i]
        # fields come in increasing position: a lane that ends before this field can never be filled,
        # and with max_windows * 4 == 32 every lane of every window has to be
        for start, lanes in windows:
            for b in range(4):
                if lanes[b] is None and start + 8 * b + 8 < p + width:
                    return
        for start, lanes in windows:
            for b in range(4):
                if lanes[b] is None and start + 8 * b <= p and p + width <= start + 8 * b + 8:
                    lanes[b] = p
                    place(i + 1)
                    lanes[b] = None
        if len(windows) < max_windows:
            # a new window takes this field in its lowest lane (its lanes fill in increasing position)
            for start in range(max(0, p + width - 8), min(p, total_bits - 32) + 1):
                windows.append((start, [p, None, None, None]))
                place(i + 1)
                windows.pop()

    old = sys.getrecursionlimit()
    sys.setrecursionlimit(10000)
    try:
        place(0)
    finally:
        sys.setrecursionlimit(old)
    return found


def test_no_eight_register_unpack_of_32_whole_three_bit_fields():
    assert _covers(8, 3) == 0


def test_the_search_finds_the_int4_cover():
    # sanity of the search itself: 4-bit fields ARE covered by 8 windows of four (two per word: the
    # fields at bits 0..3 and the fields at bits 4..7 of every byte)
    assert _covers(8, 4) == 1
