"""Host-side proof by exhaustion of the invariant behind the backward kernel's bias-gradient updates.

Each elementwise warp adds dS into its own shared-memory table with a plain load-add-store.  Lane l of warp
W = 4 t + quarter holds key slot 32 ((W + c l) mod M) + l (M = 4 x tiles in use; c = 5 for two-tile windows whose
side does not divide 32, else 1), and the updates of G consecutive query columns (aligned to G) are issued
together.  That is only correct if the 32 x G table entries of such a group are pairwise distinct, and it is only
fast if the 32 entries of one query fall into 32 different banks.  The rule for G below restates the kernel's."""
import pytest


def _interleave(w, ntiles):
    return 5 if (ntiles == 2 and 32 % w != 0) else 1


def _group(w, ew, ntiles):
    """Queries per update group for a window of side w, width ew (1 = one query at a time)."""
    M = 4 * ntiles
    if ew == w and w >= 4:
        if 32 % w == 0:
            return 8 if (M == 8 and w >= 8) else 4
        if M == 8:
            return 4
    return 1


def _cases():
    for w in range(1, 17):
        for eh in range(1, w + 1):
            for ew in {w, max(1, w // 2), 1}:
                if eh * ew <= 256:
                    yield w, eh, ew


@pytest.mark.parametrize("w", range(1, 17))
def test_grouped_updates_never_meet_and_full_width_rows_are_bank_conflict_free(w):
    cs = w + 32
    for ww, eh, ew in _cases():
        if ww != w:
            continue
        n = eh * ew
        npad = (n + 15) & ~15
        ntiles = (n + 127) // 128
        M, c, G = 4 * ntiles, _interleave(w, ntiles), _group(w, ew, ntiles)

        def code(slot):
            return (slot // ew) * cs + slot % ew

        for W in range(M):
            slots = [32 * ((W + c * lane) % M) + lane for lane in range(32)]
            assert len(set(slots)) == 32
            for q0 in range(0, npad, G):
                entries = [code(q) - code(ks) for ks in slots if ks < n for q in range(q0, min(q0 + G, npad)) if q < n]
                assert len(entries) == len(set(entries)), (w, eh, ew, W, q0)
            if ew == w:          # full width: code = slot + 32 a, so the lanes' entries at one query differ mod 32
                banks = {(-code(ks)) % 32 for ks in slots}
                assert len(banks) == 32
        # every slot of every tile is held by exactly one (warp, lane)
        held = sorted(32 * ((W + c * lane) % M) + lane for W in range(M) for lane in range(32))
        assert held == list(range(128 * ntiles))


@pytest.mark.parametrize("w", range(9, 16))
def test_sixteen_slots_per_window_row_layout_of_sides_9_to_15(w):
    """Sides 9 .. 15 with 16 slots per window row: every one of the 256 slots, with or without a token, carries the
    code 48 a + b of 16-wide geometry (stride 48 whatever the side); key order c = 1; groups of 8 queries for two-tile windows.  The 32 x 8
    entries of a group are pairwise distinct, and with the kernel's margin in front of the table every entry that any
    (key slot, query column) pair can address lies inside the warp's 1472-float block."""
    cs, c0 = 48, (w - 1) * 49
    margin = (16 - w) * 48 + 8                            # the kernel's dbias_margin(w)
    entries_of_table = 1472

    def code(slot):
        return (slot // 16) * cs + slot % 16

    for eh in range(9, w + 1):                            # two tiles: 16 eh > 128
        n = 16 * eh
        for W in range(8):
            slots = [32 * ((W + lane) % 8) + lane for lane in range(32)]
            for q0 in range(0, n, 8):
                entries = [code(q) - code(ks) for ks in slots for q in range(q0, q0 + 8)]
                assert len(entries) == len(set(entries)), (w, eh, W, q0)
                lo, hi = min(entries) + c0 + margin, max(entries) + c0 + margin
                assert 0 <= lo and hi < entries_of_table, (w, eh, lo, hi)
                for q in range(q0, q0 + 8):               # one query: the warp's 32 key rows update 32 different banks
                    assert len({(code(q) - code(ks)) % 32 for ks in slots}) == 32
    # the entries of pairs that hold tokens are those of the packed layout: (a_q - a_k + w - 1) cs + (b_q - b_k + w - 1)
    for aq, bq, ak, bk in ((0, 0, w - 1, w - 1), (w - 1, w - 1, 0, 0), (3, w - 1, 5, 0)):
        assert code(16 * aq + bq) - code(16 * ak + bk) + c0 == (aq - ak + w - 1) * cs + (bq - bk + w - 1)
