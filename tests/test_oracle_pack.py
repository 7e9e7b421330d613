"""Pins for the oracle's encoded form (Eq. 3, Eq. 4, the 3-bit placement identifier of
Section 3.1 and the ShiftCtrl / MuxCtrl metadata of Section 5.1).

None of these re-use the oracle's own packing code: Eq. 4 is evaluated here with plain
integers for every pair, the stream layout is pinned by bytes worked out by hand, and the
round trip is checked against the transform the other test files already pin."""
import math

import numpy as np
import pytest

import oracle

MASKS_N4 = [m for m in range(32) if (m & 1) and (m & 16)]     # contain shifts 0 and 4; gaps <= 4 always hold
NAMED = {"5opt": 0x1F, "3opt": 0x15, "2opt": 0x11}


def all_pairs():
    a, b = np.meshgrid(np.arange(256, dtype=np.uint8), np.arange(256, dtype=np.uint8), indexing="ij")
    return np.stack([a.ravel(), b.ravel()], axis=1).reshape(-1, 16)     # 8 pairs per row


@pytest.mark.parametrize("name", list(NAMED))
@pytest.mark.parametrize("mode", [1, 2])
@pytest.mark.parametrize("rnd", [0, 1])
def test_eq4_multiplier_reproduces_the_transformed_pair(name, mode, rnd):
    # Eq. 4: 2^opt1 * in1 * w_in1 + 2^opt2 * in2 * w_in2, with the multiplexers choosing
    # the weights, must equal T(a) * w1 + T(b) * w2 for every pair and any weights.
    mask = NAMED[name]
    shifts = {s for s in range(5) if (mask >> s) & 1}
    weights = [(1, 0), (0, 1), (-128, 127), (37, -91)]
    step = 1 if name == "5opt" else 3
    for a in range(0, 256, step):
        for b in range(256):
            in1, o1, in2, o2, mux = oracle.pair_fields(a, b, mode, mask, rnd)
            assert 0 <= in1 < 16 and 0 <= in2 < 16
            if mode == 2:
                qa, qb = oracle.vsparq_pair(a, b, 4, mask, rnd)
            else:
                qa, qb = oracle.bsparq(a, 4, mask, rnd), oracle.bsparq(b, 4, mask, rnd)
            if mux == 0:
                assert o1 in shifts and o2 in shifts
            else:
                assert mode == 2 and (o1, o2) == (4, 0)           # Eq. 3: the two nibbles of one value
                assert (mux == 1) == (b == 0)
            for w1, w2 in weights:
                wa, wb = {0: (w1, w2), 1: (w1, w1), 2: (w2, w2)}[mux]
                assert (in1 << o1) * wa + (in2 << o2) * wb == qa * w1 + qb * w2, (a, b)


def test_metadata_sizes_against_the_paper():
    # Section 3.1: five placements need a 3-bit identifier.  Section 5.1: 3opt carries a
    # 2-bit ShiftCtrl and a 1-bit MuxCtrl per 4-bit value.  Grouping a pair's metadata
    # into one state number never needs more bits than those separate fields.
    per_value = {"5opt": 3 + 1, "3opt": 2 + 1, "2opt": 1 + 1}
    for name, mask in NAMED.items():
        ns = bin(mask).count("1")
        assert math.ceil(math.log2(ns)) == per_value[name] - 1
        assert oracle.pack_states(2, mask) == ns * ns + 2
        assert oracle.pack_states(1, mask) == ns * ns
        for mode in (1, 2):
            cb = oracle.pack_ctrl_bits(mode, mask)
            assert (1 << cb) >= oracle.pack_states(mode, mask) > (1 << (cb - 1))
            assert cb <= 2 * per_value[name]
    assert [oracle.pack_ctrl_bits(2, NAMED[k]) for k in ("5opt", "3opt", "2opt")] == [5, 4, 3]
    assert [oracle.pack_ctrl_bits(1, NAMED[k]) for k in ("5opt", "3opt", "2opt")] == [5, 4, 2]


def test_stream_layout_worked_by_hand():
    # vSPARQ, 5opt, rounding.  By hand (window, shift):
    #   (27,33): 27 -> (14,1)=28; 33 -> (33+2)>>2 = 8 -> (8,2)=32      data 0xE8, state 1*5+2 = 7
    #   (0,200): lone in slot 1                                          data 0xC8, state 26
    #   (5,0), (0,0): lone / none in slot 0                              data 5, 0, state 25
    #   (255,1): 255 -> (255+8)>>4 = 16 overflows the top -> (15,4)=240  data 0xF1, state 4*5+0 = 20
    #   (16,17): 16 -> (8,1); 17 -> (17+1)>>1 = 9 -> (9,1)=18            data 0x89, state 1*5+1 = 6
    #   (100,50): (100+4)>>3 = 13 -> (13,3)=104; (50+2)>>2 = 13 -> (13,2) data 0xDD, state 3*5+2 = 17
    #   (7,9): unchanged, shift 0                                        data 0x79, state 0
    # control word = 7 + 26<<5 + 25<<10 + 25<<15 + 20<<20 + 6<<25 + 17<<30 = 18476754759
    x = np.array([[27, 33, 0, 200, 5, 0, 0, 0, 255, 1, 16, 17, 100, 50, 7, 9]], dtype=np.uint8)
    data, ctrl = oracle.pack(x, 2, 0x1F, 1)
    assert list(data) == [0xE8, 0xC8, 0x05, 0x00, 0xF1, 0x89, 0xDD, 0x79]
    assert list(ctrl) == [0x47, 0xE7, 0x4C, 0x4D, 0x04]
    back = oracle.unpack(data, ctrl, x.shape, 2, 0x1F)
    assert list(back[0]) == [28, 32, 0, 200, 5, 0, 0, 0, 240, 1, 16, 18, 104, 52, 7, 9]


@pytest.mark.parametrize("mask", MASKS_N4)
@pytest.mark.parametrize("mode", [1, 2])
@pytest.mark.parametrize("rnd", [0, 1])
def test_round_trip_equals_transform_for_every_pair(mask, mode, rnd):
    x = all_pairs()
    data, ctrl = oracle.pack(x, mode, mask, rnd)
    cb = oracle.pack_ctrl_bits(mode, mask)
    assert data.size == x.size // 2 and ctrl.size == x.size // 16 * cb
    back = oracle.unpack(data, ctrl, x.shape, mode, mask)
    assert np.array_equal(back, oracle.transform(x, mode, 4, mask, rnd))
    # every stored state is a valid one
    words = np.zeros(ctrl.size // cb, dtype=np.uint64)
    for k in range(cb):
        words |= ctrl.reshape(-1, cb)[:, k].astype(np.uint64) << np.uint64(8 * k)
    for j in range(8):
        st = (words >> np.uint64(j * cb)) & np.uint64((1 << cb) - 1)
        assert int(st.max()) < oracle.pack_states(mode, mask)


def test_lone_value_is_stored_whole():
    # a lone non-zero keeps all 8 bits (Eq. 3): its data byte is the activation itself
    x = np.zeros((256, 16), dtype=np.uint8)
    x[:, 0] = np.arange(256)
    x[:, 3] = np.arange(256)
    data, _ = oracle.pack(x, 2, 0x11, 0)
    d = data.reshape(256, 8)
    assert np.array_equal(d[:, 0], np.arange(256)) and np.array_equal(d[:, 1], np.arange(256))


def test_footprint():
    # bits per activation: 4 data bits + half the pair's control bits; below the 8 bits of the
    # raw activation and below the separate-field format of Section 5.1 (4 + ShiftCtrl + MuxCtrl)
    for name, literal in (("5opt", 8), ("3opt", 7), ("2opt", 6)):
        bits = 4 + oracle.pack_ctrl_bits(2, NAMED[name]) / 2
        assert bits < literal <= 8
    assert 4 + oracle.pack_ctrl_bits(2, 0x1F) / 2 == 6.5


def test_rejects_ragged_rows():
    with pytest.raises(ValueError):
        oracle.pack(np.zeros((2, 24), dtype=np.uint8), 2, 0x1F, 1)


# ---- any window width (Section 5.1: 3- and 2-bit windows) -----------------------------------

COMBOS_N = [(4, 0x1F), (4, 0x15), (3, 0x3F), (3, 0x35), (3, 0x29), (2, 0x7F), (2, 0x55), (2, 0x6B)]


@pytest.mark.parametrize("n,mask", COMBOS_N)
@pytest.mark.parametrize("mode", [1, 2])
@pytest.mark.parametrize("rnd", [0, 1])
def test_eq4_for_any_width_reproduces_the_transformed_pair(n, mask, mode, rnd):
    # Eq. 4 evaluated with plain integers: 2^opt1 * in1 * w_in1 + 2^opt2 * in2 * w_in2 with the
    # multiplexers choosing the weights equals T(a) * w1 + T(b) * w2; a lone value arrives as the
    # two adjacent n-bit halves of its 2n-bit window (opt1 = opt2 + n).
    shifts = {s for s in range(9 - n) if (mask >> s) & 1}
    for a in range(0, 256, 3 if n == 4 else 1):
        for b in list(range(0, 256, 5)) + [0, 1, 255]:
            in1, o1, in2, o2, mux = oracle.pair_fields_n(a, b, mode, n, mask, rnd)
            assert 0 <= in1 < (1 << n) and 0 <= in2 < (1 << n)
            if mode == 2:
                qa, qb = oracle.vsparq_pair(a, b, n, mask, rnd)
            else:
                qa, qb = oracle.bsparq(a, n, mask, rnd), oracle.bsparq(b, n, mask, rnd)
            if mux == 0:
                assert o1 in shifts and o2 in shifts
            else:
                assert mode == 2 and o1 == o2 + n and 0 <= o2 <= 8 - 2 * n
                assert (mux == 1) == (b == 0)
            for w1, w2 in [(1, 0), (0, 1), (-128, 127), (37, -91)]:
                wa, wb = {0: (w1, w2), 1: (w1, w1), 2: (w2, w2)}[mux]
                assert (in1 << o1) * wa + (in2 << o2) * wb == qa * w1 + qb * w2, (a, b)
            if n == 4:
                assert (in1, o1, in2, o2, mux) == oracle.pair_fields(a, b, mode, mask, rnd)


def test_state_counts_and_widths_for_narrow_windows():
    # two windows: ns^2 placements; a lone value: its 2n-bit window sits at one of 9 - 2n shifts, in either slot
    for n, mask in COMBOS_N:
        ns = bin(mask).count("1")
        assert oracle.pack_states_n(1, n, mask) == ns * ns
        assert oracle.pack_states_n(2, n, mask) == ns * ns + 2 * (9 - 2 * n)
        for mode in (1, 2):
            cb = oracle.pack_ctrl_bits_n(mode, n, mask)
            assert (1 << cb) >= oracle.pack_states_n(mode, n, mask) > (1 << (cb - 1))
    # Section 5.1's full sets: 6opt and 7opt need 6 control bits per pair: 6 and 5 bits per activation
    assert oracle.pack_ctrl_bits_n(2, 3, 0x3F) == 6 and oracle.pack_ctrl_bits_n(2, 2, 0x7F) == 6
    assert (2 * 3 + 6) / 2 == 6 and (2 * 2 + 6) / 2 == 5
    assert oracle.pack_ctrl_bits_n(2, 4, 0x1F) == oracle.pack_ctrl_bits(2, 0x1F)


@pytest.mark.parametrize("n,mask", COMBOS_N)
@pytest.mark.parametrize("mode", [1, 2])
@pytest.mark.parametrize("rnd", [0, 1])
def test_round_trip_for_any_width_equals_the_transform(n, mask, mode, rnd):
    x = all_pairs()
    data, ctrl = oracle.pack_n(x, mode, n, mask, rnd)
    assert data.size == x.size // 16 * 2 * n
    back = oracle.unpack_n(data, ctrl, x.shape, mode, n, mask)
    assert np.array_equal(back, oracle.transform(x, mode, n, mask, rnd))
    if n == 4:      # the same stream as the byte-per-pair form
        d4, c4 = oracle.pack(x, mode, mask, rnd)
        assert np.array_equal(data, d4) and np.array_equal(ctrl, c4)


def test_stream_bytes_worked_out_by_hand_for_three_bit_windows():
    # vSPARQ, n = 3, all six placements, rounding.  One unit of 16 activations = 8 pairs:
    #   (0, 0)     lone, first slot, w = 0 at s_l = 0          field 0b000000  state 36 + 0
    #   (200, 0)   lone: 200 = 0b11001000 -> 6-bit window 0b110010 at s_l = 2 (exact)
    #                                                           field 0b110010  state 36 + 2
    #   (0, 77)    lone, second slot: 77 = 0b1001101 -> shift 1: (77 + 1) >> 1 = 39 = 0b100111
    #                                                           field 0b100111  state 36 + 3 + 1
    #   (5, 3)     windows 5 (shift 0), 3 (shift 0)            field 0b101011  state 0
    #   (27, 100)  27 = 0b11011 -> shift 2: (27 + 2) >> 2 = 7 ; 100 = 0b1100100 -> shift 4: (100 + 8) >> 4 = 6
    #                                                           field 0b111110  state 2 * 6 + 4
    #   (255, 255) saturate: 7 at shift 5 both                  field 0b111111  state 5 * 6 + 5
    #   (31, 63)   31 -> shift 2: (31 + 2) >> 2 = 8 carries to 32 = 4 << 3 ; 63 -> shift 3: (63 + 4) >> 3 = 8 -> 64 = 4 << 4
    #                                                           field 0b100100  state 3 * 6 + 4
    #   (1, 1)     field 0b001001  state 0
    x = np.array([[0, 0, 200, 0, 0, 77, 5, 3, 27, 100, 255, 255, 31, 63, 1, 1]], dtype=np.uint8)
    fields = [0b000000, 0b110010, 0b100111, 0b101011, 0b111110, 0b111111, 0b100100, 0b001001]
    states = [36, 38, 40, 0, 16, 35, 22, 0]
    dword = sum(f << (6 * j) for j, f in enumerate(fields))
    cword = sum(s << (6 * j) for j, s in enumerate(states))
    data, ctrl = oracle.pack_n(x, 2, 3, 0x3F, 1)
    assert list(data) == [(dword >> (8 * k)) & 0xFF for k in range(6)]
    assert list(ctrl) == [(cword >> (8 * k)) & 0xFF for k in range(6)]
    want = [0, 0, 200, 0, 0, 78, 5, 3, 28, 96, 224, 224, 32, 64, 1, 1]
    assert list(oracle.unpack_n(data, ctrl, x.shape, 2, 3, 0x3F)[0]) == want
    assert list(oracle.transform(x, 2, 3, 0x3F, 1)[0]) == want
