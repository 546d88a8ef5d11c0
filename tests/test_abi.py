"""CPU-side checks of the C ABI: the library loads, exports what the header declares, and
rejects bad arguments on the host before touching the device."""
import ctypes
import os
import re

import pytest

import oracle
from paper_2412_19829_b200 import binding as gf

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    names = set()
    inc = os.path.join(ROOT, "include")
    for fn in os.listdir(inc):
        if fn.endswith(".h"):
            text = open(os.path.join(inc, fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(gformer_\w+)\s*\(", text))
    return sorted(names)


def test_header_declares_the_four_entry_points():
    names = declared_symbols()
    for must in ("gformer_window_attn", "gformer_causal_linear_attn", "gformer_hybrid_attn",
                 "gformer_decode_step", "gformer_workspace_bytes"):
        assert must in names


def test_library_exports_every_declared_symbol():
    L = gf.lib()
    for name in declared_symbols():
        assert hasattr(L, name), name


def test_status_strings_and_version():
    assert gf.version() >= 100
    assert gf.status_string(gf.GF_OK) == "ok"
    assert len({gf.status_string(i) for i in range(6)}) == 6


def test_default_head_split_matches_oracle_reading():
    for H in (1, 2, 3, 8, 12, 16, 24, 32, 40, 64, 96):
        assert gf.default_h_sparse(H) == oracle.default_h_sparse(H)


def test_workspace_bytes_nonzero():
    assert gf.workspace_bytes(1, 32, 32768, 128, 512, 6, gf.GF_BF16) >= 256


def test_tuning_rejects_unknown_keys():
    L = gf.lib()
    assert L.gformer_set_tuning(99, 1) == gf.GF_ERR_INVALID_ARG
    assert L.gformer_set_tuning(gf.GF_TUNE_LINEAR_SPLIT, -2) == gf.GF_ERR_INVALID_ARG
    assert L.gformer_set_tuning(gf.GF_TUNE_LINEAR_SPLIT, 5000) == gf.GF_ERR_INVALID_ARG
    assert L.gformer_set_tuning(gf.GF_TUNE_LINEAR_SPLIT, -1) == gf.GF_OK  # never cut a chain
    assert gf.linear_plan(26, 32768, 128) == (1, 256)
    assert L.gformer_set_tuning(gf.GF_TUNE_LINEAR_SPLIT, 0) == gf.GF_OK
    assert L.gformer_set_tuning(gf.GF_TUNE_LINEAR_CTAS, -1) == gf.GF_ERR_INVALID_ARG
    assert L.gformer_set_tuning(gf.GF_TUNE_LINEAR_CTAS, 70000) == gf.GF_ERR_INVALID_ARG
    assert L.gformer_set_tuning(gf.GF_TUNE_LINEAR_CTAS, 0) == gf.GF_OK


def test_workspace_covers_every_plan():
    # the scratch is sized for the largest segment count the plan may choose, whatever CTA count
    # the launch ends up with: it never shrinks when the chunks-per-segment knob is left on auto
    auto = gf.workspace_bytes(1, 32, 32768, 128, 512, 6, gf.GF_BF16)
    gf.set_tuning(gf.GF_TUNE_LINEAR_SPLIT, 8)
    try:
        fixed = gf.workspace_bytes(1, 32, 32768, 128, 512, 6, gf.GF_BF16)
    finally:
        gf.set_tuning(gf.GF_TUNE_LINEAR_SPLIT, 0)
    assert auto >= fixed


def _state_scratch(chains, segments, d):
    # per segment: one 128-byte flag line and one published state (S: 128 x d floats, z: d floats)
    return 256 + chains * segments * (128 + (128 * d + d) * 4)


def test_linear_plan_covers_the_chain_and_fits_the_workspace():
    for chains in (1, 2, 13, 26, 104, 148, 200, 832):
        for N in (1, 100, 128, 129, 1000, 4096, 32768, 65536, 262144):
            for d in (64, 128):
                ws = gf.workspace_bytes(1, chains, N, d, 1, 0, gf.GF_BF16)
                for ctas in (0, 1, 37, 148):
                    G, L = gf.linear_plan(chains, N, d, ctas)
                    nch = -(-N // 128)
                    assert 1 <= G <= nch
                    assert L == -(-nch // G)  # balanced segments: the longest has ceil(nch / G) chunks
                    whole, G2, L2 = gf.linear_plan_parts(chains, N, d, ctas)
                    assert (G2, L2) == (G, L) and 0 <= whole <= chains
                    if G > 1:
                        assert 3 < nch / G <= 32
                        # the first `whole` chains are not cut and need no scratch
                        assert whole % (ctas or 148) == 0
                        assert ws >= _state_scratch(chains - whole, G, d), (chains, N, d, ctas, G)
                    else:
                        assert whole in (0, chains)


def test_linear_plan_named_cases():
    # the long-sequence workload: segments of at most 8 chunks (what 148 CTAs can park in L2 at d = 128)
    G, L = gf.linear_plan(26, 32768, 128)
    assert 32 <= G <= 40 and L <= 8
    # one long chain is a serial pipeline of hand-over links: few, long segments
    G, L = gf.linear_plan(1, 32768, 128)
    assert 12 <= L <= 32
    G, L = gf.linear_plan(1, 262144, 128)  # ... also when its parked tiles no longer fit L2
    assert L >= 24
    G, L = gf.linear_plan(4, 131072, 128)
    assert L >= 20
    # enough whole chains for every CTA at d = 128, or chains too short to cut: the one-pass form
    assert gf.linear_plan(832, 4096, 128)[0] == 1
    assert gf.linear_plan(148, 8192, 128)[0] == 1
    assert gf.linear_plan(10, 512, 64)[0] == 1
    assert gf.linear_plan(832, 4096, 64)[0] == 1
    # chains that nearly fill one round of CTAs, or spill thinly into a second one: whole, also when long
    # (measured on a B200: 100 chains of 32K tokens at d = 128 take 706 us whole and 841 us cut)
    for chains in (100, 120, 230, 296):
        assert gf.linear_plan_parts(chains, 32768, 128) == (chains, 1, 256), chains
    assert gf.linear_plan(120, 32768, 64)[0] == 1 and gf.linear_plan(296, 32768, 64)[0] == 1
    # somewhat more chains than CTAs, long: the full rounds whole, the leftover chains cut in a launch of their own
    # (measured: 150 chains of 32K tokens at d = 128 take 946 us this way, 1271 us all cut, 1453 us all whole)
    for chains, d in ((150, 128), (156, 128), (208, 128), (300, 128), (150, 64), (230, 64), (832, 64)):
        whole, G, L = gf.linear_plan_parts(chains, 32768, d)
        assert whole == chains // 148 * 148 and G > 1 and 4 <= L <= 32, (chains, d)
        assert gf.linear_plan(chains, 32768, d) == (G, L)
        w37 = gf.linear_plan_parts(chains, 32768, d, 37)[0]
        assert w37 % 37 == 0 or w37 == chains
    # ... but not when the second launch would cost what it saves (the 4K prefill: 832 short chains)
    assert gf.linear_plan_parts(832, 4096, 64) == (832, 1, 32)
    assert gf.linear_plan_parts(26, 32768, 128)[0] == 0
    # ... while half a round of long chains is cut
    assert gf.linear_plan(74, 32768, 128)[0] > 1 and gf.linear_plan(90, 32768, 64)[0] > 1
    # fewer chains than CTAs, long: cut, in segments of about what stays in L2 at d = 64 (16 chunks of 16 KB tiles)
    G, L = gf.linear_plan(104, 16384, 64)
    assert G > 1 and L <= 20
    gf.set_tuning(gf.GF_TUNE_LINEAR_SPLIT, 8)
    try:
        assert gf.linear_plan(26, 32768, 128) == (32, 8)
        assert gf.linear_plan(3, 1000, 64) == (1, 8)
    finally:
        gf.set_tuning(gf.GF_TUNE_LINEAR_SPLIT, 0)


def test_linear_plan_argument_errors():
    L = gf.lib()
    g, l = ctypes.c_int(-7), ctypes.c_int(-7)
    assert L.gformer_linear_plan(0, 128, 64, 0, ctypes.byref(g), ctypes.byref(l)) == gf.GF_ERR_INVALID_ARG
    assert L.gformer_linear_plan(1, 0, 64, 0, ctypes.byref(g), ctypes.byref(l)) == gf.GF_ERR_INVALID_ARG
    assert L.gformer_linear_plan(1, 128, 64, -1, ctypes.byref(g), ctypes.byref(l)) == gf.GF_ERR_INVALID_ARG
    assert L.gformer_linear_plan(1, 128, 96, 0, ctypes.byref(g), ctypes.byref(l)) == gf.GF_ERR_UNSUPPORTED
    assert L.gformer_linear_plan(1, 128, 64, 0, None, ctypes.byref(l)) == gf.GF_ERR_INVALID_ARG
    assert (g.value, l.value) == (-7, -7)
    wh = ctypes.c_int(-7)
    assert L.gformer_linear_plan_parts(0, 128, 64, 0, ctypes.byref(wh), ctypes.byref(g), ctypes.byref(l)) == gf.GF_ERR_INVALID_ARG
    assert L.gformer_linear_plan_parts(1, 128, 96, 0, ctypes.byref(wh), ctypes.byref(g), ctypes.byref(l)) == gf.GF_ERR_UNSUPPORTED
    assert L.gformer_linear_plan_parts(1, 128, 64, 0, None, ctypes.byref(g), ctypes.byref(l)) == gf.GF_ERR_INVALID_ARG
    assert (wh.value, g.value, l.value) == (-7, -7, -7)
    assert L.gformer_linear_plan_parts(1, 128, 64, 0, ctypes.byref(wh), ctypes.byref(g), ctypes.byref(l)) == gf.GF_OK
    assert (wh.value, g.value, l.value) == (1, 1, 1)


def test_partition_balance_against_the_oracle():
    """Algorithm 2: the library's closed form against the oracle's bisection."""
    import numpy as np
    from oracle import partition as op

    assert gf.partition_balance(2.0, 1.0, 1.0, 1.0) == pytest.approx(1.0 / 3.0, abs=1e-15)
    rng = np.random.default_rng(21)
    for _ in range(200):
        f0, f1, p0, p1 = (float(x) for x in 10.0 ** rng.uniform(-2, 2, 4))
        size = float(rng.integers(1, 10**6))
        assert gf.partition_balance(f0, f1, p0, p1) == pytest.approx(op.balance(size, f0, f1, p0, p1), abs=1e-12)
    # measured seconds per head as the work, unit rates: 16 heads, a windowed head 3x as slow
    p = gf.partition_balance(3.0e-6, 1.0e-6, 1.0, 1.0)
    assert p == pytest.approx(op.balance(16, 3.0e-6, 1.0e-6, 1.0, 1.0), abs=1e-12) and round(p * 16) == 4


def test_partition_heads_against_the_oracle():
    """FLOP model of Sec. III-D: the library's root-and-neighbours search against the oracle's
    exhaustive one, both deciding in fp64."""
    import numpy as np
    from oracle import partition as op

    assert gf.partition_heads(1, 4, 1, 1, 1, 1.0, 1.0) == (3, 15.0, 8.0)
    rng = np.random.default_rng(22)
    cases = [(1, 32, 32768, 128, 512, 1.0e12, 1.0e15), (8, 12, 4096, 64, 256, 3.0e12, 1.0e14), (1, 1, 1, 1, 1, 1.0, 1.0),
             (64, 4096, 262144, 128, 4096, 1.0e9, 1.0e9), (1, 16, 2048, 64, 1, 1.0e15, 1.0), (1, 16, 2048, 64, 2048, 1.0, 1.0e15)]
    for _ in range(300):
        cases.append((int(rng.integers(1, 9)), int(rng.integers(1, 130)), int(rng.integers(1, 70000)),
                      int(rng.choice([1, 32, 64, 128])), int(rng.integers(1, 5000)),
                      float(10.0 ** rng.uniform(6, 16)), float(10.0 ** rng.uniform(6, 16))))
    for B, H, N, E, W, ps, pl in cases:
        h0, ls, ll = gf.partition_heads(B, H, N, E, W, ps, pl)
        want = op.partition_heads(B, H, N, E, W, ps, pl)
        s, l = op.model_latencies(B, H, N, E, W, h0, ps, pl)
        assert ls == pytest.approx(s, rel=1e-14) and ll == pytest.approx(l, rel=1e-14)
        if h0 != want:  # only where the two gaps agree to rounding may the counts differ
            sw, lw = op.model_latencies(B, H, N, E, W, want, ps, pl)
            assert abs(s - l) == pytest.approx(abs(sw - lw), rel=1e-12), (B, H, N, E, W, ps, pl, h0, want)


def test_partition_argument_errors():
    L = gf.lib()
    p = ctypes.c_double(-7.0)
    for bad in ((0.0, 1.0, 1.0, 1.0), (1.0, -1.0, 1.0, 1.0), (1.0, 1.0, float("inf"), 1.0), (1.0, 1.0, 1.0, float("nan"))):
        assert L.gformer_partition_balance(*bad, ctypes.byref(p)) == gf.GF_ERR_INVALID_ARG
    assert L.gformer_partition_balance(1.0, 1.0, 1.0, 1.0, None) == gf.GF_ERR_INVALID_ARG
    assert p.value == -7.0
    h0 = ctypes.c_int(-7)
    for bad in ((0, 4, 1, 1, 1, 1.0, 1.0), (1, 0, 1, 1, 1, 1.0, 1.0), (1, 4, 0, 1, 1, 1.0, 1.0), (1, 4, 1, 0, 1, 1.0, 1.0),
                (1, 4, 1, 1, 0, 1.0, 1.0), (1, 4, 1, 1, 1, 0.0, 1.0), (1, 4, 1, 1, 1, 1.0, float("nan"))):
        assert L.gformer_partition_heads(*bad, ctypes.byref(h0), None, None) == gf.GF_ERR_INVALID_ARG
    assert L.gformer_partition_heads(1, 4, 1, 1, 1, 1.0, 1.0, None, None, None) == gf.GF_ERR_INVALID_ARG
    assert h0.value == -7
    assert L.gformer_partition_heads(1, 4, 1, 1, 1, 1.0, 1.0, ctypes.byref(h0), None, None) == gf.GF_OK and h0.value == 3


FAKE = 0x10000  # a 16-byte-aligned non-null address; validation fails before it is ever used


@pytest.mark.parametrize("kw,expect", [
    (dict(q=0), gf.GF_ERR_INVALID_ARG),
    (dict(q=FAKE + 4), gf.GF_ERR_INVALID_ARG),
    (dict(B=0), gf.GF_ERR_INVALID_ARG),
    (dict(N=0), gf.GF_ERR_INVALID_ARG),
    (dict(w=0), gf.GF_ERR_INVALID_ARG),
    (dict(d=96), gf.GF_ERR_UNSUPPORTED),
    (dict(dtype=7), gf.GF_ERR_INVALID_ARG),
    (dict(layout=5), gf.GF_ERR_INVALID_ARG),
    (dict(o=FAKE), gf.GF_ERR_INVALID_ARG),          # o aliases q
    (dict(ws=0), gf.GF_ERR_WORKSPACE),
    (dict(ws_bytes=8), gf.GF_ERR_WORKSPACE),
])
def test_window_attn_argument_errors(kw, expect):
    a = dict(q=FAKE, k=FAKE + (1 << 30), v=FAKE + (2 << 30), o=FAKE + (3 << 30), B=1, H=2, N=64, d=64, w=32,
             scale=0.0, dtype=gf.GF_BF16, layout=gf.GF_BHND, ws=FAKE + (4 << 30), ws_bytes=4096)
    a.update(kw)
    rc = gf.lib().gformer_window_attn(a["q"], a["k"], a["v"], a["o"], a["B"], a["H"], a["N"], a["d"], a["w"],
                                      a["scale"], a["dtype"], a["layout"], a["ws"], a["ws_bytes"], None)
    assert rc == expect


def test_hybrid_and_linear_argument_errors():
    L = gf.lib()
    q, k, v, o, ws = FAKE, FAKE + (1 << 30), FAKE + (2 << 30), FAKE + (3 << 30), FAKE + (4 << 30)
    # h_sparse > H
    assert L.gformer_hybrid_attn(q, k, v, o, 1, 4, 64, 64, 32, 5, 0.0, 0, 0, gf.GF_BF16, 0, None, ws, 4096,
                                 None) == gf.GF_ERR_INVALID_ARG
    # unknown feature map
    assert L.gformer_hybrid_attn(q, k, v, o, 1, 4, 64, 64, 32, 1, 0.0, 3, 0, gf.GF_BF16, 0, None, ws, 4096,
                                 None) == gf.GF_ERR_UNSUPPORTED
    # chunk not a multiple of 64
    assert L.gformer_causal_linear_attn(q, k, v, o, 1, 4, 64, 64, 0, 100, None, None, gf.GF_BF16, 0, ws, 4096,
                                        None) == gf.GF_ERR_INVALID_ARG
    # S without z
    assert L.gformer_causal_linear_attn(q, k, v, o, 1, 4, 64, 64, 0, 0, FAKE + (5 << 30), None, gf.GF_BF16, 0,
                                        ws, 4096, None) == gf.GF_ERR_INVALID_ARG
    # state struct that disagrees with the call
    st = gf.DecodeStateC(FAKE, FAKE, FAKE, FAKE, 0, 2, 4, 64, 32, 1, gf.GF_BF16)
    assert L.gformer_hybrid_attn(q, k, v, o, 1, 4, 64, 64, 32, 1, 0.0, 0, 0, gf.GF_BF16, 0, ctypes.byref(st),
                                 ws, 4096, None) == gf.GF_ERR_INVALID_ARG


def test_decode_argument_errors():
    L = gf.lib()
    q, k, v, o = FAKE, FAKE + (1 << 30), FAKE + (2 << 30), FAKE + (3 << 30)
    st = gf.DecodeStateC(FAKE, FAKE, FAKE, FAKE, 0, 2, 4, 96, 32, 1, gf.GF_BF16)
    assert L.gformer_decode_step(q, k, v, o, ctypes.byref(st), 0.0, 0, None) == gf.GF_ERR_UNSUPPORTED
    st = gf.DecodeStateC(0, FAKE, FAKE, FAKE, 0, 2, 4, 64, 32, 1, gf.GF_BF16)
    assert L.gformer_decode_step(q, k, v, o, ctypes.byref(st), 0.0, 0, None) == gf.GF_ERR_INVALID_ARG
    assert L.gformer_decode_step(q, k, v, o, None, 0.0, 0, None) == gf.GF_ERR_INVALID_ARG
    assert st.t == 0


def test_ragged_decode_argument_errors():
    L = gf.lib()
    st = gf.DecodeStateC(FAKE, FAKE + (1 << 20), FAKE + (2 << 20), FAKE + (3 << 20), 0, 2, 4, 64, 16, 1, gf.GF_BF16)
    a = (FAKE + (4 << 20), FAKE + (5 << 20), FAKE + (6 << 20), FAKE + (7 << 20))
    assert L.gformer_decode_step_ragged(*a, ctypes.byref(st), None, 0.0, gf.GF_PHI_ELU1, None) == gf.GF_ERR_INVALID_ARG
    assert L.gformer_decode_step_ragged(*a, ctypes.byref(st), FAKE + (8 << 20) + 4, 0.0, gf.GF_PHI_ELU1, None) == \
        gf.GF_ERR_INVALID_ARG
    assert L.gformer_decode_step_ragged(a[0], a[1], a[2], 0, ctypes.byref(st), FAKE + (8 << 20), 0.0, gf.GF_PHI_ELU1,
                                        None) == gf.GF_ERR_INVALID_ARG
    # the feature map and its parameter go together, here as everywhere
    assert L.gformer_decode_step_ragged(*a, ctypes.byref(st), FAKE + (8 << 20), 0.0, gf.GF_PHI_FAVOR_POS, None) == \
        gf.GF_ERR_INVALID_ARG
    assert L.gformer_decode_step_ragged_w(*a, ctypes.byref(st), FAKE + (8 << 20), 0.0, gf.GF_PHI_FAVOR_POS, None,
                                          None) == gf.GF_ERR_INVALID_ARG
    assert L.gformer_decode_step_ragged_w(*a, ctypes.byref(st), FAKE + (8 << 20), 0.0, gf.GF_PHI_ELU1, FAKE + (9 << 20),
                                          None) == gf.GF_ERR_INVALID_ARG
    assert L.gformer_decode_step_ragged_w(*a, ctypes.byref(st), None, 0.0, gf.GF_PHI_FAVOR_POS, FAKE + (9 << 20),
                                          None) == gf.GF_ERR_INVALID_ARG
    assert st.t == 0


def test_self_layer_argument_errors():
    L = gf.lib()
    a = dict(q=FAKE, k=FAKE + (1 << 30), v=FAKE + (2 << 30), o=FAKE + (3 << 30), B=1, H=4, N=256, d=64, w=32,
             h_sparse=1, scale=0.0, phi=gf.GF_PHI_ELU1, dtype=gf.GF_BF16, layout=gf.GF_BHND, ws=FAKE + (4 << 30),
             ws_bytes=1 << 30)
    order = ("q", "k", "v", "o", "B", "H", "N", "d", "w", "h_sparse", "scale", "phi", "dtype", "layout", "ws", "ws_bytes")

    def call(**kw):
        b = dict(a, **kw)
        return L.gformer_hybrid_attn_self(*[b[n] for n in order], None)

    assert call(q=0) == gf.GF_ERR_INVALID_ARG
    assert call(w=0) == gf.GF_ERR_INVALID_ARG
    assert call(h_sparse=5) == gf.GF_ERR_INVALID_ARG
    assert call(d=96) == gf.GF_ERR_UNSUPPORTED
    assert call(phi=1) == gf.GF_ERR_INVALID_ARG  # positive random features need their projections: the _w entry point
    assert call(phi=7) == gf.GF_ERR_UNSUPPORTED
    assert call(ws_bytes=8) == gf.GF_ERR_WORKSPACE
    assert call(ws=0) == gf.GF_ERR_WORKSPACE
    # the bidirectional layer's segment sums fit the workspace the size query reports
    for chains, N, d in ((1, 128, 64), (26, 32768, 128), (832, 4096, 64), (3, 100000, 128)):
        ws = gf.workspace_bytes(1, chains, N, d, 1, 0, gf.GF_BF16)
        assert ws >= 256 + chains * 2 * (d * d + d) * 4  # at least one segment slot per chain plus the totals


def test_partition_from_times_against_the_oracle():
    # seconds per head of either kind in, Algorithm 2's share and the section's rates out
    from oracle import partition as op

    B, H, N, E, W = 2, 16, 4096, 64, 128
    tw, tl = 3.0e-6, 1.0e-6
    p, h0, ps, pl = gf.partition_from_times(B, H, N, E, W, tw, tl)
    assert p == pytest.approx(op.balance(1.0, tw, tl, 1.0, 1.0), abs=1e-12)
    assert h0 == 4  # p' = 1/4 of 16 heads
    # the rates are the model's work for what was timed over the measured times: with them the model
    # gives back the measurements (one windowed head alone; all H heads linear)
    s1, _ = op.model_latencies(B, H, N, E, W, 1, ps, pl)
    _, lall = op.model_latencies(B, H, N, E, W, 0, ps, pl)
    assert s1 == pytest.approx(tw, rel=1e-12) and lall == pytest.approx(H * tl, rel=1e-12)
    for bad in ((0, H, N, E, W, tw, tl), (B, H, N, E, W, 0.0, tl), (B, H, N, E, W, tw, float("inf"))):
        with pytest.raises(gf.GformerError):
            gf.partition_from_times(*bad)


def test_feature_map_argument_errors():
    # the positive random features (Sec. III-A / III-C) come with a projection pointer; elu + 1 must not have one
    L = gf.lib()
    q, k, v, o, ws, W = FAKE, FAKE + (1 << 30), FAKE + (2 << 30), FAKE + (3 << 30), FAKE + (4 << 30), FAKE + (5 << 30)
    big = 1 << 30
    lin = lambda phi, Wp: L.gformer_causal_linear_attn_w(q, k, v, o, 1, 4, 64, 64, phi, Wp, 0, None, None, gf.GF_BF16, 0,
                                                         ws, big, None)
    assert lin(gf.GF_PHI_FAVOR_POS, None) == gf.GF_ERR_INVALID_ARG
    assert lin(gf.GF_PHI_ELU1, W) == gf.GF_ERR_INVALID_ARG
    assert lin(gf.GF_PHI_FAVOR_POS, W + 4) == gf.GF_ERR_INVALID_ARG  # misaligned
    assert lin(5, W) == gf.GF_ERR_UNSUPPORTED
    hyb = lambda phi, Wp: L.gformer_hybrid_attn_w(q, k, v, o, 1, 4, 64, 64, 32, 1, 0.0, phi, Wp, 0, gf.GF_BF16, 0, None,
                                                  ws, big, None)
    assert hyb(gf.GF_PHI_FAVOR_POS, None) == gf.GF_ERR_INVALID_ARG
    assert hyb(gf.GF_PHI_ELU1, W) == gf.GF_ERR_INVALID_ARG
    st = gf.DecodeStateC(FAKE, FAKE, FAKE, FAKE, 0, 2, 4, 64, 32, 1, gf.GF_BF16)
    assert L.gformer_decode_step_w(q, k, v, o, ctypes.byref(st), 0.0, gf.GF_PHI_FAVOR_POS, None, None) == gf.GF_ERR_INVALID_ARG
    assert L.gformer_decode_step(q, k, v, o, ctypes.byref(st), 0.0, gf.GF_PHI_FAVOR_POS, None) == gf.GF_ERR_INVALID_ARG
    assert st.t == 0
    # the features of Q and K live in the workspace on the tensor-core path: two bf16 tensors of the linear heads
    B, H, N, d, h0 = 2, 8, 4096, 128, 2
    plain = gf.workspace_bytes(B, H, N, d, 1, h0, gf.GF_BF16)
    favor = gf.workspace_bytes(B, H, N, d, 1, h0, gf.GF_BF16, gf.GF_PHI_FAVOR_POS)
    assert favor >= plain + 2 * B * (H - h0) * N * d * 2
    assert hyb(gf.GF_PHI_FAVOR_POS, W) in (gf.GF_OK, gf.GF_ERR_CUDA)  # arguments are fine (no device here: the launch fails)
