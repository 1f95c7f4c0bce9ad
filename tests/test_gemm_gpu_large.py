"""Parity at the full sizes of the three large workloads, in the launch configuration the
benchmark times: sampled rows and whole tiles computed one by one by the oracle, plus a
whole-matrix randomised identity that holds at any size.

Sampling: for every tile row, 4 complete rows of C (they cross every tile and every
column) at in-tile offsets that land in each 32-lane quarter of the accumulator and in
both CTAs of a pair and walk through all residues mod 8 as the tile row varies; the first
and last row of the matrix; and 12 complete tiles (corners, both sides of the half-way
boundary, seeded random).
"""

import os

import numpy as np
import pytest

import paper_2508_20258_b200 as sp
from oracle import gemm as G
from paper_2508_20258_b200 import synth

pytestmark = pytest.mark.gpu
TOL = 1e-2
torch = pytest.importorskip("torch")


def dev_bf16(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def sample_rows(M, tile_m):
    Tm = -(-M // tile_m)
    rows = {0, M - 1}
    for tm in range(Tm):
        for j in range(4):
            r = tm * tile_m + (37 * tm + (tile_m // 4) * j + 11) % tile_m
            if r < M:
                rows.add(r)
    return sorted(rows)


def sample_tiles(Tm, Tn, seed):
    rng = np.random.default_rng(seed)
    tiles = {(0, 0), (0, Tn - 1), (Tm - 1, 0), (Tm - 1, Tn - 1),
             ((Tm + 1) // 2 - 1, Tn // 3), ((Tm + 1) // 2, Tn // 3)}
    while len(tiles) < min(12, Tm * Tn):
        tiles.add((int(rng.integers(Tm)), int(rng.integers(Tn))))
    return sorted(tiles)


# What the benchmark times by default on the 256x512 tile (8192^3 and the large-L2-pressure workload): the die-pinned
# split with serpentine bands of eight tile rows, K walked in alternating directions (the rounding of C then depends on
# the order: such runs are held to the oracle, not to bit-identity with the other orders), C stores marked evict_first;
# and the unpinned order it falls back to where no two-way L2 structure is measured.
BENCH_FLAGS = sp.FLAG_SERPENTINE | sp.FLAG_K_ALTERNATE | sp.FLAG_HINT_C_EVICT_FIRST
BENCH_DEFAULT = (sp.DIE_SPLIT, dict(split_axis=0, inner_scheme=sp.GROUP_M, inner_group=8, flags=BENCH_FLAGS | sp.FLAG_DIE_PINNED))
BENCH_FALLBACK = (sp.GROUP_M, dict(group=16, flags=BENCH_FLAGS))

CASES = [
    ("cfg3", (256, 512), [(sp.GROUP_N, dict(group=8)), (sp.ROW_MAJOR, {}),
                          (sp.DIE_SPLIT, dict(split_axis=1, inner_scheme=sp.GROUP_N, inner_group=4, flags=2)),
                          BENCH_DEFAULT, BENCH_FALLBACK]),
    ("cfg5", (256, 512), [(sp.GROUP_M, dict(group=16)), BENCH_DEFAULT, BENCH_FALLBACK]),
    # the die-pinned split (flags=2) is the order the benchmark times on the 256x256 tile and on cfg5
    ("cfg3", None, [(sp.ROW_MAJOR, {}), (sp.GROUP_M, dict(group=8)), (sp.HILBERT, {}),
              (sp.DIE_SPLIT, dict(split_axis=0, inner_scheme=sp.GROUP_M, inner_group=8)),
              (sp.DIE_SPLIT, dict(split_axis=0, inner_scheme=sp.GROUP_M, inner_group=8, flags=2))]),
    ("cfg4", None, [(sp.ROW_MAJOR, {}), (sp.ROW_MAJOR, dict(flags=BENCH_FLAGS)), (sp.GROUP_M, dict(group=4)), (sp.GROUP_N, dict(group=2))]),
    ("cfg5", None, [(sp.GROUP_M, dict(group=16)), (sp.HILBERT, {}),
              (sp.DIE_SPLIT, dict(split_axis=0, inner_scheme=sp.GROUP_M, inner_group=8, flags=2))]),
]


@pytest.mark.parametrize("name,tile,schemes", CASES)
def test_large_workload_sampled(name, tile, schemes):
    w, A, B = synth.make_workload(name)
    if tile is not None:
        import dataclasses
        w = dataclasses.replace(w, tile_m=tile[0], tile_n=tile[1])
    dA, dB = dev_bf16(A), dev_bf16(B)
    dC = torch.empty((w.M, w.N), dtype=torch.bfloat16, device="cuda")
    rows = sample_rows(w.M, w.tile_m)
    ref_rows, S_rows = G.gemm_rows(A, B, rows)
    Tm, Tn = -(-w.M // w.tile_m), -(-w.N // w.tile_n)
    tiles = sample_tiles(Tm, Tn, w.seed)
    tile_refs = [G.gemm_block(A, B, tm * w.tile_m, min((tm + 1) * w.tile_m, w.M), tn * w.tile_n,
                              min((tn + 1) * w.tile_n, w.N)) for (tm, tn) in tiles]
    # randomised identity: C x = A (B x) for x in {+-1}^N, in fp64
    Af = synth.bf16_bits_to_f32(A).astype(np.float64)
    Bf = synth.bf16_bits_to_f32(B).astype(np.float64)
    xs = [np.random.default_rng(100 + i).choice([-1.0, 1.0], size=w.N) for i in range(2)]
    want_cx = [Af @ (Bf @ x) for x in xs]
    del Af, Bf
    first_bits = None
    for scheme, kw in schemes:
        dC.fill_(float("nan"))
        p = sp.make_params(tile_m=w.tile_m, tile_n=w.tile_n, out_dtype=0, **kw)
        try:
            sp.gemm(dA, dB, dC, scheme, p)
        except sp.SpError as err:
            if (kw.get("flags", 0) & sp.FLAG_DIE_PINNED) and err.status == sp.ERR_UNSUPPORTED:
                continue                      # no two-way L2 structure measured on this device
            raise
        assert sp.get_status() == 0
        bits = dC.view(torch.int16).cpu().numpy().view(np.uint16)
        got_rows = G.bf16_bits_to_f64(bits[rows, :])
        r = G.compare(got_rows, ref_rows, S_rows, K=w.K)
        assert r["max_err"] <= TOL, (name, scheme, kw, r)
        assert r["strict_violations"] == 0, (name, scheme, kw, r)     # diagnostic tier: RNE to bf16 plus fp32 accumulation
        assert r["fro_rel"] <= 3e-3, r
        for (tm, tn), (ref, S) in zip(tiles, tile_refs):
            blk = bits[tm * w.tile_m:(tm + 1) * w.tile_m, tn * w.tile_n:(tn + 1) * w.tile_n]
            rt = G.compare(G.bf16_bits_to_f64(blk), ref, S)
            assert rt["max_err"] <= TOL, (name, scheme, kw, tm, tn, rt)
        order_dependent = bool(kw.get("flags", 0) & sp.FLAG_K_ALTERNATE)
        if first_bits is None or order_dependent:
            if not order_dependent:
                first_bits = bits
            Cf = G.bf16_bits_to_f64(bits)
            norms = np.sqrt((Cf ** 2).sum(axis=1))
            for x, want in zip(xs, want_cx):
                # bf16 keeps 8 significand bits: round-to-nearest errs by at most half an ulp, |e_ij| <= 2^-8 |C_ij|
                # (uniform within that), signs independent of x -> sigma_i <= 2^-8/sqrt(3) * ||C_i||; gate 6 sigma.
                # A dropped 256-wide tile segment moves a row sum by ~16 * sigma_C, about 13x this gate.
                assert (np.abs(Cf @ x - want) <= 6 * 2.0 ** -8 / np.sqrt(3) * norms + 1e-9).all()
            assert not np.isnan(Cf).any()
            del Cf
        else:
            assert np.array_equal(bits, first_bits)      # same bits under every order


def test_output_larger_than_4_gib_is_addressed_correctly():
    """C of 49152 x 49152 bf16 is 4.8 GB: byte offsets beyond 2^32.  K is one k-block, so the product is cheap and the
    oracle can check whole rows, among them the last ones."""
    M = N = 49152
    K = 64
    A, B = synth.make_int_inputs(M, N, K, seed=77)
    dA, dB = dev_bf16(A), dev_bf16(B)
    dC = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    rows = [0, 1, 255, 256, 21845, 32767, 32768, 43690, 43691, M - 257, M - 2, M - 1]   # byte offsets up to 4.83e9
    ref, _ = G.gemm_rows(A, B, rows)
    want = G.bf16_bits_to_f64(synth.f32_to_bf16_bits(ref.astype(np.float32)))           # small integers: exact, then RNE
    for scheme, kw, tile in [(sp.HILBERT, {}, (256, 512)), (sp.GROUP_M, dict(group=8), (256, 256)),
                             (sp.ROW_MAJOR, dict(flags=sp.FLAG_CLC), (128, 256))]:
        dC.fill_(float("nan"))
        sp.gemm(dA, dB, dC, scheme, sp.make_params(tile_m=tile[0], tile_n=tile[1], **kw))
        assert sp.get_status() == 0
        got = G.bf16_bits_to_f64(dC[rows].view(torch.int16).cpu().numpy().view(np.uint16))
        assert np.array_equal(got, want), (scheme, tile)
        assert not bool(torch.isnan(dC[:, N - 1].float()).any()) and not bool(torch.isnan(dC[M - 1].float()).any())
        assert not bool(torch.isnan(dC[::997].float()).any())


@pytest.mark.skipif(os.environ.get("SP_FULL_ORACLE") != "1", reason="full fp64 product of 8192^3 takes minutes of CPU: set SP_FULL_ORACLE=1")
def test_cfg3_whole_matrix_against_the_full_oracle_product():
    w, A, B = synth.make_workload("cfg3")
    dA, dB = dev_bf16(A), dev_bf16(B)
    dC = torch.empty((w.M, w.N), dtype=torch.bfloat16, device="cuda")
    sp.gemm(dA, dB, dC, sp.GROUP_N, sp.make_params(tile_m=256, tile_n=512, group=8))
    assert sp.get_status() == 0
    bits = dC.view(torch.int16).cpu().numpy().view(np.uint16)
    for r0 in range(0, w.M, 512):                     # band by band, to bound the host memory of the fp64 arrays
        rows = np.arange(r0, min(r0 + 512, w.M))
        ref, S = G.gemm_rows(A, B, rows)
        r = G.compare(G.bf16_bits_to_f64(bits[rows]), ref, S, K=w.K)
        assert r["max_err"] <= TOL and r["strict_violations"] == 0, (r0, r)
