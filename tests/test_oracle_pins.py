"""Pins for the CPU oracle: each test checks it against something other than itself.

The paper prints no numeric example, so the pins are: the IEEE definitions of fp16/bf16 via numpy
and torch casts, exact integer / rational brute force on tiny shapes, identities, numpy's float64
matmul, the translation closed form (Listing 1), hand-worked fixtures under tests/golden/, and
direct numpy restatements of the byte-movement semantics (Table 3).
"""
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from paper_2511_12500_b200 import inputs

GOLD = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------------------- codec
def test_decode_fp16_all_patterns_matches_numpy():
    bits = np.arange(65536, dtype=np.uint16)
    ref = bits.view(np.float16).astype(np.float64)
    got = oracle.decode(bits, "fp16")
    assert np.array_equal(np.isnan(ref), np.isnan(got))
    ok = ~np.isnan(ref)
    assert np.array_equal(ref[ok], got[ok])
    assert np.array_equal(np.signbit(ref[ok]), np.signbit(got[ok]))


def test_decode_bf16_all_patterns_matches_bit_shift():
    bits = np.arange(65536, dtype=np.uint16)
    ref = (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    got = oracle.decode(bits, "bf16")
    ok = ~np.isnan(ref)
    assert np.array_equal(np.isnan(ref), np.isnan(got))
    assert np.array_equal(ref[ok], got[ok])
    assert np.array_equal(np.signbit(ref[ok]), np.signbit(got[ok]))


@pytest.mark.parametrize("dtype", ["fp16", "bf16"])
def test_encode_round_trips_every_non_nan_pattern(dtype):
    bits = np.arange(65536, dtype=np.uint16)
    vals = oracle.decode(bits, dtype)
    ok = ~np.isnan(vals)
    assert np.array_equal(oracle.encode(vals[ok], dtype), bits[ok])


def test_encode_fp16_matches_numpy_direct_cast():
    rng = np.random.default_rng(1)
    x = np.concatenate([rng.uniform(-70000, 70000, 200000), rng.normal(0, 1e-4, 200000),
                        rng.normal(0, 1e-7, 100000), [0.0, -0.0, 65504.0, 65519.9, 65520.0, 1e9, -1e9,
                                                      2.0 ** -24, 2.0 ** -25, 2.0 ** -25 * 1.0000001, 2.0 ** -14]])
    with np.errstate(over="ignore"):
        ref = x.astype(np.float16).view(np.uint16)   # numpy converts double -> half directly (one rounding)
    assert np.array_equal(oracle.encode(x, "fp16"), ref)


def test_encode_bf16_matches_torch_on_fp32_values_and_ties():
    rng = np.random.default_rng(2)
    x32 = np.concatenate([rng.normal(0, 1, 300000), rng.normal(0, 1e-30, 1000), rng.normal(0, 1e30, 1000)]).astype(np.float32)
    ref = torch.from_numpy(x32).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(oracle.encode(x32.astype(np.float64), "bf16"), ref)
    # ties to even at 1 + 2^-8 (between 1.0 and 1 + 2^-7) and 1 + 3*2^-8
    assert oracle.encode(np.array([1 + 2.0 ** -8]), "bf16")[0] == 0x3F80
    assert oracle.encode(np.array([1 + 3 * 2.0 ** -8]), "bf16")[0] == 0x3F82
    # a value just above the tie must round up even though an fp32 detour would land on the tie
    assert oracle.encode(np.array([1 + 2.0 ** -8 + 2.0 ** -40]), "bf16")[0] == 0x3F81
    # overflow to inf, largest finite stays
    assert oracle.encode(np.array([3.4e38]), "bf16")[0] == 0x7F80
    assert oracle.encode(np.array([float(np.float32(3.3895314e38))]), "bf16")[0] == 0x7F7F


# ----------------------------------------------------------------------------- translate
def test_translate_golden_cases():
    for line in open(os.path.join(GOLD, "translate_cases.txt")):
        if line.startswith("#") or not line.strip():
            continue
        b0, b1, b2, bpr, ptr, frm, to, exp = map(int, line.split())
        assert oracle.translate([b0, b1, b2], bpr, ptr, frm, to) == exp


def test_translate_algebra_exhaustive_tiny_heap():
    bases, bpr = [4096, 64, 1024, 512], 64
    W = len(bases)
    for a in range(W):
        for off in range(bpr):
            p = bases[a] + off
            assert oracle.translate(bases, bpr, p, a, a) == p
            for b in range(W):
                q = oracle.translate(bases, bpr, p, a, b)
                assert q - bases[b] == off                       # offset preserved
                assert oracle.translate(bases, bpr, q, b, a) == p  # inverse
                for c in range(W):
                    assert oracle.translate(bases, bpr, q, b, c) == oracle.translate(bases, bpr, p, a, c)
    with pytest.raises(IndexError):
        oracle.translate(bases, bpr, bases[0] + bpr, 0, 1)   # one past the end
    with pytest.raises(IndexError):
        oracle.translate(bases, bpr, bases[0] - 1, 0, 1)
    with pytest.raises(ValueError):
        oracle.translate(bases, bpr, bases[0], 0, 4)


# ----------------------------------------------------------------------------- GEMM
def _int_inputs(seed, W, M, nl, K, dtype, k=3):
    A = inputs.matrix(seed, 0, M, K, f"smallint:{k}", dtype)
    Bs = [inputs.matrix(seed, 1 + r, nl, K, f"smallint:{k}", dtype) for r in range(W)]
    return A, Bs


@pytest.mark.parametrize("dtype", ["fp16", "bf16"])
@pytest.mark.parametrize("W,M,nl,K", [(1, 3, 5, 7), (2, 4, 3, 16), (3, 16, 2, 5), (4, 7, 4, 9)])
def test_gemm_brute_force_exact_integers(dtype, W, M, nl, K):
    A, Bs = _int_inputs(7, W, M, nl, K, dtype)
    Ai = oracle.decode(A, dtype).astype(np.int64)
    Bi = [oracle.decode(b, dtype).astype(np.int64) for b in Bs]
    c16 = oracle.gemm_block(A, Bs, dtype)
    got = oracle.decode(c16, dtype)
    for m in range(M):
        for n in range(W * nl):
            r, j = divmod(n, nl)
            exact = sum(int(Ai[m, k]) * int(Bi[r][j, k]) for k in range(K))  # python ints, i-j-k order
            assert got[m, n] == exact, (m, n)


def test_gemm_unrounded_sum_matches_exact_rationals():
    W, M, nl, K = 2, 5, 3, 33
    A, Bs = inputs.gemm_inputs(11, W, M, W * nl, K, "uniform", "fp16")
    Ad = oracle.decode(A, "fp16")
    Bd = [oracle.decode(b, "fp16") for b in Bs]
    _, c64 = oracle.gemm_block(A, Bs, "fp16", want_exact=True)
    for m in range(M):
        for n in range(W * nl):
            r, j = divmod(n, nl)
            exact = sum(Fraction(float(Ad[m, k])) * Fraction(float(Bd[r][j, k])) for k in range(K))
            scale = sum(abs(Ad[m, k] * Bd[r][j, k]) for k in range(K)) + 1e-300
            assert abs(Fraction(float(c64[m, n])) - exact) <= Fraction(scale) * Fraction(1, 10 ** 14)


@pytest.mark.parametrize("dtype", ["fp16", "bf16"])
def test_gemm_matches_numpy_float64_matmul(dtype):
    W, M, nl, K = 4, 37, 24, 200
    A, Bs = inputs.gemm_inputs(12, W, M, W * nl, K, "normal002" if dtype == "bf16" else "uniform", dtype)
    c16, c64 = oracle.gemm_block(A, Bs, dtype, want_exact=True)
    Ad = oracle.decode(A, dtype)
    Bcat = np.concatenate([oracle.decode(b, dtype) for b in Bs], axis=0)   # [N, K]
    ref = Ad @ Bcat.T
    bound = (np.abs(Ad) @ np.abs(Bcat).T) * 1e-12 + 1e-300
    assert np.all(np.abs(ref - c64) <= bound)
    # the rounded result is the correctly rounded unrounded one (numpy's direct double->half cast decides for fp16)
    if dtype == "fp16":
        assert np.array_equal(c16, c64.astype(np.float16).view(np.uint16))


@pytest.mark.parametrize("dtype", ["fp16", "bf16"])
def test_gemm_identity_B_reproduces_A(dtype):
    W, M, K = 2, 9, 16
    A = inputs.matrix(3, 0, M, K, "uniform", dtype)
    A[A == 0x8000] = 0  # no negative zeros: 0 + (-0)*1 is +0 in any summation order
    eye = oracle.encode(np.eye(K), dtype)
    Bs = [np.ascontiguousarray(eye[r * (K // W):(r + 1) * (K // W)]) for r in range(W)]
    assert np.array_equal(oracle.gemm_block(A, Bs, dtype), A)


@pytest.mark.parametrize("dtype", ["fp16", "bf16"])
def test_gemm_zero_A_gives_positive_zero(dtype):
    A = np.zeros((5, 12), dtype=np.uint16)
    Bs = [inputs.matrix(4, 1 + r, 6, 12, "uniform", dtype) for r in range(2)]
    assert not oracle.gemm_block(A, Bs, dtype).any()


def test_gemm_one_hot_row_copies_a_B_row_and_pow2_scaling_is_exact():
    dtype, K = "bf16", 24
    Bs = [inputs.matrix(5, 1 + r, 4, K, "uniform", dtype) for r in range(2)]
    for b in Bs:
        b[b == 0x8000] = 0
    A = np.zeros((K, K), dtype=np.uint16)
    for k in range(K):
        A[k, k] = oracle.encode(np.array([4.0]), dtype)[0]      # A = 4 I  =>  C[k, n] = 4 * Bcat[n, k]
    C = oracle.decode(oracle.gemm_block(A, Bs, dtype), dtype)
    Bcat = np.concatenate([oracle.decode(b, dtype) for b in Bs], axis=0)
    assert np.array_equal(C, 4.0 * Bcat.T)


def test_gemm_block_equals_slice_of_full():
    W, M, nl, K = 2, 40, 24, 50
    A, Bs = inputs.gemm_inputs(13, W, M, W * nl, K, "uniform", "fp16")
    full = oracle.gemm_block(A, Bs, "fp16")
    blk = oracle.gemm_block(A, Bs, "fp16", 7, 33, 19, 41)   # crosses the rank boundary at n = 24
    assert np.array_equal(blk, full[7:33, 19:41])


def test_tiny_hand_worked_fixture():
    rows = {"A": [], "B0": [], "B1": [], "C": [], "OFFSET": []}
    for line in open(os.path.join(GOLD, "tiny_gemm_all_scatter.txt")):
        if line.startswith("#") or not line.strip():
            continue
        key, *vals = line.split()
        rows[key].append([int(v) for v in vals])
    dtype = "fp16"
    A = oracle.encode(np.array(rows["A"], dtype=np.float64), dtype)
    Bs = [oracle.encode(np.array(rows[k], dtype=np.float64), dtype) for k in ("B0", "B1")]
    C = np.array(rows["C"], dtype=np.float64)
    M, N, W = 2, 4, 2
    img = oracle.HeapImage(W, 256, fill=0xAB)
    img.gemm_all_scatter(A, Bs, dtype, c_off=64, flag_off=0, epoch=5)
    for s in range(W):
        assert np.array_equal(oracle.decode(img.view(s, 64, M * N * 2, np.uint16), dtype).reshape(M, N), C)
    r, m, rn, off = rows["OFFSET"][0]
    flat = oracle.decode(img.view(0, 64, M * N * 2, np.uint16), dtype)
    assert flat[off] == C[m, rn + r * (N // W)]


# ----------------------------------------------------------------------------- scatter / flags / locks
def test_all_scatter_replication_sentinel_and_flags():
    W, M, nl, K, dtype = 4, 130, 136, 16, "bf16"     # ragged in both directions
    N = W * nl
    A, Bs = inputs.gemm_inputs(21, W, M, N, K, "uniform", dtype)
    c_off, flag_off, lock_off = 512, 0, 256
    bpr = c_off + M * N * 2 + 128
    img = oracle.HeapImage(W, bpr, fill=0xCD)
    c_full = img.gemm_all_scatter(A, Bs, dtype, c_off, flag_off, epoch=3, lock_off=lock_off)
    nt = oracle.num_tiles(M, N, W)
    assert nt == 2 * W * 2 and nt * 4 <= 256
    for s in range(W):
        assert np.array_equal(img.view(s, c_off, M * N * 2, np.uint16).reshape(M, N), c_full)   # all W copies identical
        assert np.all(img.view(s, flag_off, nt * 4, np.int32) == 3)
        assert np.all(img.view(s, c_off + M * N * 2, 128) == 0xCD)          # past C: untouched
        assert np.all(img.view(s, nt * 4, 256 - nt * 4) == 0xCD)           # between flags and locks: untouched
        locks = img.view(s, lock_off, nt * 4, np.int32)
        tnl = 2
        for t in range(nt):
            owner = (t % (W * tnl)) // tnl
            assert locks[t] == (0 if owner == s else np.frombuffer(bytes([0xCD] * 4), np.int32)[0])


def test_tile_rect_partitions_C_without_straddling_ranks():
    for (M, N, W) in [(256, 256, 2), (130, 544, 4), (128, 28672, 8), (1, 8, 1), (300, 24, 3)]:
        nl = N // W
        cover = np.zeros((M, N), dtype=np.int32)
        for t in range(oracle.num_tiles(M, N, W)):
            m0, m1, n0, n1 = oracle.tile_rect(t, M, N, W)
            assert m1 > m0 and n1 > n0 and m1 - m0 <= 128 and n1 - n0 <= 128
            assert n0 // nl == (n1 - 1) // nl
            cover[m0:m1, n0:n1] += 1
        assert np.all(cover == 1)


# ----------------------------------------------------------------------------- put / get / atomics
def test_put_get_semantics_against_numpy_slicing():
    W, bpr = 3, 4096
    rng = np.random.default_rng(5)
    img = oracle.HeapImage(W, bpr)
    img.mem[:] = rng.integers(0, 256, img.mem.size, dtype=np.uint8)
    before = img.mem.copy().reshape(W, bpr)
    rows, rb, sp, dp, so, do = 5, 24, 40, 56, 100, 1000
    img.put(so, do, rows, rb, sp, dp, from_rank=0, to_rank=2)
    exp = before.copy()
    for i in range(rows):
        exp[2, do + i * dp: do + i * dp + rb] = before[0, so + i * sp: so + i * sp + rb]
    assert np.array_equal(img.mem.reshape(W, bpr), exp)
    img.get(so, do, rows, rb, sp, dp, from_rank=1, to_rank=2)      # rank 1 pulls from rank 2
    exp2 = exp.copy()
    for i in range(rows):
        exp2[1, do + i * dp: do + i * dp + rb] = exp[2, so + i * sp: so + i * sp + rb]
    assert np.array_equal(img.mem.reshape(W, bpr), exp2)
    with pytest.raises(ValueError):
        img.put(bpr - 8, 0, 1, 16, 16, 16, 0, 1)


def test_atomics_sequential_semantics():
    img = oracle.HeapImage(2, 256)
    old = [int(img.atomic_add(16, 1, 4, 1, 1)[0]) for _ in range(10)]
    assert old == list(range(10)) and img.view(1, 16, 4, np.int32)[0] == 10 and img.view(0, 16, 4, np.int32)[0] == 0
    assert img.atomic_cas(16, 1, 4, 1, cmp=3, val=99)[0] == 10 and img.view(1, 16, 4, np.int32)[0] == 10   # miss
    assert img.atomic_cas(16, 1, 4, 1, cmp=10, val=99)[0] == 10 and img.view(1, 16, 4, np.int32)[0] == 99  # hit
    olds = img.atomic_add(32, 4, 8, 0, -2)     # strided vector form, negative addend wraps like int32
    assert list(olds) == [0, 0, 0, 0] and list(img.view(0, 32, 32, np.int32)[::2]) == [-2] * 4


def test_u64_atomics_against_python_integers():
    """64-bit add wraps modulo 2**64 and returns the previous word; cas writes only on a match.  Checked against python's
    unbounded integers (reduced mod 2**64) on values that overflow 32 bits and 64 bits, strided, in one rank only."""
    rng = np.random.default_rng(11)
    n, stride, off = 33, 16, 64
    init = [int(x) for x in rng.integers(0, 2**64, n, dtype=np.uint64)]
    init[0], init[1], init[2] = 2**64 - 1, 2**32 - 1, 0
    img = oracle.HeapImage(3, 1024)
    img.view(2, off, n * stride, np.uint64)[::2] = np.array(init, dtype=np.uint64)
    for val in (1, 2**32, 2**63 + 5, 2**64 - 1):
        old = img.atomic_add_u64(off, n, stride, 2, val)
        assert [int(x) for x in old] == init
        init = [(x + val) % 2**64 for x in init]
        assert [int(x) for x in img.view(2, off, n * stride, np.uint64)[::2]] == init
    assert not img.view(2, off, n * stride, np.uint64)[1::2].any()          # the words between the strided ones
    assert not img.slot(0).any() and not img.slot(1).any()                  # other ranks untouched
    # cas: the high half alone must not match
    word = 0x1234_5678_9ABC_DEF0
    img.view(1, 8, 8, np.uint64)[0] = word
    assert int(img.atomic_cas_u64(8, 1, 8, 1, word & 0xFFFFFFFF, 7)[0]) == word and int(img.view(1, 8, 8, np.uint64)[0]) == word
    assert int(img.atomic_cas_u64(8, 1, 8, 1, word ^ (1 << 63), 7)[0]) == word and int(img.view(1, 8, 8, np.uint64)[0]) == word
    assert int(img.atomic_cas_u64(8, 1, 8, 1, word, 2**64 - 2)[0]) == word and int(img.view(1, 8, 8, np.uint64)[0]) == 2**64 - 2
    with pytest.raises(ValueError):
        img.atomic_add_u64(1024 - 4, 1, 8, 0, 1)                            # the word would leave the slot


def test_remaining_atomics_against_numpy_semantics():
    rng = np.random.default_rng(9)
    init = rng.integers(-2**31, 2**31 - 1, 64, dtype=np.int64).astype(np.int32)
    val = int(np.int32(rng.integers(-2**31, 2**31 - 1)))
    ref = {"add": (init.astype(np.int64) + val).astype(np.int32), "xchg": np.full_like(init, val), "and": init & np.int32(val),
           "or": init | np.int32(val), "xor": init ^ np.int32(val), "min": np.minimum(init, np.int32(val)), "max": np.maximum(init, np.int32(val))}
    for op, expect in ref.items():
        img = oracle.HeapImage(2, 1024)
        img.view(1, 128, 256, np.int32)[:] = init
        old = img.atomic_rmw(op, 128, 64, 4, 1, val)
        assert np.array_equal(old, init), op
        assert np.array_equal(img.view(1, 128, 256, np.int32), expect), op
        assert not img.slot(0).any()


def test_copy_between_two_other_ranks():
    W, bpr = 4, 2048
    rng = np.random.default_rng(6)
    img = oracle.HeapImage(W, bpr)
    img.mem[:] = rng.integers(0, 256, img.mem.size, dtype=np.uint8)
    before = img.mem.copy().reshape(W, bpr)
    img.copy(64, 1024, 3, 20, 32, 48, from_rank=1, to_rank=3)
    exp = before.copy()
    for i in range(3):
        exp[3, 1024 + i * 48: 1024 + i * 48 + 20] = before[1, 64 + i * 32: 64 + i * 32 + 20]
    assert np.array_equal(img.mem.reshape(W, bpr), exp)


# ----------------------------------------------------------------------------- consumer
def test_consumer_matches_library_float32_add():
    M, N = 9, 40
    c = inputs.matrix(31, 0, M, N, "uniform", "fp16")
    b = inputs.vector(31, 100, N, "uniform", "fp16")
    ref = (c.view(np.float16).astype(np.float32) + b.view(np.float16).astype(np.float32)[None, :]).astype(np.float16)
    assert np.array_equal(oracle.consume_bias_rows(c, b, "fp16"), ref.view(np.uint16))
    c = inputs.matrix(32, 0, M, N, "uniform", "bf16")
    b = inputs.vector(32, 100, N, "uniform", "bf16")
    tc = torch.from_numpy(c.view(np.int16)).view(torch.bfloat16).float()
    tb = torch.from_numpy(b.view(np.int16)).view(torch.bfloat16).float()
    ref = (tc + tb[None, :]).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(oracle.consume_bias_rows(c, b, "bf16"), ref)


# ----------------------------------------------------------------------------- all-store
def test_all_store_end_state():
    W, S, tile = 4, 1000, 256
    T = -(-S // tile)
    payload_off, recv_off, flag_off = 0, 1024, 1024 + W * S
    bpr = flag_off + W * T * 4 + 64
    img = oracle.HeapImage(W, bpr, fill=0x11)
    pay = [inputs.payload_bytes(41, 200 + r, S) for r in range(W)]
    for r in range(W):
        img.view(r, payload_off, S)[:] = pay[r]
        img.view(r, flag_off, W * T * 4, np.int32)[:] = 6
    img.all_store(payload_off, recv_off, flag_off, S, tile, epoch=7)
    for s in range(W):
        for r in range(W):
            assert np.array_equal(img.view(s, recv_off + r * S, S), pay[r])
        assert np.all(img.view(s, flag_off, W * T * 4, np.int32) == 7)
        assert np.all(img.view(s, flag_off + W * T * 4, 64) == 0x11)
    img.all_store(payload_off, recv_off, flag_off, S, tile, epoch=7)       # cas(6 -> 7) misses now: flags stay
    assert np.all(img.view(0, flag_off, W * T * 4, np.int32) == 7)


# ----------------------------------------------------------------------------- input generator
def test_generator_is_counter_based_and_in_range():
    full = inputs.matrix(inputs.SEED0, 0, 64, 48, "uniform", "fp16")
    part = inputs.matrix(inputs.SEED0, 0, 64, 48, "uniform", "fp16", 10, 20)
    assert np.array_equal(full[10:20], part)
    v = oracle.decode(full, "fp16")
    assert v.min() >= -1.0 and v.max() <= 1.0 and abs(v.mean()) < 0.05
    z = oracle.decode(inputs.matrix(inputs.SEED0, 1, 200, 200, "normal002", "bf16"), "bf16")
    assert abs(z.std() - 0.02) < 0.001 and abs(z.mean()) < 0.001
    t = oracle.decode(inputs.matrix(1, 2, 100, 100, "ternary:0.25", "bf16"), "bf16")
    assert set(np.unique(t)) <= {-1.0, 0.0, 1.0} and 0.15 < np.mean(t != 0) < 0.35
