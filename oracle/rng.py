"""Oracle random streams: Philox4x32-10, open-interval uniforms, a bit-reproducible
normal sampler, synthetic intermediate labels (Eq. 1 of the paper) and the
default Linear initialisation the paper refers to (Section 2).

TEST INFRASTRUCTURE ONLY.  Everything here is written from the published
definition of Philox (Salmon, Moraes, Dror, Shaw, SC'11) and from the written
sampler specification below; it shares nothing with the CUDA implementation.

Pins (tests/test_oracle_rng.py): a big-integer scalar re-derivation of the
round function, bijectivity on a counter range, agreement with the cuRAND
*host* Philox4_32_10 generator (a library routine that needs no GPU),
closed-form moments, a Kolmogorov-Smirnov test against the exact normal CDF,
and the libm values of log / sin / cos.

Counter layout (a choice of this project; the paper does not name a generator):
    key     = (seed mod 2^32, seed div 2^32)
    counter = (q mod 2^32, q div 2^32, segment_id, 4*layer + tag)
for element e of a row-major tensor, q = e div 4 and the output word is e mod 4;
tag 0 = intermediate labels (layer 0), 1 = weight matrix, 2 = bias vector.
Every element therefore depends only on (seed, segment_id, layer, tag, e).
"""
import numpy as np

PHILOX_M0 = 0xD2511F53
PHILOX_M1 = 0xCD9E8D57
PHILOX_W0 = 0x9E3779B9
PHILOX_W1 = 0xBB67AE85
MASK32 = 0xFFFFFFFF

TAG_LABELS = 0
TAG_WEIGHT = 1
TAG_BIAS = 2


def philox4x32_10(c0, c1, c2, c3, k0, k1):
    """Philox4x32 with 10 rounds on arrays of 32-bit words (held in uint64).

    One round (SC'11, Section 3.3 / the S-P network of the 4x32 variant):
        (hi0, lo0) = M0 * c0,  (hi1, lo1) = M1 * c2       (32x32 -> 64 bit)
        c' = (hi1 ^ c1 ^ k0,  lo1,  hi0 ^ c3 ^ k1,  lo0)
    and between rounds the key is bumped by the Weyl constants (W0, W1).
    """
    c0 = np.asarray(c0, dtype=np.uint64) & MASK32
    c1 = np.asarray(c1, dtype=np.uint64) & MASK32
    c2 = np.asarray(c2, dtype=np.uint64) & MASK32
    c3 = np.asarray(c3, dtype=np.uint64) & MASK32
    k0 = np.uint64(int(k0) & MASK32)
    k1 = np.uint64(int(k1) & MASK32)
    for r in range(10):
        p0 = np.uint64(PHILOX_M0) * c0
        p1 = np.uint64(PHILOX_M1) * c2
        hi0, lo0 = p0 >> np.uint64(32), p0 & np.uint64(MASK32)
        hi1, lo1 = p1 >> np.uint64(32), p1 & np.uint64(MASK32)
        c0, c1, c2, c3 = hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0
        if r != 9:
            k0 = (k0 + np.uint64(PHILOX_W0)) & np.uint64(MASK32)
            k1 = (k1 + np.uint64(PHILOX_W1)) & np.uint64(MASK32)
    return c0, c1, c2, c3


def stream_words(seed, segment_id, layer, tag, n_elements):
    """The first n_elements 32-bit words of stream (seed, segment_id, layer, tag)."""
    n_blocks = (n_elements + 3) // 4
    q = np.arange(n_blocks, dtype=np.uint64)
    w = philox4x32_10(q & np.uint64(MASK32), q >> np.uint64(32),
                      np.uint64(segment_id), np.uint64(4 * layer + tag),
                      seed & MASK32, (seed >> 32) & MASK32)
    return np.stack(w, axis=1).reshape(-1)[:n_elements]


def uniform_open01(words):
    """Map 32-bit words to fp32 uniforms strictly inside (0, 1).

    u = (2*(r >> 9) + 1) * 2^-24: an odd 24-bit integer times a power of two, so it
    is exact in fp32, never 0 and never 1 (the open interval of Eq. 1).
    """
    k = (np.asarray(words, dtype=np.uint64) >> np.uint64(9)).astype(np.int64)
    return ((2 * k + 1).astype(np.float32) * np.float32(2.0 ** -24)).astype(np.float32)


# ---- bit-reproducible standard normal ------------------------------------------------
# Specification (a choice of this project).  Only integer operations and individually
# rounded IEEE-754 binary64 +, -, *, /, sqrt are used, in exactly the order written,
# so that any independent implementation following the same text agrees bit for bit.
#
# Words (r0, r1) of one Philox block give two normals (Box-Muller, 1958):
#   n  = 2*(r0 >> 9) + 1                      odd integer in [1, 2^24); u1 = n * 2^-24
#   L  = ln(u1) = (e - 24)*LN2 + 2*atanh(s)   with n = m * 2^e, m in [1, 2); if m > SQRT2:
#        m = m/2, e = e + 1;  s = (m - 1)/(m + 1);  z = s*s;
#        atanh part P = s*(C0 + z*(C1 + ... + z*C7)),  Ck = 2/(2k+1)   (Horner, inner first)
#   rad = sqrt(-2 * L)
#   j  = r1 >> 8 (24 bits); quadrant = j >> 22; t = j & (2^22 - 1); octant bit o = t >> 21;
#        t' = t & (2^21 - 1); if o: t' = 2^21 - 1 - t';  psi = (t' + 0.5) * (PI/4 * 2^-21)
#        sin psi, cos psi by their Taylor polynomials in y = psi*psi (degrees 15 and 14);
#        if o: swap;  rotate by the quadrant.
#   z0 = fp32(rad * cos), z1 = fp32(rad * sin)   (round to nearest even)
LN2 = float.fromhex("0x1.62e42fefa39efp-1")
SQRT2 = float.fromhex("0x1.6a09e667f3bcdp+0")
PI_4_2M21 = float.fromhex("0x1.921fb54442d18p-1") * 2.0 ** -21   # (pi/4) * 2^-21, exact scaling
ATANH_C = [2.0 / (2 * k + 1) for k in range(8)]                   # correctly rounded quotients
SIN_C = [1.0, -1.0 / 6, 1.0 / 120, -1.0 / 5040, 1.0 / 362880, -1.0 / 39916800, 1.0 / 6227020800,
         -1.0 / 1307674368000]
COS_C = [1.0, -1.0 / 2, 1.0 / 24, -1.0 / 720, 1.0 / 40320, -1.0 / 3628800, 1.0 / 479001600,
         -1.0 / 87178291200]


def _horner(coeffs, y):
    acc = np.full_like(y, coeffs[-1])
    for c in reversed(coeffs[:-1]):
        acc = acc * y          # one rounded multiply
        acc = acc + c          # one rounded add
    return acc


def spec_log_u(n):
    """ln(n * 2^-24) for odd integers n in [1, 2^24), by the specification above (fp64)."""
    n = np.asarray(n, dtype=np.int64)
    e = np.zeros(n.shape, dtype=np.int64)
    for bit in range(1, 24):                       # e = floor(log2 n), integer only
        e = np.where(n >= (1 << bit), bit, e)
    m = n.astype(np.float64) / np.exp2(e.astype(np.float64))   # exact: division by a power of two
    big = m > SQRT2
    m = np.where(big, m * 0.5, m)
    e = np.where(big, e + 1, e)
    s = (m - 1.0) / (m + 1.0)
    z = s * s
    p = s * _horner(ATANH_C, z)
    return (e - 24).astype(np.float64) * LN2 + p


def spec_sincos(j):
    """(cos, sin) of the angle selected by the 24-bit integer j, by the specification above."""
    j = np.asarray(j, dtype=np.int64)
    quad = j >> 22
    t = j & ((1 << 22) - 1)
    o = (t >> 21) == 1
    tp = t & ((1 << 21) - 1)
    tp = np.where(o, (1 << 21) - 1 - tp, tp)
    psi = (tp.astype(np.float64) + 0.5) * PI_4_2M21
    y = psi * psi
    s = psi * _horner(SIN_C, y)
    c = _horner(COS_C, y)
    s, c = np.where(o, c, s), np.where(o, s, c)
    cos_q = np.select([quad == 0, quad == 1, quad == 2], [c, -s, -c], default=s)
    sin_q = np.select([quad == 0, quad == 1, quad == 2], [s, c, -s], default=-c)
    return cos_q, sin_q


def normal_pairs(r0, r1):
    """Two fp32 standard normals from each word pair (r0, r1)."""
    n = 2 * (np.asarray(r0, dtype=np.uint64) >> np.uint64(9)).astype(np.int64) + 1
    j = (np.asarray(r1, dtype=np.uint64) >> np.uint64(8)).astype(np.int64)
    rad = np.sqrt(-2.0 * spec_log_u(n))
    c, s = spec_sincos(j)
    return (rad * c).astype(np.float32), (rad * s).astype(np.float32)


def standard_normal(words):
    """fp32 normals for a word stream whose length is a multiple of 4:
    element 4q+0/1 = (z0, z1) of words (4q, 4q+1); element 4q+2/3 = (z0, z1) of words (4q+2, 4q+3)."""
    w = np.asarray(words, dtype=np.uint64).reshape(-1, 2)
    z0, z1 = normal_pairs(w[:, 0], w[:, 1])
    return np.stack([z0, z1], axis=1).reshape(-1)


# ---- the method's random tensors -----------------------------------------------------
DIST_UNIFORM_KAPPA = 0      # Eq. 1: SIL_ij ~ kappa * U(0,1)
DIST_NORMAL = 1             # N(0,1) targets used by the synthetic workloads


def gen_labels(seed, segment_id, n_classes, n_p, dist=DIST_UNIFORM_KAPPA, kappa=10.0):
    """Synthetic intermediate labels for one cut (Eq. 1; Section 3 gives 60 x 47, kappa = 10).

    Returned as [M, N_P] fp32, i.e. the paper's N_P x M matrix stored column by column:
    row j is the target vector of class j.  Element (j, i) is stream element j*N_P + i.
    """
    n = n_classes * n_p
    words = stream_words(seed, segment_id, 0, TAG_LABELS, 4 * ((n + 3) // 4))
    if dist == DIST_UNIFORM_KAPPA:
        vals = (np.float32(kappa) * uniform_open01(words)).astype(np.float32)
    elif dist == DIST_NORMAL:
        vals = standard_normal(words)
    else:
        raise ValueError("unknown label distribution")
    return vals[:n].reshape(n_classes, n_p)


def init_linear(seed, segment_id, layer, fan_in, fan_out):
    """Default Linear initialisation (Section 2 cites the framework default):
    W, b ~ U(-1/sqrt(fan_in), +1/sqrt(fan_in)), drawn as (2u - 1) * bound."""
    bound = np.float32(1.0) / np.sqrt(np.float32(fan_in))
    uw = uniform_open01(stream_words(seed, segment_id, layer, TAG_WEIGHT, fan_in * fan_out))
    ub = uniform_open01(stream_words(seed, segment_id, layer, TAG_BIAS, fan_out))
    W = ((np.float32(2.0) * uw - np.float32(1.0)) * bound).astype(np.float32)
    b = ((np.float32(2.0) * ub - np.float32(1.0)) * bound).astype(np.float32)
    return W.reshape(fan_out, fan_in), b
