"""Oracle for one synchronisation + update step of QCMD adagrad / QRDA adagrad.

TEST INFRASTRUCTURE ONLY (see the package docstring).  Every function restates one
passage of the paper in numpy.  Floating point is fp64 except where a comparison
decides an integer code: there the operands are fp32, like the data they come from.

Conventions the paper leaves open (each is this library's documented reading):

* 2-bit code per coordinate: 0 -> 0, 1 -> +1, 2 -> -1, 3 is never produced and decodes
  to 0.  Coordinate i sits in 32-bit word i // 16 at bits [2*(i%16), 2*(i%16)+1].
* The sums over a worker's gradient ("canonical sum") are taken in one fixed order so
  that the fp64 result, and the fp32 threshold / scale rounded from it, do not depend
  on who computes them.  See `canonical_sum`.
* The stochastic ternary quantizer (the unbiased comparison quantizer the paper's
  theorems assume) draws from Philox4x32-10 keyed by (seed, t, m, i).
* Scalars lambda, eta, delta and the threshold coefficient are fp32 at the library
  boundary; they are promoted exactly to fp64 here.

Parity unpinned (the paper fixes none of these, so no outside value can pin them):
the order of additions inside `canonical_sum` and `canonical_prefix` (their last fp64
bits), the bit layout of `pack_codes`, and the way `philox_draws` maps (seed, t, m, i)
to counter and key words.  What the tests pin instead: both sums as sums (exact where
the partial sums are representable, within the pairwise error bound of the exactly
rounded sum otherwise; the fp32 threshold equal to the exactly rounded definition on
the seeded cases), the Philox block function by its published known-answer vectors,
and pack/unpack as inverse maps.
"""
import numpy as np

F32 = np.float32
F64 = np.float64

QUANT_THRESHOLD = 0
QUANT_TERNARY_STOCH = 1
QUANT_NONE = 2
RULE_CMD = 0
RULE_RDA = 1

# Geometry of the canonical sum: a tile is TILE_ROWS rows of TILE_COLS consecutive
# coordinates (row-major), i.e. 4096 consecutive coordinates.
TILE_ROWS = 4
TILE_COLS = 1024
TILE = TILE_ROWS * TILE_COLS


# ----------------------------------------------------------------------------------
# Canonical summation
# ----------------------------------------------------------------------------------
def _adjacent_pairs(a):
    """Pairwise (recursive halving) sum along the last axis, whose length is 2**k:
    level by level, element 2j is added to element 2j+1."""
    while a.shape[-1] > 1:
        a = a[..., 0::2] + a[..., 1::2]
    return a[..., 0]


def pairwise_sum(a):
    """Pairwise sum of a 1-D fp64 vector, zero-padded (+0.0) to the next power of two."""
    a = np.asarray(a, dtype=F64).ravel()
    n = max(1, a.size)
    p = 1 << (n - 1).bit_length()
    buf = np.zeros(p, dtype=F64)
    buf[: a.size] = a
    return F64(_adjacent_pairs(buf))


def canonical_sum(a):
    """Sum of a non-negative fp32 vector in the library's fixed order.

    The vector is cut into tiles of 4096 consecutive coordinates (the last one padded
    with +0.0).  A tile is read as 4 rows x 1024 columns; each column is summed down
    its 4 rows, in row order, in fp64; the 1024 column sums are combined by pairwise
    summation; the tile sums are combined by pairwise summation over the tile index
    (padded with +0.0 to a power of two).  All additions are fp64.
    """
    a = np.asarray(a, dtype=F32).ravel()
    d = a.size
    n_tiles = max(1, -(-d // TILE))
    buf = np.zeros(n_tiles * TILE, dtype=F32)
    buf[:d] = a
    buf = buf.reshape(n_tiles, TILE_ROWS, TILE_COLS)
    col = buf[:, 0, :].astype(F64)
    for r in range(1, TILE_ROWS):
        col = col + buf[:, r, :].astype(F64)
    tile_sums = _adjacent_pairs(col)
    return pairwise_sum(tile_sums)


# ----------------------------------------------------------------------------------
# Threshold quantization (Section 3.4, Q_Delta; threshold from Section 3.5)
# ----------------------------------------------------------------------------------
def threshold_quantize(v, coef=0.75):
    """Q_Delta(v) = s * tern with the approximate threshold of Section 3.5.

    Delta = coef/d * sum_i |v_i|                      (Section 3.5, coef = 0.75)
    tern_i = +1 if v_i > Delta, -1 if v_i < -Delta, 0 if |v_i| <= Delta   (Section 3.4)
    s = mean of |v_i| over I_Delta = {i : |v_i| > Delta}                   (s*_Delta)

    Returns (tern int8[d], s fp32, Delta fp32, |I_Delta| int).  An empty I_Delta gives
    s = 0.  The comparisons are fp32 against the fp32 Delta.
    """
    v = np.asarray(v, dtype=F32).ravel()
    d = v.size
    absv = np.abs(v)
    with np.errstate(invalid="ignore", over="ignore"):
        total = canonical_sum(absv)
        delta = F32((F64(F32(coef)) * total) / F64(d))
        pos = v > delta
        neg = v < -delta
    tern = pos.astype(np.int8) - neg.astype(np.int8)
    selected = pos | neg
    n = int(np.count_nonzero(selected))
    if n == 0:
        return tern, F32(0.0), delta, 0
    picked = canonical_sum(np.where(selected, absv, F32(0.0)))
    scale = F32(picked / F64(n))
    return tern, scale, delta, n


# ----------------------------------------------------------------------------------
# Exact optimal threshold (Section 3.4: rank the components, try each as the threshold)
# ----------------------------------------------------------------------------------
SCAN_WARP = 32
SCAN_BLOCK = SCAN_WARP * SCAN_WARP   # 1024


def _doubling_scan(x):
    """Inclusive prefix sums along the last axis by recursive doubling: at step s = 1, 2, 4, ...
    every element i >= s becomes x[i - s] + x[i], all at once."""
    x = np.array(x, dtype=F64)
    s = 1
    while s < x.shape[-1]:
        y = x.copy()
        y[..., s:] = x[..., :-s] + x[..., s:]
        x = y
        s *= 2
    return x


def _block_scan(x):
    """Inclusive prefix sums of blocks of 1024 (last axis): doubling scan inside each run of 32,
    doubling scan of the 32 run totals, then (sum of the runs before) + (value inside the run)."""
    lead = x.shape[:-1]
    runs = _doubling_scan(np.asarray(x, dtype=F64).reshape(lead + (SCAN_WARP, SCAN_WARP)))
    totals = _doubling_scan(runs[..., -1])
    before = np.concatenate([np.zeros(lead + (1,), dtype=F64), totals[..., :-1]], axis=-1)
    return (before[..., None] + runs).reshape(lead + (SCAN_BLOCK,))


def canonical_prefix(a):
    """Inclusive prefix sums P_i = a_0 + ... + a_i of a non-negative vector in fp64, in one fixed
    order (like `canonical_sum`, a convention of this library so that every implementation gets the
    same bits): blocks of 1024 elements scanned by `_block_scan`; the block totals of each group of
    1024 blocks scanned the same way; the group totals added one after the other;
    P_i = (sum of the groups before + sum of the blocks before inside the group) + value in the block."""
    a = np.asarray(a, dtype=F64).ravel()
    n = a.size
    blocks = -(-n // SCAN_BLOCK)
    groups = -(-blocks // SCAN_BLOCK)
    buf = np.zeros(groups * SCAN_BLOCK * SCAN_BLOCK, dtype=F64)
    buf[:n] = a
    inner = _block_scan(buf.reshape(groups, SCAN_BLOCK, SCAN_BLOCK))          # [g, b, i]
    block_scan = _block_scan(inner[..., -1])                                   # [g, b] inclusive over blocks
    blocks_before = np.concatenate([np.zeros((groups, 1)), block_scan[:, :-1]], axis=1)
    groups_before = np.zeros(groups, dtype=F64)
    acc = F64(0.0)
    for gi in range(groups):
        groups_before[gi] = acc
        acc = acc + block_scan[gi, -1]
    base = groups_before[:, None] + blocks_before
    return (base[..., None] + inner).reshape(-1)[:n]


def optimal_threshold(v):
    """Delta* = argmax_Delta (sum_{I_Delta} |v_i|)^2 / |I_Delta|, I_Delta = {i : |v_i| > Delta}
    (Section 3.4), by the paper's procedure: rank the |v_i| and try every component as the threshold.

    With a_0 >= a_1 >= ... the ranked magnitudes, the candidate sets are the k largest for every k
    with a_{k-1} > a_k (a strict drop: equal components fall on the same side of any threshold) and
    a_{k-1} > 0, plus k = d when a_{d-1} > 0.  The objective of k is F_k = (P_{k-1} * P_{k-1}) / k in
    fp64 with P the canonical prefix sums; the smallest k among equal maxima wins.  The threshold
    returned is the largest component outside the set, Delta* = a_k (0 when k = d or nothing is
    non-zero), so that Q_{Delta*} with its strict comparisons selects exactly those k.
    Returns (Delta* fp32, k int)."""
    a = np.sort(np.abs(np.asarray(v, dtype=F32).ravel()))[::-1]
    d = a.size
    prefix = canonical_prefix(a.astype(F64))
    objective = (prefix * prefix) / np.arange(1, d + 1, dtype=F64)
    drop = np.ones(d, dtype=bool)
    drop[:-1] = a[:-1] > a[1:]
    valid = drop & (a > 0)
    if not valid.any():
        return F32(0.0), 0
    i = int(np.argmax(np.where(valid, objective, -1.0)))     # first maximum
    return (a[i + 1] if i + 1 < d else F32(0.0)), i + 1


def quantize_at_threshold(v, delta):
    """Q_Delta(v) for a given fp32 Delta: codes by the strict fp32 comparisons of Section 3.4 and
    s*_Delta = mean of |v_i| over I_Delta (canonical sum).  Returns (tern, s fp32, |I_Delta|)."""
    v = np.asarray(v, dtype=F32).ravel()
    delta = F32(delta)
    pos = v > delta
    neg = v < -delta
    tern = pos.astype(np.int8) - neg.astype(np.int8)
    selected = pos | neg
    n = int(np.count_nonzero(selected))
    if n == 0:
        return tern, F32(0.0), 0
    picked = canonical_sum(np.where(selected, np.abs(v), F32(0.0)))
    return tern, F32(picked / F64(n)), n


def optimal_threshold_quantize(v):
    """Q_{Delta*}(v): the threshold quantizer at the exact optimal threshold.
    Returns (tern, s fp32, Delta* fp32, |I_{Delta*}|)."""
    delta, k = optimal_threshold(v)
    tern, scale, n = quantize_at_threshold(v, delta)
    assert n == k
    return tern, scale, delta, n


# ----------------------------------------------------------------------------------
# Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as
# 1, 2, 3", SC'11) and the stochastic ternary quantizer
# ----------------------------------------------------------------------------------
_PHILOX_M0 = np.uint64(0xD2511F53)
_PHILOX_M1 = np.uint64(0xCD9E8D57)
_PHILOX_W0 = 0x9E3779B9
_PHILOX_W1 = 0xBB67AE85
_MASK32 = np.uint64(0xFFFFFFFF)
_SH32 = np.uint64(32)


def philox4x32_10(c0, c1, c2, c3, k0, k1):
    """Ten rounds of Philox-4x32.  Counter words are arrays (broadcast together), key
    words are Python ints.  Returns four uint32 arrays."""
    c0, c1, c2, c3 = np.broadcast_arrays(
        *(np.asarray(c, dtype=np.uint64) & _MASK32 for c in (c0, c1, c2, c3)))
    k0 = int(k0) & 0xFFFFFFFF
    k1 = int(k1) & 0xFFFFFFFF
    for _ in range(10):
        p0 = _PHILOX_M0 * c0          # 32x32 -> 64-bit products
        p1 = _PHILOX_M1 * c2
        hi0, lo0 = p0 >> _SH32, p0 & _MASK32
        hi1, lo1 = p1 >> _SH32, p1 & _MASK32
        c0, c1, c2, c3 = (hi1 ^ c1 ^ np.uint64(k0), lo1,
                          hi0 ^ c3 ^ np.uint64(k1), lo0)
        k0 = (k0 + _PHILOX_W0) & 0xFFFFFFFF
        k1 = (k1 + _PHILOX_W1) & 0xFFFFFFFF
    return tuple(c.astype(np.uint32) for c in (c0, c1, c2, c3))


def philox_draws(seed, t, m, idx, domain=0):
    """The random word and uniform drawn for (seed, step t, worker m, coordinate idx).

    key     = (seed[31:0], seed[63:32])
    counter = (idx >> 2, m | domain << 16, t[31:0], t[63:32]); coordinate idx takes
              output word idx & 3.
    u       = (word >> 8) * 2**-24, exactly representable in fp32, in [0, 1).
    `t` and `idx` may be arrays (broadcast).  Returns (word uint32, u fp32).
    """
    idx = np.asarray(idx, dtype=np.uint64)
    t = np.asarray(t, dtype=np.uint64)
    seed = int(seed)
    words = philox4x32_10(idx >> np.uint64(2),
                          np.uint64((int(m) & 0xFFFF) | (int(domain) << 16)),
                          t & _MASK32, t >> _SH32,
                          seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF)
    lane = np.broadcast_to(idx & np.uint64(3), words[0].shape)
    word = np.choose(lane.astype(np.intp), words)
    u = (word >> np.uint32(8)).astype(F32) * F32(2.0 ** -24)
    return word, u


def ternary_stochastic_quantize(v, u, scale=None):
    """Unbiased ternary quantizer with the max-norm scaler (the comparison quantizer
    of Section 3.4 / related work: levels {-1, 0, 1} times a scaler).

    s = max_i |v_i|;  tern_i = sign(v_i) with probability |v_i| / s, else 0, realised
    as  u_i < |v_i| / s  with the fp32 division and the given uniforms u in [0, 1).
    Returns (tern int8[d], s fp32).  s = 0 gives all zeros.

    scale: when v is a slice of a longer vector, the scaler of that whole vector (its
    maximum magnitude, which the caller has taken); the slice's codes are then the
    corresponding slice of the whole vector's codes.
    """
    v = np.asarray(v, dtype=F32).ravel()
    u = np.asarray(u, dtype=F32).ravel()
    absv = np.abs(v)
    if scale is None:
        s = F32(absv.max()) if v.size else F32(0.0)
    else:
        s = F32(scale)
    if not s > 0:
        return np.zeros(v.size, dtype=np.int8), F32(0.0)
    prob = absv / s
    keep = u < prob
    tern = (np.sign(v).astype(np.int8)) * keep.astype(np.int8)
    return tern, s


# ----------------------------------------------------------------------------------
# Encoding (Section 3.5, "Encode": 2 bits per coordinate + one fp32 scale)
# ----------------------------------------------------------------------------------
def code_words(d):
    return -(-int(d) // 16)


def pack_codes(tern):
    """Ternary vector -> little-endian array of 32-bit words, 16 codes per word, the
    tail padded with code 0."""
    tern = np.asarray(tern).ravel()
    d = tern.size
    w = code_words(d)
    two_bit = np.zeros(w * 16, dtype=np.uint32)
    two_bit[:d] = np.where(tern > 0, 1, np.where(tern < 0, 2, 0))
    shifts = (2 * np.arange(16)).astype(np.uint32)
    return np.bitwise_or.reduce(two_bit.reshape(w, 16) << shifts, axis=1).astype(np.uint32)


def unpack_codes(words, d):
    """Inverse of `pack_codes` for the first d coordinates; code 3 decodes to 0."""
    words = np.asarray(words, dtype=np.uint32).ravel()
    shifts = (2 * np.arange(16)).astype(np.uint32)
    two_bit = ((words[:, None] >> shifts) & np.uint32(3)).ravel()[: int(d)]
    return (two_bit == 1).astype(np.int8) - (two_bit == 2).astype(np.int8)


def wire_bits(d):
    """Bits one worker sends for a dense model: 32 + 2d (Section 3.5, "Encode")."""
    return 32 + 2 * int(d)


# ----------------------------------------------------------------------------------
# Server side: decode and average (SynQ_t)
# ----------------------------------------------------------------------------------
def decode_average(terns, scales):
    """SynQ_t = (1/M) * sum_m s_m * tern_m, in fp64: the sum over workers in worker order,
    times the fp64 reciprocal of M (the product form in which the equation is written)."""
    terns = np.asarray(terns)
    scales = np.asarray(scales, dtype=F32)
    m_workers = terns.shape[0]
    acc = np.zeros(terns.shape[1], dtype=F64)
    for m in range(m_workers):
        acc = acc + F64(scales[m]) * terns[m].astype(F64)
    return acc * (F64(1.0) / F64(m_workers))


def requantize(gbar, quantizer, t=1, seed=0, coef=0.75, isyn=None):
    """Server side of Algorithm 1, "Quantize the aggregated gradient": q_t = Q(SynQ_t).

    The averaged gradient is held in fp32 (it is what would be sent), so gbar (fp64) is rounded
    to fp32 first and Q is applied to that vector exactly as it is applied to a worker's
    gradient.  The stochastic quantizer draws from the Philox stream of domain 1, worker 0.
    isyn (bool[d]) restricts Q to the coordinates of the synchronous indicator.
    Returns dict(tern int8[d], scale fp32, threshold fp32, count int, codes uint32[W], q fp64[d]).
    """
    gbar32 = np.asarray(gbar, dtype=F64).astype(F32)
    d = gbar32.size
    if quantizer == QUANT_THRESHOLD:
        if isyn is None:
            tern, scale, threshold, count = threshold_quantize(gbar32, coef)
        else:   # Q(S(SynQ_t, I^Syn)): only the coordinates some worker selected are quantized
            tern, scale, threshold, count, _ = threshold_quantize_selected(gbar32, isyn, coef)
    elif quantizer == QUANT_TERNARY_STOCH:
        _, u = philox_draws(seed, t, 0, np.arange(d, dtype=np.uint64), domain=1)
        tern, scale = ternary_stochastic_quantize(gbar32, u)     # the average is 0 outside I^Syn
        threshold, count = F32(0.0), int(np.count_nonzero(tern))
    else:
        raise ValueError("quantizer")
    return dict(tern=tern, scale=F32(scale), threshold=F32(threshold), count=int(count),
                codes=pack_codes(tern), q=F64(scale) * tern.astype(F64), gbar32=gbar32)


# ----------------------------------------------------------------------------------
# Worker side: accumulator H_t and the two closed-form updates
# ----------------------------------------------------------------------------------
def _scalars(lam, eta, delta):
    return F64(F32(lam)), F64(F32(eta)), F64(F32(delta))


def cmd_step(q, x, h, lam, eta, delta):
    """QCMD adagrad update (closed form of the composite-mirror-descent argmin).

    h <- h + q^2 (h holds c_t^2 = sum of squared quantized gradients, current one
    included);  H = delta + sqrt(h);  u = x - (eta/H) q;
    x <- sign(u) * [|u| - lambda*eta/H]_+ .
    Returns (x_new, h_new, a) with a = |u| * H / eta, the quantity the closed form
    compares with lambda (x_new == 0 exactly when a <= lambda).
    """
    lam, eta, delta = _scalars(lam, eta, delta)
    q = np.asarray(q, dtype=F64)
    x = np.asarray(x, dtype=F64)
    h = np.asarray(h, dtype=F64)
    h_new = h + q * q
    big_h = delta + np.sqrt(h_new)
    u = x - (eta / big_h) * q
    x_new = np.sign(u) * np.maximum(np.abs(u) - lam * eta / big_h, 0.0)
    x_new = x_new + 0.0                       # -0.0 -> +0.0
    return x_new, h_new, np.abs(u) * big_h / eta


def rda_step(q, h, z, t, lam, eta, delta):
    """QRDA adagrad update (closed form of the dual-averaging argmin).

    h <- h + q^2;  z <- z + q (z = sum of quantized gradients up to t);
    H = delta + sqrt(h);  x <- -sign(z) * (t*eta/H) * [|z|/t - lambda]_+ .
    Returns (x_new, h_new, z_new, a) with a = |z|/t, compared with lambda.
    """
    lam, eta, delta = _scalars(lam, eta, delta)
    q = np.asarray(q, dtype=F64)
    h = np.asarray(h, dtype=F64)
    z = np.asarray(z, dtype=F64)
    tt = F64(int(t))
    h_new = h + q * q
    z_new = z + q
    big_h = delta + np.sqrt(h_new)
    a = np.abs(z_new) / tt
    x_new = -np.sign(z_new) * (tt * eta / big_h) * np.maximum(a - lam, 0.0)
    x_new = x_new + 0.0
    return x_new, h_new, z_new, a


# ----------------------------------------------------------------------------------
# Sparse selection (Section 3.2: indicator I, selection S, "bitwise or" of the indicators)
# ----------------------------------------------------------------------------------
def trial_update(rule, g_m, x, h, z, t, lam, eta, delta):
    """Worker m's local trial iterate x_hat_{t+1}^(m) (Algorithm 1, "Compute the x_hat based on f'_t
    and H_hat_t"): the rule's closed-form update taken with the worker's own full-precision gradient
    and H_hat = delta + sqrt(h + g_m^2), h the accumulated squares of the quantized gradients so far.
    fp64; state is not modified."""
    if rule == RULE_CMD:
        return cmd_step(g_m, x, h, lam, eta, delta)[0]
    return rda_step(g_m, h, z, t, lam, eta, delta)[0]


def indicator(rule, g_m, x, h, z, t, lam, eta, delta):
    """I_d = 1 if x_{t,d} != 0 or x_hat_{t+1,d} != 0 (Eq. of the indicator function), decided in fp32,
    the precision of the data.  Where x_d != 0 the bit is set whatever the trial update gives, so
    the trial update matters only where x_d = 0, and there its closed form reduces to:

      QCMD:  x_hat = sign(-g) * (eta/H_hat) * [|g| - lambda]_+ , non-zero  <=>  |g| > lambda
             (H_hat = delta + sqrt(h + g^2) > 0 scales both sides of the test and drops out)
      QRDA:  x_hat != 0  <=>  |z + g| / t > lambda  <=>  |z + g| > lambda * t
             (one fp32 addition and one fp32 product, each rounded once)

    Returns a bool vector."""
    f = F32
    g_m = np.asarray(g_m, dtype=F32)
    x = np.asarray(x, dtype=F32)
    lam = f(lam)
    if rule == RULE_CMD:
        moved = np.abs(g_m) > lam
    else:
        z = np.asarray(z, dtype=F32)
        moved = np.abs(z + g_m) > lam * f(int(t))
    return (x != 0) | moved


def pack_bits(mask):
    """Bool vector -> uint32 words, bit i&31 of word i>>5, tail bits 0."""
    mask = np.asarray(mask, dtype=bool).ravel()
    w = -(-mask.size // 32)
    buf = np.zeros(w * 32, dtype=np.uint32)
    buf[: mask.size] = mask
    return np.bitwise_or.reduce(buf.reshape(w, 32) << np.arange(32, dtype=np.uint32), axis=1).astype(np.uint32)


def threshold_quantize_selected(v, selected, coef=0.75):
    """Q(S(v, I)): Q_Delta applied to the selected components only (k of them): the threshold is
    coef/k * sum_{I}|v_i|, unselected components are not sent and decode to 0.
    Returns (tern int8[d], s fp32, Delta fp32, |I_Delta| int, k int)."""
    v = np.asarray(v, dtype=F32).ravel()
    selected = np.asarray(selected, dtype=bool).ravel()
    k = int(np.count_nonzero(selected))
    absv = np.abs(v)
    if k == 0:
        return np.zeros(v.size, dtype=np.int8), F32(0.0), F32(0.0), 0, 0
    with np.errstate(invalid="ignore", over="ignore"):
        total = canonical_sum(np.where(selected, absv, F32(0.0)))
        delta = F32((F64(F32(coef)) * total) / F64(k))
        pos = selected & (v > delta)
        neg = selected & (v < -delta)
    tern = pos.astype(np.int8) - neg.astype(np.int8)
    kept = pos | neg
    n = int(np.count_nonzero(kept))
    if n == 0:
        return tern, F32(0.0), delta, 0, k
    picked = canonical_sum(np.where(kept, absv, F32(0.0)))
    return tern, F32(picked / F64(n)), delta, n, k


def ternary_stochastic_quantize_selected(v, u, selected):
    """The unbiased ternary quantizer on the selected components: s = max_{I}|v|."""
    v = np.asarray(v, dtype=F32).ravel()
    selected = np.asarray(selected, dtype=bool).ravel()
    masked = np.where(selected, v, F32(0.0))
    return ternary_stochastic_quantize(masked, u)


def sparse_wire_bits(d, k):
    """Bits one worker sends for a sparse model: 32 + d + 2k (Section 3.5, "Encode")."""
    return 32 + int(d) + 2 * int(k)


def select_quantize_workers(rule, g, x, h, z, t, lam, eta, delta, quantizer=QUANT_THRESHOLD, seed=0, coef=0.75):
    """Workers' side of Algorithm 1 with selection: indicator from the local trial update, then
    Q(S(g, I)).  Returns the dict of `quantize_workers` plus indicators bool[M,d], ind_words
    uint32[M, ceil(d/32)], selected int64[M] (k_m), isyn bool[d] (the "bitwise or")."""
    g = np.asarray(g, dtype=F32)
    m_workers, d = g.shape
    out = dict(terns=np.zeros((m_workers, d), np.int8), scales=np.zeros(m_workers, F32),
               thresholds=np.zeros(m_workers, F32), counts=np.zeros(m_workers, np.int64),
               selected=np.zeros(m_workers, np.int64), indicators=np.zeros((m_workers, d), bool))
    for m in range(m_workers):
        ind = indicator(rule, g[m], x, h, z, t, lam, eta, delta)
        out["indicators"][m] = ind
        if quantizer == QUANT_THRESHOLD:
            tern, s, thr, n, k = threshold_quantize_selected(g[m], ind, coef)
        else:
            _, u = philox_draws(seed, t, m, np.arange(d, dtype=np.uint64))
            tern, s = ternary_stochastic_quantize_selected(g[m], u, ind)
            thr, n, k = F32(0.0), int(np.count_nonzero(tern)), int(np.count_nonzero(ind))
        out["terns"][m], out["scales"][m], out["thresholds"][m] = tern, s, thr
        out["counts"][m], out["selected"][m] = n, k
    out["codes"] = np.stack([pack_codes(out["terns"][m]) for m in range(m_workers)])
    out["ind_words"] = np.stack([pack_bits(out["indicators"][m]) for m in range(m_workers)])
    out["isyn"] = out["indicators"].any(axis=0)
    return out


# ----------------------------------------------------------------------------------
# The whole step (one-way quantization: local gradients quantized, the average not)
# ----------------------------------------------------------------------------------


def quantize_workers(g, quantizer, t=1, seed=0, coef=0.75):
    """Quantize each worker's gradient row of g (M x d, fp32).

    Returns dict(terns int8[M,d], scales fp32[M], thresholds fp32[M], counts int64[M],
    codes uint32[M, W]).  For the stochastic quantizer thresholds are 0 and counts are
    the numbers of non-zero codes.
    """
    g = np.asarray(g, dtype=F32)
    m_workers, d = g.shape
    terns = np.zeros((m_workers, d), dtype=np.int8)
    scales = np.zeros(m_workers, dtype=F32)
    thresholds = np.zeros(m_workers, dtype=F32)
    counts = np.zeros(m_workers, dtype=np.int64)
    for m in range(m_workers):
        if quantizer == QUANT_THRESHOLD:
            terns[m], scales[m], thresholds[m], counts[m] = threshold_quantize(g[m], coef)
        elif quantizer == QUANT_TERNARY_STOCH:
            _, u = philox_draws(seed, t, m, np.arange(d, dtype=np.uint64))
            terns[m], scales[m] = ternary_stochastic_quantize(g[m], u)
            counts[m] = np.count_nonzero(terns[m])
        else:
            raise ValueError("quantizer")
    codes = np.stack([pack_codes(terns[m]) for m in range(m_workers)])
    return dict(terns=terns, scales=scales, thresholds=thresholds, counts=counts, codes=codes)


def densify_touched(g, touched):
    """A gradient held in sparse form: worker m stores only the entries its minibatch touched
    (touched[m, i] True); every other entry IS +0.0, whatever the array g holds there.  The
    quantizer and the update are those of the dense vector this returns (M x d, fp32): a zero
    entry is inside [-Delta, Delta] and codes 0 (Section 3.4), adds nothing to sum|g| nor to
    max|g|, and is kept with probability 0 by the stochastic quantizer."""
    g = np.asarray(g, dtype=F32)
    touched = np.asarray(touched, dtype=bool)
    if touched.shape != g.shape:
        raise ValueError("touched must have the shape of g")
    return np.where(touched, g, F32(0.0)).astype(F32)


def step(rule, g, x, h, z, t, lam, eta, delta, quantizer=QUANT_THRESHOLD, seed=0, coef=0.75,
         double_quant=False, select=False, touched=None):
    """One iteration: quantize every worker's gradient, decode and average, update the
    accumulator and apply the rule's closed-form update.  State in, state out (fp64).

    double_quant=True is Algorithm 1 as printed: the average is quantized again on the server
    (q_t = Q(SynQ_t)) and the workers update from q_t; False is the one-way variant.
    select=True adds the sparse selection: each worker sends only the coordinates its indicator
    marks (and, with double_quant, the server quantizes only those of the synchronous indicator).

    touched (bool M x d) marks the stored entries of sparse gradients: the step is that of
    `densify_touched(g, touched)`.

    quantizer == QUANT_NONE skips quantization: q is the fp64 mean of the rows of g
    (the 32-bit CMD / RDA adagrad baseline).
    Returns dict(x, h, z, a, q, quant) where `a` is the quantity compared with lambda
    and `quant` the output of `quantize_workers` (None without quantization).
    """
    g = np.asarray(g, dtype=F32)
    if touched is not None:
        g = densify_touched(g, touched)
    if quantizer == QUANT_NONE:
        quant = None
        q = g.astype(F64).sum(axis=0) / F64(g.shape[0])
    else:
        if select:
            quant = select_quantize_workers(rule, g, x, h, z, t, lam, eta, delta, quantizer, seed=seed, coef=coef)
        else:
            quant = quantize_workers(g, quantizer, t=t, seed=seed, coef=coef)
        q = decode_average(quant["terns"], quant["scales"])
    requant = None
    if double_quant:
        if quantizer == QUANT_NONE:
            raise ValueError("double quantization needs a quantizer")
        requant = requantize(q, quantizer, t=t, seed=seed, coef=coef, isyn=quant["isyn"] if select else None)
        q = requant["q"]
    if rule == RULE_CMD:
        x_new, h_new, a = cmd_step(q, x, h, lam, eta, delta)
        z_new = None if z is None else np.asarray(z, dtype=F64)
    elif rule == RULE_RDA:
        x_new, h_new, z_new, a = rda_step(q, h, z, t, lam, eta, delta)
    else:
        raise ValueError("rule")
    return dict(x=x_new, h=h_new, z=z_new, a=a, q=q, quant=quant, requant=requant)
