/*
 * LoCo oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, single-threaded CPU statement of what the LoCo hot path
 * computes (arXiv 2407.04480), written step by step in the paper's order and
 * notation.  Only the tests, the smoke check and the benchmark's CPU-baseline
 * leg may call it.  It shares no code, header, table or constant with the CUDA
 * library; the wire and state layouts are restated here from their written
 * definition.
 *
 * Arithmetic: IEEE binary32, one rounding per written operation (compile with
 * -ffp-contract=off -fno-fast-math), round-to-nearest-even everywhere, so that
 * integer results (codes, 8-bit error state, block scales) can be compared
 * bit for bit.  A double-precision twin of the same steps lives in
 * loco_definition.py and is used on tiny vectors to check the invariants.
 *
 * What follows the paper and where:
 *   compressor / decompressor ............ Eq. 1
 *   compensation h = g + dec(e; s_e) ...... Algorithm 1 step 1, Eq. 2
 *   low-bit gradient ..................... Algorithm 1 step 1, Eq. 3
 *   local dequantisation d ............... Algorithm 1 step 2
 *   moving-average error ................. Algorithm 1 step 2, Eq. 5
 *   reset / 8-bit error compression ...... Algorithm 1 step 2, Eq. 7
 *   average of the N dequantised parts ... Algorithm 1 step 3, Eq. 8
 *   Adam-family update with g~ ............ Algorithm 1 step 3, Adam-family equations (Sec. on LoCo-integrated Adam)
 *   partition of the vector into N parts . Sec. 3.3 (FSDP / all2all paragraph)
 *
 * Readings where the paper is silent (all restated in the design notes):
 *   - "nearest integer" ties go to even (the rounding of the PyTorch default
 *     the text of Eq. 1 points to);
 *   - the p-bit range is [-2^(p-1), 2^(p-1)-1] as the text under Eq. 1 says;
 *   - with an 8-bit stored error the previous high-precision error of Eq. 5 is
 *     its stored image dec(e_k; s_e) (STATE_INT8); the two fp32 variants keep
 *     e~ itself (STATE_FP32: compensate with e~;  STATE_FP32_Q8COMP:
 *     compensate with dec(comp(e~)), the form the proof of Lemma 1 uses);
 *   - reset test is the algorithm's literal "k % T_c == 0" on the caller's
 *     0-based k; T_c = 0 switches it off;
 *   - per-block absmax scaling (SCALE_BLOCK_ABSMAX) has no counterpart in the
 *     paper: it replaces the global s (and s_e) by per-block scales
 *     amax/qmax, and is defined here only so that both sides agree;
 *   - non-finite h: NaN gives code 0, +-Inf the saturated code, and in both
 *     cases the compression error of that element is taken as 0;
 *   - the element-wise clipping of g named in the experiments section has no stated threshold: `clip` is a
 *     parameter (0 = off), applied to g before step 1;
 *   - stochastic rounding (not in the paper, which rounds to nearest): floor(h x s + u) with u from a
 *     Philox4x32-10 stream keyed by a seed and indexed by (element, iteration), so that it can be reproduced anywhere;
 *   - 1-bit LoCo (the paper names it in the GPT-2 experiment and never defines it; Eq. 1 with p = 1 would give the
 *     range {-1, 0}): bits = 1 sends the sign, q = -1 if h < 0 else +1 (so +-0 and NaN give +1), one wire bit per
 *     element (1 = negative), and d = q / s with the global scale, or d = q x (mean |h| of the block) with block
 *     scales -- the magnitude that minimises the squared error of a sign code; that mean is taken in fp32 by
 *     pairwise (balanced binary tree) summation over the block's B positions, absent and non-finite elements
 *     entering as 0, divided by the number of elements of the block that exist.  Steps 2 (Eq. 5, Eq. 7) unchanged;
 *   - Eq. 8 is summed in worker order in fp32, then divided by (float)N;
 *   - the Adam-family step is taken exactly as printed (no bias correction, delta inside the root), with
 *     eta_k = eta / sqrt(v_k + delta) evaluated as one square root and one division.
 *
 * Pins (tests/test_oracle_pins.py): code range, half-step bound and saturation
 * error of Lemma "round", brute-force nearest code, idempotence, identity
 * compression => zero error, beta = 1 => classic error feedback, closed-form
 * unrolling of Eq. 5, the identity of Lemma 1 in its three storage forms, the
 * telescoping sum of Lemma 2's proof, reset, averaging versus the real-number
 * mean, storage sizes of Table 1's text, brute force over all byte values of
 * the packing, and a hand-worked example (tests/golden/); for the fused Adam-family step: the sign-update special
 * case (beta1 = beta2 = 1, delta = 0), the closed form of the moments under a constant gradient, a zero gradient,
 * agreement with the textbook formulas in float64, and a hand-worked dyadic example.
 * The block-scaled 8-bit state (scale rule amax/127, largest code 127, half-step bound, reset, Lemma 1's identity in
 * its 8-bit form) and the bf16 conversions (against an independent conversion, ties, NaN, Inf, denormals) have
 * pins of their own; the 1-bit compressor is pinned by its optimality on brute-forced blocks, the order of its
 * pairwise sum on a hand-worked block, Lemma 1's identity and the packing of all 256 bytes.
 * Unpinned by anything in the paper: the value of beta, the block size, the
 * block-scaled variant as a whole and the 1-bit compressor ("parity unpinned" for SCALE_BLOCK_ABSMAX and
 * for bits = 1: they are pinned only by what the mathematics fixes once the reading is chosen).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { ORC_F32 = 0, ORC_BF16 = 1 };
enum { ORC_SCALE_FIXED = 0, ORC_SCALE_BLOCK_ABSMAX = 1 };
enum { ORC_STATE_INT8 = 0, ORC_STATE_FP32 = 1, ORC_STATE_NONE = 2, ORC_STATE_FP32_Q8COMP = 3 };
enum { ORC_FLAG_NONFINITE = 1u };

/* Algorithm 1's inputs (s, s_e, T_c, beta) plus the storage choices. */
typedef struct {
    int32_t bits;           /* p of Eq. 1 for the gradient codes: 2, 4 or 8; 1 = sign code (1-bit LoCo) */
    int32_t scale_mode;     /* ORC_SCALE_* */
    int32_t block_size;     /* B, BLOCK_ABSMAX only */
    float   s;              /* Eq. 1 / Eq. 3 */
    float   s_e;            /* Eq. 2 / Eq. 7 */
    float   beta;           /* Eq. 5: weight of the NEW compression error */
    int32_t reset_period;   /* T_c of Eq. 7; 0 = never */
    int32_t state_fmt;      /* ORC_STATE_* */
    int32_t grad_dtype;     /* ORC_F32 / ORC_BF16 */
    int32_t out_dtype;      /* ORC_F32 / ORC_BF16 */
    int32_t num_partitions; /* N parts of Sec. 3.3 */
    float   clip;           /* > 0: element-wise clipping of the local gradient to [-clip, clip] before Algorithm 1
                               (the Sky-MoE pre-training runs of the experiments section); 0 = off */
    int32_t rounding;       /* 0: nearest integer, Eq. 1 (the paper);  1: stochastic rounding (extension) */
    uint32_t seed_lo, seed_hi;  /* key of the Philox stream used by stochastic rounding */
} orc_config;

/* ---------- Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3", SC'11) ----------
 * Counter-based generator: out = philox(counter[4], key[2]); ten rounds of two 32x32->64 multiplications by fixed
 * constants, xors with the key, and a Weyl bump of the key between rounds.  Written from the published definition;
 * the tests check the published known-answer vectors. */
void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3], k0 = key[0], k1 = key[1];
    for (int r = 0; r < 10; ++r) {
        if (r > 0) { k0 += W0; k1 += W1; }
        const uint64_t p0 = (uint64_t)M0 * c0, p1 = (uint64_t)M1 * c2;
        const uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0, hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
        const uint32_t n0 = hi1 ^ c1 ^ k0, n1 = lo1, n2 = hi0 ^ c3 ^ k1, n3 = lo0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* The number in (0, 1) that stochastic rounding adds to element i of the bucket at iteration k: one byte of the 16 that
 * philox(counter = (i/16 low, i/16 high, k low, k high), key = seed) returns -- byte (i mod 4) of word ((i mod 16) / 4),
 * least significant byte first -- taken as (byte + 1/2) / 256: 256 equally likely values, each in the middle of its
 * cell, so that the probability of rounding up equals frac(y) to within 1/512. */
static float sr_uniform(const orc_config *c, uint64_t i, int64_t k) {
    const uint64_t blk = i >> 4;
    const uint32_t ctr[4] = {(uint32_t)blk, (uint32_t)(blk >> 32), (uint32_t)(uint64_t)k, (uint32_t)((uint64_t)k >> 32)};
    const uint32_t key[2] = {c->seed_lo, c->seed_hi};
    uint32_t out[4];
    orc_philox4x32_10(ctr, key, out);
    const uint32_t byte = (out[(i >> 2) & 3] >> (8 * (unsigned)(i & 3))) & 0xFFu;
    return ((float)byte + 0.5f) * 0.00390625f;                     /* (byte + 1/2) / 256, exact */
}
float orc_sr_uniform(const orc_config *c, uint64_t i, int64_t k) { return sr_uniform(c, i, k); }

/* Optional per-element record of one send step, for the invariant tests. */
typedef struct {
    float   *c;      /* dec(e_k) (or e~_k for STATE_FP32): what was added to g */
    float   *h;      /* compensated gradient                                   */
    int32_t *q;      /* low-bit code                                           */
    float   *d;      /* locally dequantised code                               */
    float   *delta;  /* h - d                                                  */
    float   *e_new;  /* e~_{k+1} before any 8-bit compression or reset         */
} orc_trace;

/* ---------- bf16 <-> fp32 (bit definitions of the format) ---------- */
static float bf16_to_f32(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}
static uint16_t f32_to_bf16_rne(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x0040u); /* quiet NaN */
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7fffu + lsb;
    return (uint16_t)(u >> 16);
}
uint16_t orc_f32_to_bf16(float f) { return f32_to_bf16_rne(f); }
float orc_bf16_to_f32(uint16_t b) { return bf16_to_f32(b); }
void orc_f32_to_bf16_array(const float *f, uint64_t n, uint16_t *b) { for (uint64_t i = 0; i < n; ++i) b[i] = f32_to_bf16_rne(f[i]); }
void orc_bf16_to_f32_array(const uint16_t *b, uint64_t n, float *f) { for (uint64_t i = 0; i < n; ++i) f[i] = bf16_to_f32(b[i]); }

/* ---------- Eq. 1 ---------- */
static int32_t qmin_of(int p) { return -(1 << (p - 1)); }
static int32_t qmax_of(int p) { return (1 << (p - 1)) - 1; }

/* round_p-bit(y): nearest integer (ties to even), then the p-bit range. y is finite or +-Inf. */
static int32_t round_pbit(float y, int p) {
    float r = rintf(y);
    float lo = (float)qmin_of(p), hi = (float)qmax_of(p);
    if (r < lo) r = lo;
    if (r > hi) r = hi;
    return (int32_t)r;
}

/* compressor(h; s, p) = round_p-bit(h x s), elementwise. */
void orc_compressor(const float *h, uint64_t n, float s, int32_t p, int32_t *q) {
    for (uint64_t i = 0; i < n; ++i) q[i] = round_pbit(h[i] * s, p);
}
/* decompressor(q; s) = float(q) / s, elementwise. */
void orc_decompressor(const int32_t *q, uint64_t n, float s, float *out) {
    for (uint64_t i = 0; i < n; ++i) out[i] = (float)q[i] / s;
}

/* ---------- layouts (written definition, restated) ---------- */
static uint64_t round_up(uint64_t x, uint64_t m) { return (x + m - 1) / m * m; }

static int config_ok(const orc_config *c) {
    if (!c) return 0;
    if (c->bits != 1 && c->bits != 2 && c->bits != 4 && c->bits != 8) return 0;
    if (c->scale_mode != ORC_SCALE_FIXED && c->scale_mode != ORC_SCALE_BLOCK_ABSMAX) return 0;
    if (c->scale_mode == ORC_SCALE_BLOCK_ABSMAX) {
        int b = c->block_size;
        if (b < 32 || b > 4096 || (b & (b - 1))) return 0;
        if (c->state_fmt == ORC_STATE_FP32_Q8COMP) return 0;
    } else {
        if (!(c->s > 0.0f) || !isfinite(c->s)) return 0;
        if (c->state_fmt == ORC_STATE_INT8 || c->state_fmt == ORC_STATE_FP32_Q8COMP)
            if (!(c->s_e > 0.0f) || !isfinite(c->s_e)) return 0;
    }
    if (c->state_fmt < 0 || c->state_fmt > 3) return 0;
    if (c->state_fmt != ORC_STATE_NONE && !(c->beta >= 0.0f && c->beta <= 1.0f)) return 0;
    if (c->reset_period < 0) return 0;
    if (c->grad_dtype != ORC_F32 && c->grad_dtype != ORC_BF16) return 0;
    if (c->out_dtype != ORC_F32 && c->out_dtype != ORC_BF16) return 0;
    if (c->num_partitions < 1) return 0;
    if (!(c->clip >= 0.0f) || !isfinite(c->clip)) return 0;
    if (c->rounding != 0 && c->rounding != 1) return 0;
    if (c->bits == 1 && c->rounding != 0) return 0;       /* a sign code has nothing to round */
    return 1;
}

/* Length unit of a partition: 256 elements, or the block if that is larger. */
static uint64_t part_unit(const orc_config *c) {
    uint64_t u = 256;
    if (c->scale_mode == ORC_SCALE_BLOCK_ABSMAX && (uint64_t)c->block_size > u) u = (uint64_t)c->block_size;
    return u;
}
/* Lp: padded elements per partition. */
uint64_t orc_partition_capacity(const orc_config *c, uint64_t n) {
    if (!config_ok(c) || n == 0) return 0;
    uint64_t per = (n + (uint64_t)c->num_partitions - 1) / (uint64_t)c->num_partitions;
    return round_up(per, part_unit(c));
}
/* Valid (unpadded) elements of partition j. */
uint64_t orc_partition_elems(const orc_config *c, uint64_t n, int32_t j) {
    uint64_t lp = orc_partition_capacity(c, n);
    if (lp == 0 || j < 0 || j >= c->num_partitions) return 0;
    uint64_t lo = (uint64_t)j * lp;
    if (lo >= n) return 0;
    uint64_t hi = lo + lp;
    if (hi > n) hi = n;
    return hi - lo;
}
static uint64_t code_bytes_of(const orc_config *c, uint64_t lp) { return lp * (uint64_t)c->bits / 8; }
static uint64_t scale_bytes_of(const orc_config *c, uint64_t lp) {
    return c->scale_mode == ORC_SCALE_BLOCK_ABSMAX ? (lp / (uint64_t)c->block_size) * 4 : 0;
}
/* Stride of one partition in the communication buffer. */
uint64_t orc_partition_bytes(const orc_config *c, uint64_t n) {
    uint64_t lp = orc_partition_capacity(c, n);
    if (lp == 0) return 0;
    return round_up(code_bytes_of(c, lp) + scale_bytes_of(c, lp), 128);
}
uint64_t orc_packed_bytes(const orc_config *c, uint64_t n) {
    return orc_partition_bytes(c, n) * (uint64_t)(config_ok(c) ? c->num_partitions : 0);
}
/* Error state: 1 byte per element for the paper's 8-bit format (Table 1's text), 4 for fp32. */
uint64_t orc_state_bytes(const orc_config *c, uint64_t n) {
    if (!config_ok(c) || n == 0) return 0;
    switch (c->state_fmt) {
    case ORC_STATE_NONE: return 0;
    case ORC_STATE_INT8: {
        uint64_t b = round_up(n, 256);
        if (c->scale_mode == ORC_SCALE_BLOCK_ABSMAX)
            b += round_up(((n + (uint64_t)c->block_size - 1) / (uint64_t)c->block_size) * 4, 256);
        return b;
    }
    default: return round_up(n * 4, 256);
    }
}

/* Write the p-bit two's-complement field of element `o` of a partition's code area. */
static void put_code(uint8_t *codes, uint64_t o, int p, int32_t q) {
    if (p == 1) q = q < 0 ? 1 : 0;           /* sign code: the wire bit is 1 for -1, 0 for +1 */
    int per = 8 / p;
    uint64_t byte = o / (uint64_t)per;
    int shift = (int)(o % (uint64_t)per) * p;
    uint8_t mask = (uint8_t)(((1u << p) - 1u) << shift);
    uint8_t field = (uint8_t)((((uint32_t)q) & ((1u << p) - 1u)) << shift);
    codes[byte] = (uint8_t)((codes[byte] & (uint8_t)~mask) | field);
}
static int32_t get_code(const uint8_t *codes, uint64_t o, int p) {
    int per = 8 / p;
    uint64_t byte = o / (uint64_t)per;
    int shift = (int)(o % (uint64_t)per) * p;
    int32_t v = (int32_t)((codes[byte] >> shift) & ((1u << p) - 1u));
    if (p == 1) return v ? -1 : 1;            /* sign code */
    if (v >= (1 << (p - 1))) v -= (1 << p);
    return v;
}
/* Exposed for the brute-force packing tests. */
void orc_pack_codes(const int32_t *q, uint64_t n, int32_t p, uint8_t *bytes /* zeroed by caller */) {
    for (uint64_t i = 0; i < n; ++i) put_code(bytes, i, p, q[i]);
}
void orc_unpack_codes(const uint8_t *bytes, uint64_t n, int32_t p, int32_t *q) {
    for (uint64_t i = 0; i < n; ++i) q[i] = get_code(bytes, i, p);
}

static float load_grad(const orc_config *c, const void *grad, uint64_t i) {
    float g = c->grad_dtype == ORC_BF16 ? bf16_to_f32(((const uint16_t *)grad)[i]) : ((const float *)grad)[i];
    /* element-wise clipping of g (experiments section); a NaN stays a NaN, +-Inf becomes +-clip */
    if (c->clip > 0.0f && !isnan(g)) {
        if (g > c->clip) g = c->clip;
        if (g < -c->clip) g = -c->clip;
    }
    return g;
}

/* Quantise one compensated value against a multiplier (s, or the block's inverse scale).
 * Returns the code; *err0 is set when the element's compression error is defined as 0. */
static int32_t quantise(const orc_config *c, uint64_t i, int64_t k, float h, float mult, int p, int *err0, uint64_t *status) {
    *err0 = 0;
    if (p == 1) {
        /* 1-bit LoCo: the sign, q in {+1, -1}; the compression error of a non-finite element is taken as 0 */
        if (isnan(h) || isinf(h)) { *err0 = 1; status[0] |= ORC_FLAG_NONFINITE; }
        return h < 0.0f ? -1 : 1;
    }
    if (isnan(h)) { *err0 = 1; status[0] |= ORC_FLAG_NONFINITE; return 0; }
    if (isinf(h)) { *err0 = 1; status[0] |= ORC_FLAG_NONFINITE; return h > 0 ? qmax_of(p) : qmin_of(p); }
    float y = h * mult;                       /* h x s of Eq. 1 */
    if (c->rounding == 1) {
        /* stochastic rounding (extension): floor(y + u), u uniform over 256 values in (0, 1): up with probability frac(y) */
        const float t = y + sr_uniform(c, i, k);
        float r = floorf(t);
        const float lo = (float)qmin_of(p), hi = (float)qmax_of(p);
        if (r < lo || r > hi) status[1] += 1;
        if (r < lo) r = lo;
        if (r > hi) r = hi;
        return (int32_t)r;
    }
    float r = rintf(y);
    /* saturated: the nearest integer falls outside the p-bit range (second case of Lemma "round") */
    if (r < (float)qmin_of(p) || r > (float)qmax_of(p)) status[1] += 1;
    int32_t q = round_pbit(y, p);
    return q;
}

/* Pairwise summation in fp32: the sum of a[0..len) is the sum of its first half plus the sum of its second half,
 * len a power of two. */
static float pairwise_sum(const float *a, uint64_t len) {
    if (len == 1) return a[0];
    return pairwise_sum(a, len / 2) + pairwise_sum(a + len / 2, len / 2);
}
float orc_pairwise_sum(const float *a, uint64_t len) { return pairwise_sum(a, len); }

/*
 * One LoCo send step for one worker and one bucket (Algorithm 1, steps 1 and 2),
 * followed by packing the codes into the partitioned communication buffer.
 *
 *   grad   n elements (fp32 or bf16), read only
 *   state  the worker's error state, updated in place
 *   comm   communication buffer of orc_packed_bytes(); code and scale areas are
 *          fully written, bytes past them inside a stride are left alone
 *   k      the paper's 0-based iteration counter
 *   status [0] flag bits (or-ed in), [1] count of saturated gradient codes (added to), [2] count of saturated
 *          8-bit error codes (added to): elements whose e~ x s_e has its nearest integer outside [-128, 127], the
 *          clamp of Eq. 7 (global s_e only; a block-scaled state cannot saturate)
 * Returns 0, or -1 on a bad configuration.
 */
int orc_send_step(const orc_config *cfg, uint64_t n, const void *grad, void *state,
                  uint8_t *comm, int64_t k, orc_trace *tr, uint64_t *status) {
    if (!config_ok(cfg) || k < 0) return -1;
    if (n == 0) return 0;
    const int p = cfg->bits;
    const int fixed = cfg->scale_mode == ORC_SCALE_FIXED;
    const int fmt = cfg->state_fmt;
    const uint64_t B = fixed ? 1 : (uint64_t)cfg->block_size;
    const uint64_t lp = orc_partition_capacity(cfg, n);
    const uint64_t stride = orc_partition_bytes(cfg, n);
    const uint64_t cbytes = code_bytes_of(cfg, lp);
    const float beta = cfg->beta;
    const float omb = 1.0f - beta;            /* (1 - beta) of Eq. 5, rounded once */
    const int reset = cfg->reset_period > 0 && (k % (int64_t)cfg->reset_period) == 0;   /* Eq. 7 */
    uint64_t st_local[3] = {0, 0, 0};
    if (!status) status = st_local;

    int8_t *e8 = (int8_t *)state;                              /* STATE_INT8 codes */
    float *e8_scale = fixed ? NULL : (float *)((uint8_t *)state + round_up(n, 256));
    float *ef = (float *)state;                                /* fp32 formats */

    /* zero the code areas so that padding elements carry code 0 */
    for (int32_t j = 0; j < cfg->num_partitions; ++j) {
        memset(comm + (uint64_t)j * stride, 0, cbytes);
        if (!fixed) memset(comm + (uint64_t)j * stride + cbytes, 0, scale_bytes_of(cfg, lp));
    }

    float *hb = (float *)malloc(sizeof(float) * B);
    float *cb = (float *)malloc(sizeof(float) * B);
    float *pb = (float *)malloc(sizeof(float) * B);
    float *nb = (float *)malloc(sizeof(float) * B);
    float *ab = (float *)malloc(sizeof(float) * B);
    if (!hb || !cb || !pb || !nb || !ab) { free(hb); free(cb); free(pb); free(nb); free(ab); return -1; }

    for (uint64_t b0 = 0; b0 < n; b0 += B) {
        const uint64_t len = (b0 + B <= n) ? B : n - b0;
        const uint64_t blk = b0 / B;

        /* Step 1: h = g + decompressor(e_k; s_e) */
        for (uint64_t t = 0; t < len; ++t) {
            const uint64_t i = b0 + t;
            float c, prev;
            switch (fmt) {
            case ORC_STATE_INT8:
                c = fixed ? (float)e8[i] / cfg->s_e : (float)e8[i] * e8_scale[blk];
                prev = c;
                break;
            case ORC_STATE_FP32:
                c = ef[i];
                prev = c;
                break;
            case ORC_STATE_FP32_Q8COMP:
                prev = ef[i];
                {
                    const float ye = prev * cfg->s_e, re = rintf(ye);
                    if (re < -128.0f || re > 127.0f) status[2] += 1;
                    c = (float)round_pbit(ye, 8) / cfg->s_e;
                }
                break;
            default:
                c = 0.0f;
                prev = 0.0f;
            }
            cb[t] = c;
            pb[t] = prev;
            hb[t] = load_grad(cfg, grad, i) + c;
        }

        /* scale of the block (extension); the paper's s otherwise */
        float mult = cfg->s, scale = 0.0f;
        if (!fixed && p == 1) {
            /* sign code: the block's magnitude is the mean of |h| (pairwise sum over the B positions / elements that exist) */
            for (uint64_t t = 0; t < B; ++t) ab[t] = (t < len && isfinite(hb[t])) ? fabsf(hb[t]) : 0.0f;
            scale = pairwise_sum(ab, B) / (float)len;
            mult = 0.0f;
        } else if (!fixed) {
            float amax = 0.0f;
            for (uint64_t t = 0; t < len; ++t)
                if (isfinite(hb[t]) && fabsf(hb[t]) > amax) amax = fabsf(hb[t]);
            const float qm = (float)qmax_of(p);
            scale = amax > 0.0f ? amax / qm : 0.0f;
            mult = amax > 0.0f ? qm / amax : 0.0f;
        }

        /* Step 1: code;  Step 2: d, delta, moving average */
        for (uint64_t t = 0; t < len; ++t) {
            const uint64_t i = b0 + t;
            int err0;
            const int32_t q = quantise(cfg, i, k, hb[t], mult, p, &err0, status);
            const float d = fixed ? (float)q / cfg->s : (float)q * scale;
            const float delta = err0 ? 0.0f : hb[t] - d;
            const float e_new = (omb * pb[t]) + (beta * delta);      /* Eq. 5 */
            nb[t] = e_new;
            const uint64_t j = i / lp, o = i % lp;
            put_code(comm + j * stride, o, p, q);
            if (tr) {
                if (tr->c) tr->c[i] = cb[t];
                if (tr->h) tr->h[i] = hb[t];
                if (tr->q) tr->q[i] = q;
                if (tr->d) tr->d[i] = d;
                if (tr->delta) tr->delta[i] = delta;
                if (tr->e_new) tr->e_new[i] = e_new;
            }
        }
        if (!fixed) {
            const uint64_t j = b0 / lp, o = b0 % lp;
            memcpy(comm + j * stride + cbytes + (o / B) * 4, &scale, 4);
        }

        /* Step 2: reset, or keep / compress the new error (Eq. 7) */
        if (fmt == ORC_STATE_NONE) continue;
        if (reset) {
            for (uint64_t t = 0; t < len; ++t) {
                if (fmt == ORC_STATE_INT8) e8[b0 + t] = 0; else ef[b0 + t] = 0.0f;
            }
            if (fmt == ORC_STATE_INT8 && !fixed) e8_scale[blk] = 0.0f;
        } else if (fmt == ORC_STATE_INT8) {
            float emult = cfg->s_e, escale = 0.0f;
            if (!fixed) {
                float amax = 0.0f;
                for (uint64_t t = 0; t < len; ++t)
                    if (fabsf(nb[t]) > amax) amax = fabsf(nb[t]);
                escale = amax > 0.0f ? amax / 127.0f : 0.0f;
                emult = amax > 0.0f ? 127.0f / amax : 0.0f;
                e8_scale[blk] = escale;
            }
            for (uint64_t t = 0; t < len; ++t) {
                const float ye = nb[t] * emult, re = rintf(ye);
                if (fixed && (re < -128.0f || re > 127.0f)) status[2] += 1;     /* the clamp of Eq. 7 acts */
                e8[b0 + t] = (int8_t)round_pbit(ye, 8);                          /* compressor(e~; s_e, 8) */
            }
        } else {
            for (uint64_t t = 0; t < len; ++t) ef[b0 + t] = nb[t];
        }
    }
    free(hb); free(cb); free(pb); free(nb); free(ab);
    return 0;
}

/*
 * Receive side (Algorithm 1 step 3, Eq. 8) for `count` consecutive partitions
 * starting at `first`: parts[w] points at partition `first` inside worker w's
 * communication buffer (the following partitions sit one stride further each).
 * out receives the valid elements of those partitions, contiguously.
 */
int orc_reduce(const orc_config *cfg, uint64_t n, const uint8_t *const *parts, int32_t num_workers,
               int32_t first, int32_t count, void *out) {
    if (!config_ok(cfg) || num_workers < 1 || first < 0 || count < 0 ||
        first + count > cfg->num_partitions) return -1;
    if (n == 0 || count == 0) return 0;
    const int p = cfg->bits;
    const int fixed = cfg->scale_mode == ORC_SCALE_FIXED;
    const uint64_t lp = orc_partition_capacity(cfg, n);
    const uint64_t stride = orc_partition_bytes(cfg, n);
    const uint64_t cbytes = code_bytes_of(cfg, lp);
    const uint64_t B = fixed ? 1 : (uint64_t)cfg->block_size;
    uint64_t w_out = 0;
    for (int32_t j = first; j < first + count; ++j) {
        const uint64_t valid = orc_partition_elems(cfg, n, j);
        const uint64_t off = (uint64_t)(j - first) * stride;
        for (uint64_t o = 0; o < valid; ++o) {
            float acc = 0.0f;
            for (int32_t w = 0; w < num_workers; ++w) {
                const uint8_t *base = parts[w] + off;
                const int32_t q = get_code(base, o, p);
                float d;
                if (fixed) {
                    d = (float)q / cfg->s;                               /* decompressor, Eq. 1 */
                } else {
                    float sc;
                    memcpy(&sc, base + cbytes + (o / B) * 4, 4);
                    d = (float)q * sc;
                }
                acc = acc + d;
            }
            const float g = acc / (float)num_workers;                      /* the 1/N of Eq. 8 */
            if (cfg->out_dtype == ORC_BF16) ((uint16_t *)out)[w_out] = f32_to_bf16_rne(g);
            else ((float *)out)[w_out] = g;
            ++w_out;
        }
    }
    return 0;
}

/*
 * Receive side followed by the Adam-family update of the same elements (Algorithm 1 step 3: "use g~_k to update
 * theta_k"; the Adam-family equations of the section on LoCo-integrated Adam-family optimizers):
 *     g      = (1/N) sum_n dec(q^n)                       Eq. 8, in fp32, NOT rounded to the output type first
 *     m_k    = (1 - beta1) m_{k-1} + beta1 g              (beta1 weights the new gradient, as the paper writes it)
 *     v_k    = (1 - beta2) v_{k-1} + beta2 g^2
 *     eta_k  = eta / sqrt(v_k + delta)                    Adam's pre-conditioner v(.) = 1/sqrt(v_k + delta)
 *     theta  = theta - eta_k * m_k
 * There is no bias correction and delta sits inside the square root: that is what the paper prints.
 * Every operation is one IEEE fp32 operation; (1 - beta) is rounded once.  m, v, theta hold the valid elements of
 * the `count` partitions contiguously and are updated in place; grad_out (may be NULL) receives g in out_dtype.
 */
typedef struct { float lr, beta1, beta2, delta; } orc_adam;

int orc_reduce_adam(const orc_config *cfg, uint64_t n, const uint8_t *const *parts, int32_t num_workers,
                    int32_t first, int32_t count, const orc_adam *ad, float *m, float *v, float *theta,
                    void *grad_out) {
    if (!config_ok(cfg) || !ad || num_workers < 1 || first < 0 || count < 0 ||
        first + count > cfg->num_partitions) return -1;
    if (n == 0 || count == 0) return 0;
    const int p = cfg->bits;
    const int fixed = cfg->scale_mode == ORC_SCALE_FIXED;
    const uint64_t lp = orc_partition_capacity(cfg, n);
    const uint64_t stride = orc_partition_bytes(cfg, n);
    const uint64_t cbytes = code_bytes_of(cfg, lp);
    const uint64_t B = fixed ? 1 : (uint64_t)cfg->block_size;
    const float omb1 = 1.0f - ad->beta1, omb2 = 1.0f - ad->beta2;
    uint64_t w_out = 0;
    for (int32_t j = first; j < first + count; ++j) {
        const uint64_t valid = orc_partition_elems(cfg, n, j);
        const uint64_t off = (uint64_t)(j - first) * stride;
        for (uint64_t o = 0; o < valid; ++o) {
            float acc = 0.0f;
            for (int32_t w = 0; w < num_workers; ++w) {
                const uint8_t *base = parts[w] + off;
                const int32_t q = get_code(base, o, p);
                float d;
                if (fixed) {
                    d = (float)q / cfg->s;
                } else {
                    float sc;
                    memcpy(&sc, base + cbytes + (o / B) * 4, 4);
                    d = (float)q * sc;
                }
                acc = acc + d;
            }
            const float g = acc / (float)num_workers;                       /* Eq. 8 */
            const float mk = (omb1 * m[w_out]) + (ad->beta1 * g);
            const float gg = g * g;
            const float vk = (omb2 * v[w_out]) + (ad->beta2 * gg);
            const float den = sqrtf(vk + ad->delta);
            const float eta_k = ad->lr / den;
            const float upd = eta_k * mk;
            m[w_out] = mk;
            v[w_out] = vk;
            theta[w_out] = theta[w_out] - upd;
            if (grad_out) {
                if (cfg->out_dtype == ORC_BF16) ((uint16_t *)grad_out)[w_out] = f32_to_bf16_rne(g);
                else ((float *)grad_out)[w_out] = g;
            }
            ++w_out;
        }
    }
    return 0;
}
