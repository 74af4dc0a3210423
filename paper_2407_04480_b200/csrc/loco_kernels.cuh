// LoCo send / receive kernels for sm_100a.
//
// Both passes are elementwise streams over HBM (no contraction, no tensor cores).  At HBM speed the
// send pass has about 25 issue slots per element, and the logic / min-max / convert instructions
// share one pipe that accepts a warp instruction only every second clock, so the instruction mix is
// part of the design:
//   * integers enter and leave fp32 through the mantissa of a "magic" float (1.5 * 2^23 + k) instead of
//     through I2F / F2I, except for the 8-bit error codes, which use the one F2I per element that the
//     slow conversion pipe can absorb followed by a saturating two-at-a-time byte pack;
//   * the division of Eq. 1's decompressor is replaced by one fused multiply-add, or by a three-step
//     Newton-Raphson sequence, only after the host has checked that the replacement reproduces the IEEE
//     division bit for bit on every code it can meet; otherwise the division is kept;
//   * codes are packed by a Horner chain of integer multiply-adds (they run on the fp32 pipe);
//   * non-finite inputs are detected with one fused multiply-add per element (h * 0 accumulates NaN)
//     and the rare rows that contain one are redone by a plain, careful routine.
//   * the fp32 steps of the send pass run two elements at a time on the packed fp32x2 instructions, which
//     halves their issue slots; the inputs of a warp's next rows travel through a cp.async ring in shared
//     memory, so the bytes in flight do not depend on registers or on the phase the warp is in.
// Work unit of the send pass: a "wide row" of 512 consecutive elements handled by one warp, 16 consecutive
// elements per lane; of the receive pass and of the careful routine: a row of 256 elements, 8 per lane.
// Every warp-wide access covers one contiguous span.
//
// Rounding discipline: every floating-point step of Algorithm 1 is one IEEE fp32 operation rounded to
// nearest even, written with intrinsics, so that nothing is contracted into an FMA by the compiler; an
// FMA is used only where it is proven (on the host, exhaustively) to give the same bits.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace loco {

enum : int { GRAD_F32 = 0, GRAD_BF16 = 1 };
enum : int { ST_INT8 = 0, ST_FP32 = 1, ST_NONE = 2, ST_Q8COMP = 3 };
enum : int { MODE_FIXED = 0, MODE_BLOCK = 1 };
// How dec(code; scale) = code / scale is evaluated on the fast path.
enum : int { DEC_FMA = 0,      // one fused multiply-add on the magic-biased code
             DEC_NEWTON = 1,   // q0 = c * r; rem = fma(-q0, scale, c); q0 + rem * r
             DEC_DIVIDE = 2 }; // neither was proven: every row takes the careful routine (IEEE division)

constexpr int kRow = 256;          // elements per warp row
constexpr int kLaneElems = 8;      // elements per lane per row
constexpr int kThreads = 256;      // threads per CTA
constexpr int kWarps = kThreads / 32;
constexpr float kMagic = 12582912.0f;       // 1.5 * 2^23: adding it rounds to an integer, ties to even
constexpr unsigned kMagicBits = 0x4B400000u;
constexpr float kFltMax = 3.402823466e+38f;
constexpr unsigned kFlagNonFinite = 1u;
constexpr unsigned kFull = 0xffffffffu;
constexpr int kMaxScatter = 64;    // most partitions a scattering send pass can address

// Algorithm 1's scalars and the forms the host chose for the decompressors: the same for every bucket of a call.
struct SendCommon {
    float s, s_e, beta, omb;
    float inv_s, inv_se;             // fl(1/s), fl(1/s_e) for the Newton-Raphson form (inv_s is also the 1-bit magnitude)
    float dq_a, dq_b;                // DEC_FMA: dec(q; s)   = fma(kMagic + 2^(p-1) + q, dq_a, dq_b)
    float de_a, de_b;                // DEC_FMA: dec(e; s_e) = fma(kMagic + 128 + e,     de_a, de_b)
    int dq_mode, de_mode;            // DEC_* chosen by the host for s and for s_e
    int fast;                        // 0: every row takes the careful routine
    int block_log2;                  // log2(B), BLOCK mode
    int reset;                       // k % T_c == 0
    int collect_stats;
    float clip;                      // > 0: element-wise clipping of g to [-clip, clip] before step 1
    int stochastic;                  // stochastic rounding of the gradient codes (extension)
    unsigned seed_lo, seed_hi;       // key of its Philox stream
    unsigned sr_keys[20];            // the ten round keys (seed + r x the Weyl constants), low and high word interleaved
    unsigned k_lo, k_hi;             // the iteration counter, part of the Philox counter
};

// One bucket of a send pass.  Derived sizes: code bytes of a partition = lp * BITS / 8, byte offset of the state
// scales (BLOCK + INT8) = n rounded up to 256.
struct SendBucket {
    const void *grad;
    void *state;
    uint8_t *comm;
    unsigned long long *status;      // [0] flags, [1] saturated gradient codes, [2] saturated 8-bit error codes
    unsigned long long n;            // bucket elements
    unsigned long long lp;           // elements per partition (multiple of 256 and of B)
    unsigned long long stride;       // bytes per partition
    unsigned grid_x;                 // multi-bucket launches: CTAs per partition that work on this bucket
    unsigned reserved;
};

struct SendParams {
    SendCommon c;
    SendBucket b;
    int scatter;                     // 1: partition j is written to part_dst[j] instead of comm + j * stride
    uint8_t *part_dst[kMaxScatter];  // destinations of the partitions (this GPU's memory or a peer's)
};

// Several buckets in one launch: the table travels as a kernel parameter (the parameter space of sm_70 and later
// holds 32,764 bytes), so nothing is allocated and a captured launch carries its own copy.
constexpr int kMaxMulti = 448;
struct SendMultiParams {
    SendCommon c;
    int count;                       // buckets = gridDim.z
    SendBucket b[kMaxMulti];
};
static_assert(sizeof(SendMultiParams) <= 32764, "kernel parameter space");

// What a receive pass needs that is the same for every bucket of a call.
struct ReduceCommon {
    unsigned long long first;        // first partition
    int num_workers;
    int block_log2;
    float s;
    float n_workers_f, inv_n;
    int int_path;                    // codes may be summed as integers (power-of-two s, N <= 16)
    float ra, rb;                    // int path: sum/s (and /N when exact) = fma(kMagic + S, ra, rb)
    int div_mode;                    // division by N: 0 folded into ra/rb or a multiply, 1 Newton-Raphson, 2 IEEE
    float gen_mul;                   // generic FIXED path, gen_mode 0: a multiplier that reproduces q/s for every code; sign code: fl(1/s)
    float inv_s;                     // fl(1/s) for gen_mode 1
    int gen_mode;                    // generic FIXED path: 0 multiply, 1 Newton-Raphson division, 2 IEEE division
    // fused Adam-family step (kernels instantiated with ADAM): moments and weights of the same elements as `out`
    float *adam_m, *adam_v, *adam_theta;
    float lr, beta1, beta2, omb1, omb2, delta;
};

// One bucket of a receive pass.
struct ReduceBucket {
    void *out;
    unsigned long long n, lp, stride, code_bytes;
    unsigned grid_x;                 // multi-bucket launches: CTAs per partition that work on this bucket
    int out_align32;                 // the output pointer is 32-byte aligned: 256-bit stores may be used
};

struct ReduceParams {
    ReduceCommon c;
    ReduceBucket b;
    const uint8_t *parts[64];        // partition `first` of each worker
};

// Several buckets in one launch (grid.z): bucket z's workers are parts[z * num_workers ...].
constexpr int kMaxReduceBuckets = 280;
constexpr int kMaxReducePtrs = 2304;
struct ReduceMultiParams {
    ReduceCommon c;
    int count;
    ReduceBucket b[kMaxReduceBuckets];
    const uint8_t *parts[kMaxReducePtrs];
};
static_assert(sizeof(ReduceMultiParams) <= 32764, "kernel parameter space");

// ------------------------------------------------------------------------------------------
// small helpers

template <int BITS> struct QRange {
    static constexpr float lo = -float(1 << (BITS - 1));
    static constexpr float hi = float((1 << (BITS - 1)) - 1);
    static constexpr float off = float(1 << (BITS - 1));
};

// Nearest integer (ties to even) of y clamped to [lo, hi]; `bits` receives a word whose low
// byte is the two's-complement code.  Clamping first is the same as rounding first because
// both ends are integers and rounding is monotone.
__device__ __forceinline__ float round_clamp(float y, float lo, float hi, unsigned &bits) {
    float t = fminf(fmaxf(y, lo), hi);
    float m = __fadd_rn(t, kMagic);
    bits = __float_as_uint(m);
    return __fadd_rn(m, -kMagic);
}

// Philox4x32-10 (Salmon et al., SC'11), from its published definition: ten rounds of two 32x32->64 multiplications by
// fixed constants, xors with the key, a Weyl bump of the key between rounds.
// `keys`: the round keys (k0 + r 0x9E3779B9, k1 + r 0xBB67AE85), r = 0..9, formed once per call on the host and read
// here as operands from the kernel's parameters, so that the bumps cost no instructions.
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, const unsigned *keys) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const unsigned k0 = keys[2 * r], k1 = keys[2 * r + 1];
        const unsigned long long p0 = static_cast<unsigned long long>(0xD2511F53u) * c.x;      // one wide multiply: both halves
        const unsigned long long p1 = static_cast<unsigned long long>(0xCD9E8D57u) * c.z;
        c = make_uint4(static_cast<unsigned>(p1 >> 32) ^ c.y ^ k0, static_cast<unsigned>(p1),
                       static_cast<unsigned>(p0 >> 32) ^ c.w ^ k1, static_cast<unsigned>(p0));
    }
    return c;
}
// Stochastic rounding adds (b + 1/2) / 256 to h x s, b = one byte of the Philox block of the element's group of 16:
// element i of the bucket takes byte (i mod 4) of word ((i mod 16) / 4) of
// philox(counter = (i/16 low, i/16 high, k low, k high), key = seed).
__device__ __forceinline__ uint4 sr_block(unsigned long long blk, unsigned k_lo, unsigned k_hi, const unsigned *keys) {
    return philox4x32_10(make_uint4(static_cast<unsigned>(blk), static_cast<unsigned>(blk >> 32), k_lo, k_hi), keys);
}
__device__ __forceinline__ float sr_dither(unsigned word, int byte) {
    const float m = __uint_as_float(__byte_perm(word, 0x4B000000u, 0x7540 + byte));      // 2^23 + b
    return __fmaf_rn(m, 0.00390625f, -32767.998046875f);                                 // b / 256 + 1 / 512, exact
}

__device__ __forceinline__ float warp_group_max(float v, int lanes) {
    // max over aligned groups of `lanes` lanes (power of two, <= 32)
    for (int o = 1; o < lanes; o <<= 1) v = fmaxf(v, __shfl_xor_sync(kFull, v, o));
    return v;
}

// code / scale on the fast path, from the magic-biased float m = kMagic + bias + code.
__device__ __forceinline__ float dec_fast(float m, float bias_magic, int mode, float a, float b, float scale,
                                          float inv) {
    if (mode == DEC_FMA) return __fmaf_rn(m, a, b);
    const float c = __fadd_rn(m, -bias_magic);          // the code itself, exact
    const float q0 = __fmul_rn(c, inv);
    const float rem = __fmaf_rn(-q0, scale, c);
    return __fmaf_rn(rem, inv, q0);
}

template <int GRAD>
__device__ __forceinline__ float load_grad1(const void *grad, unsigned long long i) {
    if (GRAD == GRAD_BF16)
        return __uint_as_float(static_cast<unsigned>(static_cast<const uint16_t *>(grad)[i]) << 16);
    return static_cast<const float *>(grad)[i];
}

__device__ __forceinline__ float byte_to_float(unsigned w, int b) {
    return __int2float_rn(static_cast<int>(static_cast<signed char>((w >> (8 * b)) & 0xffu)));
}

// d = sat8(a) | sat8(b) << 8 | c << 16 (signed saturation of two 32-bit integers to bytes)
__device__ __forceinline__ unsigned pack_sat_s8(int a, int b, unsigned c) {
    unsigned d;
    asm("cvt.pack.sat.s8.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(b), "r"(a), "r"(c));
    return d;
}

__device__ __forceinline__ unsigned pack4_bytes(unsigned a, unsigned b, unsigned c, unsigned d) {
    // low bytes of a, b, c, d -> one word, a lowest
    return __byte_perm(__byte_perm(a, b, 0x0040), __byte_perm(c, d, 0x0040), 0x5410);
}

// (a & b) | c in one instruction (the mask and the exponent live in registers)
__device__ __forceinline__ unsigned and_or(unsigned a, unsigned b, unsigned c) {
    unsigned d;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}

// (a ^ b) & c in one instruction
__device__ __forceinline__ unsigned xor_and(unsigned a, unsigned b, unsigned c) {
    unsigned d;
    asm("lop3.b32 %0, %1, %2, %3, 0x28;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}

// Streaming accesses: every byte of both passes is touched exactly once.
__device__ __forceinline__ uint4 ld_stream16(const void *p) { return __ldcs(static_cast<const uint4 *>(p)); }
__device__ __forceinline__ uint2 ld_stream8(const void *p) { return __ldcs(static_cast<const uint2 *>(p)); }
__device__ __forceinline__ unsigned ld_stream4(const void *p) { return __ldcs(static_cast<const unsigned *>(p)); }
__device__ __forceinline__ void st_stream16(void *p, uint4 v) { __stcs(static_cast<uint4 *>(p), v); }
__device__ __forceinline__ void st_stream8(void *p, uint2 v) { __stcs(static_cast<uint2 *>(p), v); }
__device__ __forceinline__ void st_stream4(void *p, unsigned v) { __stcs(static_cast<unsigned *>(p), v); }
__device__ __forceinline__ void st_stream2(void *p, uint16_t v) { __stcs(static_cast<unsigned short *>(p), v); }

// ------------------------------------------------------------------------------------------
// send, careful routine: Algorithm 1 steps 1-2 with every operation written out as the paper states it
// (IEEE division for the decompressor), any value accepted, any block size.  It serves the rows the fast
// routine cannot take: partial and padding rows, rows that hold a NaN or an Inf, blocks wider than a wide row.
//
// Its unit is `nrows` consecutive rows of 256 elements (8 per lane) of one partition: one row when a block fits
// a row (the blocks of the row are then shared by groups of lanes), or the B / 256 rows of one block.  A block
// that spans several rows is walked up to three times -- block statistic of h; codes, new error and its
// statistic; 8-bit error codes -- recomputing h from the inputs each time (nothing of the state is overwritten
// before its last read), so that no register or shared memory has to hold a whole block.

struct CarefulCounts { unsigned saturated, state_saturated, nonfinite; };

// Eight elements of one lane: the gradient, what is added to it, e~_k of Eq. 5, h and whether h is finite.
struct CarefulVals {
    float c[8], prev[8], h[8];
    bool fin[8];
    unsigned long long i0;          // bucket index of the lane's first element
    int valid;                      // leading elements that exist
};

template <int BITS>
__device__ __forceinline__ void store_codes8(uint8_t *dst, const unsigned (&code)[8]) {
    if (BITS == 8) {
        uint2 v;
        v.x = pack4_bytes(code[0], code[1], code[2], code[3]);
        v.y = pack4_bytes(code[4], code[5], code[6], code[7]);
        *reinterpret_cast<uint2 *>(dst) = v;
    } else if (BITS == 4) {
        unsigned w = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) w |= (code[j] & 0xfu) << (4 * j);
        *reinterpret_cast<unsigned *>(dst) = w;
    } else if (BITS == 2) {
        unsigned w = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) w |= (code[j] & 0x3u) << (2 * j);
        *reinterpret_cast<uint16_t *>(dst) = static_cast<uint16_t>(w);
    } else {
        unsigned w = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) w |= (code[j] & 0x1u) << j;
        *dst = static_cast<uint8_t>(w);
    }
}

// Step 1 for the lane's 8 elements of the row at partition-local offset `orow`: g (clipped if asked), the
// compensation c, e~_k, h = g + c.  Counts the 8-bit images of e~_k that Eq. 1's range clamps (Q8COMP only).
template <int GRAD, int STATE, int MODE>
__device__ __forceinline__ void careful_load(const SendCommon &C, const SendBucket &Bk, unsigned long long part,
                                             unsigned long long orow, int lane, bool count, CarefulVals &V,
                                             unsigned &state_saturated) {
    V.i0 = part * Bk.lp + orow + static_cast<unsigned long long>(lane) * kLaneElems;
    V.valid = V.i0 >= Bk.n ? 0 : (Bk.n - V.i0 >= 8 ? 8 : static_cast<int>(Bk.n - V.i0));
    const int8_t *st8 = static_cast<const int8_t *>(Bk.state);
    const float *stf = static_cast<const float *>(Bk.state);
    float sscale = 0.0f;
    if (STATE == ST_INT8 && MODE == MODE_BLOCK && V.valid > 0) {
        const float *st_scales = reinterpret_cast<const float *>(static_cast<const uint8_t *>(Bk.state) + ((Bk.n + 255ull) & ~255ull));
        sscale = st_scales[V.i0 >> C.block_log2];
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        float g = 0.0f, c = 0.0f, prev = 0.0f;
        if (j < V.valid) {
            g = load_grad1<GRAD>(Bk.grad, V.i0 + j);
            if (C.clip > 0.0f && g == g) g = fminf(fmaxf(g, -C.clip), C.clip);          // NaN stays NaN
            if (STATE == ST_INT8) {
                const float ei = __int2float_rn(static_cast<int>(st8[V.i0 + j]));
                c = (MODE == MODE_FIXED) ? __fdiv_rn(ei, C.s_e) : __fmul_rn(ei, sscale);    // dec(e_k; s_e), Eq. 2
                prev = c;
            } else if (STATE == ST_FP32) {
                c = stf[V.i0 + j];
                prev = c;
            } else if (STATE == ST_Q8COMP) {
                prev = stf[V.i0 + j];
                const float y = __fmul_rn(prev, C.s_e);
                if (count && (y >= 127.5f || y < -128.5f)) state_saturated += 1u;          // nearest integer outside [-128, 127]
                unsigned bits;
                c = __fdiv_rn(round_clamp(y, -128.0f, 127.0f, bits), C.s_e);
            }
        }
        V.c[j] = c;
        V.prev[j] = prev;
        V.h[j] = __fadd_rn(g, c);                             // step 1 / Eq. 2
        V.fin[j] = fabsf(V.h[j]) <= kFltMax;                  // false for NaN and +-Inf
    }
}

// The lane's share of a block's statistic: the largest finite |h| (codes of 2 bits and more), or the pairwise
// sum of the finite |h| (sign code; absent elements are zeros here and enter as such).
template <int BITS>
__device__ __forceinline__ float careful_lane_stat(const CarefulVals &V) {
    float a[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) a[j] = V.fin[j] ? fabsf(V.h[j]) : 0.0f;
    if (BITS == 1)
        return __fadd_rn(__fadd_rn(__fadd_rn(a[0], a[1]), __fadd_rn(a[2], a[3])), __fadd_rn(__fadd_rn(a[4], a[5]), __fadd_rn(a[6], a[7])));
    float m = 0.0f;
#pragma unroll
    for (int j = 0; j < 8; ++j) m = fmaxf(m, a[j]);
    return m;
}
// ... combined over aligned groups of `lanes` lanes: every lane of a group ends with the same value (fp32 addition
// commutes, so the butterfly is the balanced tree over the group's positions in index order).
template <int BITS>
__device__ __forceinline__ float careful_group_stat(float v, int lanes) {
    for (int o = 1; o < lanes; o <<= 1) {
        const float w = __shfl_xor_sync(kFull, v, o);
        v = (BITS == 1) ? __fadd_rn(v, w) : fmaxf(v, w);
    }
    return v;
}

// scale and multiplier of a block from its statistic; `len` = elements of the block that exist (sign code only)
template <int BITS>
__device__ __forceinline__ void careful_block_scale(float stat, unsigned long long len, float &scale, float &mult) {
    if (BITS == 1) {
        scale = __fdiv_rn(stat, static_cast<float>(len));      // mean |h|; len >= 1 wherever the result is used
        mult = 0.0f;
    } else {
        constexpr float hi = QRange<BITS>::hi;
        scale = stat > 0.0f ? __fdiv_rn(stat, hi) : 0.0f;
        mult = stat > 0.0f ? __fdiv_rn(hi, stat) : 0.0f;
    }
}

// Eq. 1 / Eq. 3, step 2 and Eq. 5 for the lane's 8 elements, given the multiplier (s, or the block's inverse scale) and
// the block's scale.  code: low bits of each word = the wire field.
template <int BITS, int MODE, bool STOCH>
__device__ __forceinline__ void careful_quantise(const SendCommon &C, const CarefulVals &V, float mult, float scale, bool count,
                                                 unsigned (&code)[8], float (&e_new)[8], CarefulCounts &N) {
    float u8[8];
    if (STOCH) {                                            // i0 is a multiple of 8: one half of a block of 16
        const uint4 r = sr_block(V.i0 >> 4, C.k_lo, C.k_hi, C.sr_keys);
        const bool upper = ((V.i0 >> 3) & 1ull) != 0ull;
        const unsigned w0 = upper ? r.z : r.x, w1 = upper ? r.w : r.y;
#pragma unroll
        for (int j = 0; j < 4; ++j) { u8[j] = sr_dither(w0, j); u8[4 + j] = sr_dither(w1, j); }
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const float h = V.h[j];
        const bool fin = V.fin[j];
        if (!fin && j < V.valid && count) N.nonfinite = 1u;
        float d;
        if (BITS == 1) {
            // sign code: q = -1 if h < 0 else +1 (so +-0 and NaN give +1); the wire bit is 1 for -1
            const bool neg = h < 0.0f;
            code[j] = neg ? 1u : 0u;
            const float q = neg ? -1.0f : 1.0f;
            d = (MODE == MODE_FIXED) ? __fdiv_rn(q, C.s) : __fmul_rn(q, scale);
        } else {
            constexpr float lo = QRange<BITS>::lo, hi = QRange<BITS>::hi;
            const float hq = (h != h) ? 0.0f : h;               // NaN is sent as code 0
            float y = __fmul_rn(hq, mult);                      // h x s of Eq. 1
            if (!fin) y = hq;                                   // +-Inf saturates whatever the scale
            float r;
            if (STOCH && fin) {                                 // floor(y + u): up with probability frac(y)
                const float fl = floorf(__fadd_rn(y, u8[j]));
                if (count && C.collect_stats && j < V.valid && (fl < lo || fl > hi)) N.saturated += 1u;
                r = fminf(fmaxf(fl, lo), hi);
                code[j] = static_cast<unsigned>(__float2int_rn(r));
            } else {
                r = round_clamp(y, lo, hi, code[j]);            // round_p-bit
                // nearest integer outside the range: y >= hi + 1/2 (hi is odd, the tie goes up and out) or
                // y < lo - 1/2 (lo is even, the tie stays in); a block scale keeps every code inside
                if (MODE != MODE_BLOCK && count && C.collect_stats && !STOCH && fin && j < V.valid &&
                    (y >= hi + 0.5f || y < lo - 0.5f)) N.saturated += 1u;
            }
            d = (MODE == MODE_FIXED) ? __fdiv_rn(r, C.s) : __fmul_rn(r, scale);     // step 2: dec(q; s)
        }
        const float delta = fin ? __fsub_rn(h, d) : 0.0f;
        // an absent element has no error (with the sign code its h = 0 would otherwise leave -d behind and enter the
        // block's largest error)
        e_new[j] = j < V.valid ? __fadd_rn(__fmul_rn(C.omb, V.prev[j]), __fmul_rn(C.beta, delta)) : 0.0f;   // Eq. 5
    }
}

// `nrows` consecutive rows of partition `part` starting at partition-local offset `o` (a multiple of 256, and of B
// when nrows > 1).  pbase: where the partition's codes and scales go.  Elements >= n are treated as absent (code 0, no
// state).  Out of line and reading the kernel's parameters in place (they are __grid_constant__, so their address can
// be taken without a local copy), so that the fast routine's register allocation is not disturbed by this rarely taken
// path.
template <int GRAD, int STATE, int BITS, int MODE, bool STOCH>
__device__ __noinline__ CarefulCounts send_careful(const SendCommon &C, const SendBucket &Bk, uint8_t *pbase,
                                                   unsigned long long part, unsigned long long o, int nrows, int lane) {
    CarefulCounts N = {0u, 0u, 0u};
    const bool wide = MODE == MODE_BLOCK && C.block_log2 > 8;   // one block spanning all rows of the unit (nrows = B / 256)
    const int lanes_per_block = (MODE != MODE_BLOCK) ? 1 : (C.block_log2 >= 8 ? 32 : (1 << (C.block_log2 - 3)));
    const unsigned long long code_bytes = Bk.lp * BITS / 8;
    int8_t *st8 = static_cast<int8_t *>(Bk.state);
    float *stf = static_cast<float *>(Bk.state);
    float *st_scales = reinterpret_cast<float *>(static_cast<uint8_t *>(Bk.state) + ((Bk.n + 255ull) & ~255ull));
    const bool stats = C.collect_stats != 0;

    // ---- a block wider than a row: its statistic first ------------------------------------------------------
    float wscale = 0.0f, wmult = 0.0f;
    const unsigned long long block0 = part * Bk.lp + o;         // bucket index of the unit's first element
    if (wide) {
        float level[5];                                         // partial sums of 2^l rows (sign code): a binary counter
        float amax = 0.0f;
        for (int r = 0; r < nrows; ++r) {
            CarefulVals V;
            unsigned dummy = 0u;
            careful_load<GRAD, STATE, MODE>(C, Bk, part, o + static_cast<unsigned long long>(r) * kRow, lane, false, V, dummy);
            float v = careful_group_stat<BITS>(careful_lane_stat<BITS>(V), 32);
            if (BITS == 1) {
                int l = 0;
                for (int t = r; t & 1; t >>= 1, ++l) v = __fadd_rn(level[l], v);   // earlier rows on the left
                level[l] = v;
            } else {
                amax = fmaxf(amax, v);
            }
        }
        unsigned long long len = 1ull << C.block_log2;
        if (block0 < Bk.n && Bk.n - block0 < len) len = Bk.n - block0;
        int top = 0;
        while ((1 << top) < nrows) ++top;
        careful_block_scale<BITS>(BITS == 1 ? level[top] : amax, len, wscale, wmult);
    }

    // ---- codes, new error (and, for a wide block with the 8-bit state, the statistic of the new error) -------
    float e_amax = 0.0f;
    for (int r = 0; r < nrows; ++r) {
        const unsigned long long orow = o + static_cast<unsigned long long>(r) * kRow;
        CarefulVals V;
        careful_load<GRAD, STATE, MODE>(C, Bk, part, orow, lane, stats, V, N.state_saturated);
        float scale = wscale, mult = (MODE == MODE_FIXED) ? C.s : wmult;
        if (MODE == MODE_BLOCK && !wide) {
            const float stat = careful_group_stat<BITS>(careful_lane_stat<BITS>(V), lanes_per_block);
            const unsigned long long b0 = (V.i0 >> C.block_log2) << C.block_log2;
            unsigned long long len = 1ull << C.block_log2;
            if (b0 < Bk.n && Bk.n - b0 < len) len = Bk.n - b0;
            careful_block_scale<BITS>(stat, len, scale, mult);
        }
        unsigned code[8];
        float e_new[8];
        careful_quantise<BITS, MODE, STOCH>(C, V, mult, scale, true, code, e_new, N);

        const unsigned long long ol = orow + static_cast<unsigned long long>(lane) * kLaneElems;   // partition-local
        store_codes8<BITS>(pbase + ol * BITS / 8, code);
        if (MODE == MODE_BLOCK && !wide) {
            if ((lane & (lanes_per_block - 1)) == 0 && ((ol & ((1ull << C.block_log2) - 1)) == 0))
                *reinterpret_cast<float *>(pbase + code_bytes + (ol >> C.block_log2) * 4) = scale;
        }

        // Eq. 7: reset, or keep / compress the new error
        if (STATE == ST_INT8) {
            if (C.reset) {
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    if (j < V.valid) st8[V.i0 + j] = 0;
                if (MODE == MODE_BLOCK && !wide && (lane & (lanes_per_block - 1)) == 0 &&
                    (V.i0 & ((1ull << C.block_log2) - 1)) == 0 && V.valid > 0)
                    st_scales[V.i0 >> C.block_log2] = 0.0f;
            } else if (wide) {
#pragma unroll
                for (int j = 0; j < 8; ++j) e_amax = fmaxf(e_amax, fabsf(e_new[j]));
            } else {
                float emult = C.s_e, escale = 0.0f;
                if (MODE == MODE_BLOCK) {
                    float am = 0.0f;
#pragma unroll
                    for (int j = 0; j < 8; ++j) am = fmaxf(am, fabsf(e_new[j]));
                    am = careful_group_stat<8>(am, lanes_per_block);
                    escale = am > 0.0f ? __fdiv_rn(am, 127.0f) : 0.0f;
                    emult = am > 0.0f ? __fdiv_rn(127.0f, am) : 0.0f;
                }
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const float y = __fmul_rn(e_new[j], emult);
                    if (MODE == MODE_FIXED && stats && j < V.valid && (y >= 127.5f || y < -128.5f)) N.state_saturated += 1u;
                    unsigned eb;
                    (void)round_clamp(y, -128.0f, 127.0f, eb);            // compressor(e~; s_e, 8)
                    if (j < V.valid) st8[V.i0 + j] = static_cast<int8_t>(eb & 0xffu);
                }
                if (MODE == MODE_BLOCK && (lane & (lanes_per_block - 1)) == 0 &&
                    (V.i0 & ((1ull << C.block_log2) - 1)) == 0 && V.valid > 0)
                    st_scales[V.i0 >> C.block_log2] = escale;
            }
        } else if (STATE == ST_FP32 || STATE == ST_Q8COMP) {
#pragma unroll
            for (int j = 0; j < 8; ++j)
                if (j < V.valid) stf[V.i0 + j] = C.reset ? 0.0f : e_new[j];
        }
    }
    if (wide) {
        if (lane == 0) *reinterpret_cast<float *>(pbase + code_bytes + (o >> C.block_log2) * 4) = wscale;
        if (STATE == ST_INT8 && block0 < Bk.n) {
            if (C.reset) {
                if (lane == 0) st_scales[block0 >> C.block_log2] = 0.0f;
            } else {
                // ---- 8-bit codes of the new error, which is formed once more from the untouched inputs ----------
                e_amax = careful_group_stat<8>(e_amax, 32);
                const float escale = e_amax > 0.0f ? __fdiv_rn(e_amax, 127.0f) : 0.0f;
                const float emult = e_amax > 0.0f ? __fdiv_rn(127.0f, e_amax) : 0.0f;
                for (int r = 0; r < nrows; ++r) {
                    CarefulVals V;
                    unsigned dummy = 0u;
                    careful_load<GRAD, STATE, MODE>(C, Bk, part, o + static_cast<unsigned long long>(r) * kRow, lane, false, V, dummy);
                    unsigned code[8];
                    float e_new[8];
                    CarefulCounts unused = {0u, 0u, 0u};
                    careful_quantise<BITS, MODE, STOCH>(C, V, wmult, wscale, false, code, e_new, unused);
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        unsigned eb;
                        (void)round_clamp(__fmul_rn(e_new[j], emult), -128.0f, 127.0f, eb);
                        if (j < V.valid) st8[V.i0 + j] = static_cast<int8_t>(eb & 0xffu);
                    }
                }
                __syncwarp();
                if (lane == 0) st_scales[block0 >> C.block_log2] = escale;
            }
        }
    }
    return N;
}

// ------------------------------------------------------------------------------------------
// send, fast routine: "wide rows" of 512 elements, 16 consecutive elements per lane, computed two at a
// time with the packed fp32x2 instructions of sm_100 (one issue slot for two IEEE operations).

constexpr int kWide = 512;         // elements per wide row
constexpr int kWideLane = 16;      // elements per lane per wide row

typedef unsigned long long f32x2;  // two fp32 in one 64-bit register pair: low word = the even element

__device__ __forceinline__ f32x2 pk2(float lo, float hi) {
    f32x2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ f32x2 dup2(float v) { return pk2(v, v); }
__device__ __forceinline__ void unpk2(f32x2 v, float &lo, float &hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ f32x2 fadd2(f32x2 a, f32x2 b) { f32x2 d; asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b)); return d; }
__device__ __forceinline__ f32x2 fsub2(f32x2 a, f32x2 b) { f32x2 d; asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b)); return d; }
__device__ __forceinline__ f32x2 fmul2(f32x2 a, f32x2 b) { f32x2 d; asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b)); return d; }
__device__ __forceinline__ f32x2 ffma2(f32x2 a, f32x2 b, f32x2 c) { f32x2 d; asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c)); return d; }
// a + b rounded toward minus infinity: with b = kMagic (+ bias) the sum's mantissa holds floor(a) (+ bias)
__device__ __forceinline__ f32x2 fadd2_down(f32x2 a, f32x2 b) { f32x2 d; asm("add.rm.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b)); return d; }
// The assembler contracts a packed multiply that feeds a packed add or subtract into one packed FMA even
// though both carry an explicit rounding mode (seen as single-rounded results on sm_100a, CUDA 12.9; the same
// happens when the product is written fma(a, b, -0)).  Where Algorithm 1 rounds the product and the sum
// separately there are two ways out: the sum with scalar instructions, which are never contracted
// (fadd2_after_mul), or the product as fma(a, b, +0) (fmul2_pz), where the sign of a zero does not matter.
__device__ __forceinline__ f32x2 fadd2_after_mul(f32x2 a, f32x2 b) {
    float a0, a1, b0, b1;
    unpk2(a, a0, a1);
    unpk2(b, b0, b1);
    return pk2(__fadd_rn(a0, b0), __fadd_rn(a1, b1));
}
// fma(a, b, +0) is the rounded product except that a product of -0 comes out as +0, and no later add can be contracted
// with it.  Usable where that sign cannot show: in a running sum that starts at +0 (such a sum is never -0), and where
// everything computed from the result is stored as integer codes or as scales taken from magnitudes.
__device__ __forceinline__ f32x2 fmul2_pz(f32x2 a, f32x2 b) {
    f32x2 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(0ull));
    return d;
}
__device__ __forceinline__ unsigned hfma2_bf16(unsigned a, unsigned b, unsigned c) {
    unsigned d;
    asm("fma.rn.bf16x2 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}

// Per-lane base pointers of one partition: everything a wide row needs is base + row * (bytes per row).
struct LanePtrs {
    uint8_t *state;           // this lane's 16 state elements of wide row 0 (int8 or fp32)
    uint8_t *codes;           // this lane's code bytes of wide row 0 in the partition's code area
    float *wire_scales;       // BLOCK: the partition's scale area
    float *state_scales;      // BLOCK + INT8: scale of the bucket's block 0
    unsigned long long elem0; // bucket index of this lane's first element of wide row 0
    unsigned lane_elem;       // partition-local index of this lane's first element of wide row 0
    unsigned lane_block;      // BLOCK: index, within a wide row, of the block this lane's elements belong to
    bool leader;              // BLOCK: this lane stores the scales of its block (the first lane of the block)
};

// ---- per-warp ring of asynchronous copies (cp.async) -------------------------------------------
// Every warp stages the inputs of its next wide rows in shared memory with cp.async, in 16-byte chunks
// laid out so that a copy instruction of the warp reads 512 contiguous bytes of global memory; the bytes in
// flight occupy no registers, and the depth of the ring, not the phase a warp happens to be in, decides how
// much of the HBM latency is covered.  A lane's own elements span several chunks that other lanes copied,
// so a chunk c is stored at position c ^ ((c >> 3) & (chunks per lane - 1)): both the copies and the
// 16-byte reads of 8 consecutive lanes then fall into 8 different bank groups.  cp.async.wait_group
// followed by __syncwarp() orders the warp's reads after all of its lanes' copies.
// Shared memory is addressed by its 32-bit window offset throughout.
__device__ __forceinline__ void cp_async16(unsigned saddr, const void *gmem) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" :: "r"(saddr), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async4(unsigned saddr, const void *gmem) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" :: "r"(saddr), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async8(unsigned saddr, const void *gmem) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" :: "r"(saddr), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" :: "n"(N) : "memory"); }
__device__ __forceinline__ uint4 lds16(unsigned saddr) {
    uint4 v;
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(saddr) : "memory");
    return v;
}
__device__ __forceinline__ uint2 lds8(unsigned saddr) {
    uint2 v;
    asm volatile("ld.shared.v2.b32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(saddr) : "memory");
    return v;
}
__device__ __forceinline__ unsigned lds2(unsigned saddr) {
    unsigned short v;
    asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(saddr) : "memory");
    return v;
}
__device__ __forceinline__ unsigned lds4(unsigned saddr) {
    unsigned v;
    asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v) : "r"(saddr) : "memory");
    return v;
}
__device__ __forceinline__ void st_stream32(void *p, const unsigned *v) {      // one 256-bit store
    asm volatile("st.global.cs.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                 :: "l"(p), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]) : "memory");
}

template <int GRAD, int STATE, int MODE>
struct Ring {
    static constexpr int kGradChunks = (GRAD == GRAD_BF16) ? 2 : 4;                          // 16-byte chunks per lane
    static constexpr int kStateChunks = (STATE == ST_INT8) ? 1 : (STATE == ST_NONE ? 0 : 4);
    static constexpr int kScaleBytes = (STATE == ST_INT8 && MODE == MODE_BLOCK) ? 4 : 0;
    static constexpr int kWarpSlotBytes = (kGradChunks + kStateChunks) * 512 + kScaleBytes * 32;
    static constexpr int kSlotStride = kWarpSlotBytes * kWarps;
    static constexpr int kFit = 73728 / kSlotStride;
    static constexpr int kDepth = kFit > 6 ? 6 : kFit;
    static constexpr int kBytes = kDepth * kSlotStride;
    static constexpr int kStateOff = kGradChunks * 512;
    static constexpr int kScaleOff = (kGradChunks + kStateChunks) * 512;
    static_assert(kDepth >= 2, "the ring needs at least two slots");
};

// The lane's own shared-memory addresses inside slot 0 of its warp's ring.
template <int GRAD, int STATE>
struct RingAddr {
    static constexpr int GC = (GRAD == GRAD_BF16) ? 2 : 4;
    static constexpr int SC = (STATE == ST_INT8 || STATE == ST_NONE) ? 1 : 4;
    unsigned g_stage;       // where this lane's copy of chunk (32 k + lane) goes for k = 0; add 512 k
    unsigned e_stage;
    unsigned g_fetch[GC];   // where this lane's own chunks are
    unsigned e_fetch[SC];
    unsigned sc;            // state scale
};

template <int GRAD, int STATE, int MODE>
__device__ __forceinline__ void ring_addresses(unsigned ring0, int lane, int warp_in_cta, RingAddr<GRAD, STATE> &A) {
    using R = Ring<GRAD, STATE, MODE>;
    constexpr int GC = R::kGradChunks;
    constexpr int SC = RingAddr<GRAD, STATE>::SC;
    const unsigned wbase = ring0 + warp_in_cta * R::kWarpSlotBytes;
    const unsigned L = static_cast<unsigned>(lane);
    A.g_stage = wbase + ((L ^ ((L >> 3) & (GC - 1))) << 4);
    const unsigned xg = (GC == 2) ? ((L >> 2) & 1u) : ((L >> 1) & 3u);
#pragma unroll
    for (int k = 0; k < GC; ++k) A.g_fetch[k] = wbase + ((GC * L + (static_cast<unsigned>(k) ^ xg)) << 4);
    if (SC == 4) {
        A.e_stage = wbase + R::kStateOff + ((L ^ ((L >> 3) & 3u)) << 4);
        const unsigned xe = (L >> 1) & 3u;
#pragma unroll
        for (int k = 0; k < SC; ++k) A.e_fetch[k] = wbase + R::kStateOff + ((4 * L + (static_cast<unsigned>(k) ^ xe)) << 4);
    } else {
        A.e_stage = wbase + R::kStateOff + (L << 4);
        A.e_fetch[0] = A.e_stage;
    }
    A.sc = wbase + R::kScaleOff + (L << 2);
}

// Issue the copies of one wide row.  g_row / e_row: global address of the row's first byte plus lane * 16.
template <int GRAD, int STATE, int MODE>
__device__ __forceinline__ void stage_row(const RingAddr<GRAD, STATE> &A, unsigned slot_off, const uint8_t *g_row,
                                          const uint8_t *e_row, const float *scale_ptr) {
    using R = Ring<GRAD, STATE, MODE>;
#pragma unroll
    for (int k = 0; k < R::kGradChunks; ++k) cp_async16(A.g_stage + slot_off + 512 * k, g_row + 512 * k);
#pragma unroll
    for (int k = 0; k < R::kStateChunks; ++k) cp_async16(A.e_stage + slot_off + 512 * k, e_row + 512 * k);
    if (R::kScaleBytes) cp_async4(A.sc + slot_off, scale_ptr);
}

template <int GRAD, int STATE>
struct WideIn {
    static constexpr int GW = (GRAD == GRAD_BF16) ? 8 : 16;                          // gradient words per lane
    static constexpr int EW = (STATE == ST_INT8) ? 4 : (STATE == ST_NONE ? 1 : 16);  // state words per lane
    unsigned g[GW];
    unsigned e[EW];
    float sscale;                                                                    // BLOCK + INT8
};

template <int GRAD, int STATE, int MODE>
__device__ __forceinline__ void fetch_row(const RingAddr<GRAD, STATE> &A, unsigned slot_off, WideIn<GRAD, STATE> &in) {
    using R = Ring<GRAD, STATE, MODE>;
    constexpr int EW = WideIn<GRAD, STATE>::EW;
#pragma unroll
    for (int k = 0; k < R::kGradChunks; ++k) {
        const uint4 v = lds16(A.g_fetch[k] + slot_off);
        in.g[4 * k] = v.x; in.g[4 * k + 1] = v.y; in.g[4 * k + 2] = v.z; in.g[4 * k + 3] = v.w;
    }
    in.e[0] = 0u;
#pragma unroll
    for (int k = 0; k < R::kStateChunks; ++k) {
        const uint4 v = lds16(A.e_fetch[k % RingAddr<GRAD, STATE>::SC] + slot_off);
        in.e[(4 * k) % EW] = v.x; in.e[(4 * k + 1) % EW] = v.y;
        in.e[(4 * k + 2) % EW] = v.z; in.e[(4 * k + 3) % EW] = v.w;
    }
    in.sscale = R::kScaleBytes ? __uint_as_float(lds4(A.sc + slot_off)) : 0.0f;
}

// The scalars of Algorithm 1 the fast routine needs, read from the parameters once per kernel.
struct SendConsts {
    float s, s_e, beta, omb, inv_s, inv_se, dq_a, dq_b, de_a, de_b, clip;
    int dq_mode, de_mode, block_log2, reset;
    // BLOCK: the scales of wide row w start at index (w << row_shl) >> row_shr of the partition's scales: 512 / B
    // blocks per row when B <= 512, one block per B / 512 rows otherwise
    unsigned row_shl, row_shr;
    // BLOCK, B > 512: a block spans `group_warps` (2, 4 or 8) wide rows, which neighbouring warps of the CTA hold at the
    // same time; they exchange their rows' maxima (sums) through shared memory
    unsigned group_warps;            // 1 when B <= 512
    unsigned xslot, xgroup;          // shared-memory addresses: this warp's slot; the slot this lane reads back
    unsigned bar_id, bar_threads;    // the named barrier of the warp's group
    unsigned k_lo, k_hi;
    const unsigned *sr_keys;         // the Philox round keys, in the kernel's parameters
};

// Field j of the packed codes sits in the low bits of mb_j = bits(kMagic + 2^(p-1) + q_j):
// sum_j mb_j * R^j = kMagicBits * sum_j R^j + sum_j (q_j + 2^(p-1)) R^j  (mod 2^32), R = 2^p; removing the
// constant and flipping each field's top bit turns the biased fields into two's complement.  The sum is a Horner
// chain of integer multiply-adds (fp32 pipe), fed with the codes from the last one down as they are produced, so that
// no code has to wait in a register for the others.
template <int BITS>
struct CodePacker {
    static constexpr int kPerWord = 32 / BITS;               // 16, 8 or 4 codes per word
    static constexpr int kWords = 16 / kPerWord;             // words for a lane's 16 codes: 1, 2 or 4
    unsigned w[kWords];
    __device__ __forceinline__ void clear() {
#pragma unroll
        for (int i = 0; i < kWords; ++i) w[i] = 0u;
    }
    // code j of the lane's 16; the codes of a word must arrive in descending order of j
    __device__ __forceinline__ void push(int j, unsigned mb) {
        w[(j / kPerWord) % kWords] = w[(j / kPerWord) % kWords] * (1u << BITS) + mb;
    }
    __device__ __forceinline__ unsigned word(int i) const {
        unsigned ones = 0u, flip = 0u;
#pragma unroll
        for (int j = 0; j < kPerWord; ++j) { ones |= 1u << (BITS * j); flip |= (1u << (BITS - 1)) << (BITS * j); }
        return (w[i % kWords] - kMagicBits * ones) ^ flip;
    }
};

// ---- the two divisions of a block scale, without the general division routine --------------------------------
// scale = amax / qmax and 1/scale = qmax / amax must carry the bits of the IEEE division (the oracle divides).
// amax / c for the three constants that occur (1, 7, 127): multiply by fl(1/c) and correct once with two fused
// multiply-adds.  qmax / amax: the hardware's approximate reciprocal, corrected the same way, for amax in
// [2^-100, 2^100]; outside that range the general division is used.  Both short forms are compared against
// __fdiv_rn for EVERY positive finite float by loco_selfcheck_block_division() (and by the GPU tests).
__device__ __forceinline__ float div_by_qmax(float a, float c, float rc) {
    const float q0 = __fmul_rn(a, rc);
    const float rem = __fmaf_rn(-q0, c, a);
    return __fmaf_rn(rem, rc, q0);
}
__device__ __forceinline__ float qmax_over(float c, float a) {
    if (__float_as_uint(a) - 0x0d800000u <= 0x71800000u - 0x0d800000u) {      // 2^-100 <= a <= 2^100
        float x;
        asm("rcp.approx.f32 %0, %1;" : "=f"(x) : "f"(a));
        const float q0 = __fmul_rn(c, x);
        const float rem = __fmaf_rn(-q0, a, c);
        return __fmaf_rn(rem, x, q0);
    }
    return __fdiv_rn(c, a);
}

// sum over aligned groups of `lanes` lanes as a balanced tree in index order (fp32 addition commutes, so both lanes
// of a pair form the same sum); every lane of a group ends with the group's sum.  `lanes` is the same for the whole
// launch, so the steps that a small group does not need are skipped by uniform predicates, not computed and dropped.
__device__ __forceinline__ float group_sum32(float v, int lanes) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        if (o < lanes) v = __fadd_rn(v, __shfl_xor_sync(kFull, v, o));
    }
    return v;
}

// The same without the fallback, for callers that have already sent every a outside [2^-100, 2^100] elsewhere.
__device__ __forceinline__ float qmax_over_midrange(float c, float a) {
    float x;
    asm("rcp.approx.f32 %0, %1;" : "=f"(x) : "f"(a));
    const float q0 = __fmul_rn(c, x);
    const float rem = __fmaf_rn(-q0, a, c);
    return __fmaf_rn(rem, x, q0);
}
__device__ __forceinline__ bool in_midrange(float a) { return __float_as_uint(a) - 0x0d800000u <= 0x71800000u - 0x0d800000u; }

template <bool WIDE>
__device__ __forceinline__ size_t scale_index(const SendConsts &K, unsigned wrow) {
    return WIDE ? static_cast<size_t>(wrow >> K.row_shr) : static_cast<size_t>(wrow) << K.row_shl;
}

// max over aligned groups of `lanes` lanes (1 to 32): four steps without a branch, the fifth (a block of 512 elements
// spans the whole warp) under a uniform one
__device__ __forceinline__ float group_max32(float v, int lanes) {
#pragma unroll
    for (int o = 1; o < 16; o <<= 1) {
        const float w = __shfl_xor_sync(kFull, v, o);
        v = o < lanes ? fmaxf(v, w) : v;
    }
    if (lanes > 16) v = fmaxf(v, __shfl_xor_sync(kFull, v, 16));
    return v;
}

// A block wider than a wide row: the warps that hold its rows combine their (warp-uniform) row values -- the maximum, or
// for the sign code the sum as a balanced tree in row order.  Every warp of the group calls this the same number of
// times; successive calls alternate between two sets of slots, so that a warp that runs ahead to its next exchange
// writes where the others have long since read (it had to pass the barrier of the exchange in between, which they
// reach only after reading).  The barrier is the hardware's named barrier for the group's threads, not a spin.
template <bool SUM>
__device__ __forceinline__ float wide_exchange(const SendConsts &K, unsigned &xphase, float v, int lane) {
    if (lane == 0) asm volatile("st.shared.f32 [%0], %1;" :: "r"(K.xslot + xphase), "f"(v) : "memory");
    asm volatile("bar.sync %0, %1;" :: "r"(K.bar_id), "r"(K.bar_threads) : "memory");
    const float x = __uint_as_float(lds4(K.xgroup + xphase));
    xphase ^= 4u * kWarps;
    return SUM ? group_sum32(x, static_cast<int>(K.group_warps)) : group_max32(x, static_cast<int>(K.group_warps));
}

// One wide row.  Returns false if some lane of the warp met a value that the fast arithmetic does not cover (NaN,
// +-Inf, a magnitude that could overflow, a block maximum outside the range of the short division sequences): the
// caller then redoes the row with the careful routine.  Invariant the caller relies on: no byte of the error state
// (codes, values or scales) has been written before the last `return false`; codes and wire scales of the row may
// already have been stored (block mode) and the careful routine stores the same bytes again.
// VAR_LEAN: both decompressors are the single fused multiply-add and no statistics are collected;
// VAR_LEAN_NR: the same, but dec(e; s_e) is the Newton-Raphson form (s_e = 6 s of the paper), still packed;
// VAR_GENERAL: the forms are chosen per call at run time (scalar code) and statistics may be collected.
// VAR_STOCHASTIC: VAR_GENERAL with stochastic rounding of the gradient codes (extension; global scale only).
// VAR_LEAN_X / VAR_LEAN_NR_X: the lean forms plus what a call may ask for on top (statistics, clipping of g).
// VAR_LEAN_SR: VAR_LEAN_X with stochastic rounding.
enum : int { VAR_LEAN = 0, VAR_LEAN_NR = 1, VAR_GENERAL = 2, VAR_STOCHASTIC = 3, VAR_LEAN_X = 4, VAR_LEAN_NR_X = 5, VAR_LEAN_SR = 6 };
// added to VAR_LEAN or VAR_GENERAL of a block-scaled kernel: a block is wider than a wide row (B > 512) and its rows sit
// on neighbouring warps, which exchange their maxima (see wide_exchange)
enum : int { VAR_WIDE_BLOCKS = 16 };
__host__ __device__ constexpr int var_base(int var) { return var & 15; }
__host__ __device__ constexpr bool var_is_wide(int var) { return (var & VAR_WIDE_BLOCKS) != 0; }
__host__ __device__ constexpr bool var_is_lean(int var) { return var_base(var) == VAR_LEAN || var_base(var) == VAR_LEAN_NR || var_base(var) == VAR_LEAN_X || var_base(var) == VAR_LEAN_NR_X || var_base(var) == VAR_LEAN_SR; }
__host__ __device__ constexpr bool var_has_extras(int var) { return var_base(var) != VAR_LEAN && var_base(var) != VAR_LEAN_NR; }
__host__ __device__ constexpr bool var_is_sr(int var) { return var_base(var) == VAR_STOCHASTIC || var_base(var) == VAR_LEAN_SR; }

// dec(e; s_e) of a pair from the magic floats m2 = kMagic + 128 + e
template <int VAR>
__device__ __forceinline__ f32x2 dec_state2(const SendConsts &K, f32x2 m2, float emagic, int de_mode) {
    if (VAR == VAR_LEAN || VAR == VAR_LEAN_X || VAR == VAR_LEAN_SR) return ffma2(m2, dup2(K.de_a), dup2(K.de_b));
    if (VAR == VAR_LEAN_NR || VAR == VAR_LEAN_NR_X) {
        const f32x2 e2 = fadd2(m2, dup2(-emagic));                   // the codes, exact
        const f32x2 inv2 = dup2(K.inv_se);
        const f32x2 q0 = fmul2(e2, inv2);
        const f32x2 rem = ffma2(q0, dup2(-K.s_e), e2);
        return ffma2(rem, inv2, q0);
    }
    float m0, m1;
    unpk2(m2, m0, m1);
    return pk2(dec_fast(m0, emagic, de_mode, K.de_a, K.de_b, K.s_e, K.inv_se),
               dec_fast(m1, emagic, de_mode, K.de_a, K.de_b, K.s_e, K.inv_se));
}

template <int GRAD, int STATE, int BITS, int MODE, int VAR>
__device__ __forceinline__ bool send_wide_row(const SendConsts &K, const LanePtrs &L, const WideIn<GRAD, STATE> &in,
                                              unsigned wrow, int lane, bool stats, unsigned &saturated, unsigned &state_saturated,
                                              unsigned &xphase) {
    constexpr float lo = QRange<BITS>::lo, hi = QRange<BITS>::hi, qmagic = kMagic + QRange<BITS>::off;
    constexpr float emagic = kMagic + 128.0f;
    constexpr bool kStateF32 = (STATE == ST_FP32 || STATE == ST_Q8COMP);
    // With the 8-bit state (or none) everything stored is a code or a scale, which the sign of a zero cannot change: the
    // products of Eq. 5 may then be taken as fma(a, b, +0) (the rounded product up to the sign of zero) and summed with
    // a packed add; with an fp32 state the sign of a zero is stored, so there the sum stays scalar (see fadd2_after_mul).
    constexpr bool kSignFree = !kStateF32;
    constexpr int GW = WideIn<GRAD, STATE>::GW, EW = WideIn<GRAD, STATE>::EW;
    constexpr bool LEAN = var_is_lean(VAR), EXTRAS = var_has_extras(VAR), WIDE = var_is_wide(VAR);
    const int dq_mode = LEAN ? DEC_FMA : K.dq_mode, de_mode = K.de_mode;
    const int lanes_per_block = (MODE == MODE_BLOCK) ? (K.block_log2 >= 9 ? 32 : (1 << (K.block_log2 - 4))) : 1;    // B <= 512 here
    const f32x2 zero2 = 0ull;

    // ---- values outside the fast arithmetic -------------------------------------------------------------
    // x * 0 is 0 for finite x and NaN otherwise; with fp32 state, g and e~ are first scaled by 4 so that
    // anything whose sum could overflow is caught as well.  With the 8-bit state the host has checked that
    // dec(e) is too small to push a finite g to infinity.
    unsigned bad_bits;
    f32x2 g2[8];
    if (GRAD == GRAD_BF16) {
#pragma unroll
        for (int k = 0; k < 8; ++k)
            g2[k] = pk2(__uint_as_float(in.g[k % GW] << 16), __uint_as_float(in.g[k % GW] & 0xffff0000u));
    } else {
#pragma unroll
        for (int k = 0; k < 8; ++k)
            g2[k] = pk2(__uint_as_float(in.g[(2 * k) % GW]), __uint_as_float(in.g[(2 * k + 1) % GW]));
    }
    if (GRAD == GRAD_BF16 && !kStateF32) {
        unsigned acc = 0u;
#pragma unroll
        for (int k = 0; k < 8; ++k) acc = hfma2_bf16(in.g[k % GW], 0u, acc);
        bad_bits = acc & 0x7fff7fffu;
    } else {
        f32x2 acc = zero2;
        const f32x2 four2 = dup2(4.0f);
#pragma unroll
        for (int k = 0; k < 8; ++k) acc = ffma2(kStateF32 ? fmul2(g2[k], four2) : g2[k], zero2, acc);
        if (kStateF32) {
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const f32x2 e2 = pk2(__uint_as_float(in.e[(2 * k) % EW]), __uint_as_float(in.e[(2 * k + 1) % EW]));
                acc = ffma2(fmul2(e2, four2), zero2, acc);
            }
        }
        bad_bits = (static_cast<unsigned>(acc) | static_cast<unsigned>(acc >> 32)) & 0x7fffffffu;
    }
    if (MODE != MODE_BLOCK) {
        if (__any_sync(kFull, bad_bits != 0u)) return false;
    }

    // ---- optional element-wise clipping of g (finite here, or the row is redone by the careful routine); the plain
    //      lean variants do not carry it, the host never launches one of them with clip > 0 ----------------------------
    if (EXTRAS && K.clip > 0.0f) {
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            float a, b;
            unpk2(g2[k], a, b);
            g2[k] = pk2(fminf(fmaxf(a, -K.clip), K.clip), fminf(fmaxf(b, -K.clip), K.clip));
        }
    }

    // ---- step 1, Eq. 2: c = what is added to g, prev = e~_k of Eq. 5, h = g + c -----------------------------
    f32x2 prev2[8], h2[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        f32x2 c2;
        if (STATE == ST_INT8) {
            const unsigned x = in.e[(k >> 1) % EW] ^ 0x80808080u;                                   // bytes e + 128
            const float m0 = __uint_as_float(__byte_perm(x, kMagicBits, 0x7650 + 2 * (k & 1)));     // kMagic + 128 + e
            const float m1 = __uint_as_float(__byte_perm(x, kMagicBits, 0x7651 + 2 * (k & 1)));
            if (MODE == MODE_BLOCK) {
                c2 = fmul2_pz(fadd2(pk2(m0, m1), dup2(-emagic)), dup2(in.sscale));   // kSignFree holds here
            } else {
                c2 = dec_state2<VAR>(K, pk2(m0, m1), emagic, de_mode);
            }
            prev2[k] = c2;
        } else if (kStateF32) {
            prev2[k] = pk2(__uint_as_float(in.e[(2 * k) % EW]), __uint_as_float(in.e[(2 * k + 1) % EW]));
            if (STATE == ST_FP32) {
                c2 = prev2[k];
            } else {
                float y0, y1;
                unpk2(fmul2(prev2[k], dup2(K.s_e)), y0, y1);
                if (EXTRAS && stats)             // nearest integer outside [-128, 127]: 127.5 goes up and out, -128.5 stays in
                    state_saturated += ((y0 >= 127.5f || y0 < -128.5f) ? 1u : 0u) + ((y1 >= 127.5f || y1 < -128.5f) ? 1u : 0u);
                const f32x2 m2 = fadd2(pk2(fminf(fmaxf(y0, -128.0f), 127.0f), fminf(fmaxf(y1, -128.0f), 127.0f)), dup2(emagic));
                c2 = dec_state2<VAR>(K, m2, emagic, de_mode);
            }
        } else {
            c2 = zero2;
            prev2[k] = zero2;
        }
        // g + 0 changes at most the sign of a zero, never a code; in block mode c is a product
        h2[k] = (STATE == ST_NONE) ? g2[k] : fadd2(g2[k], c2);
    }

    // ---- block scale (extension): absmax of the block's h over the lanes that share it ---------------------------
    float mult = K.s, scale = 0.0f;
    if (BITS == 1 && STATE != ST_INT8) {
        // the sign code sends +1 for -0 (h < 0 is false); adding +0 turns a -0 into +0 and changes nothing else.  With
        // the 8-bit state h = g + c is never -0, because c never is (a product or sum that cancels gives +0).
#pragma unroll
        for (int k = 0; k < 8; ++k) h2[k] = fadd2(h2[k], zero2);
    }
    if (MODE == MODE_BLOCK && BITS == 1) {
        // sign code: the block's magnitude is the mean of |h|, summed pairwise (a balanced tree over the block's positions)
        float a[16];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            unpk2(h2[k], a[2 * k], a[2 * k + 1]);
            a[2 * k] = fabsf(a[2 * k]);
            a[2 * k + 1] = fabsf(a[2 * k + 1]);
        }
#pragma unroll
        for (int w = 1; w < 16; w <<= 1) {
#pragma unroll
            for (int j = 0; j < 16; j += 2 * w) a[j] = __fadd_rn(a[j], a[j + w]);
        }
        float sum = group_sum32(a[0], lanes_per_block);
        if (WIDE) {                           // a NaN in place of the sum makes every warp of the block give up
            if (__any_sync(kFull, bad_bits != 0u)) sum = __uint_as_float(0x7fc00000u);
            sum = wide_exchange<true>(K, xphase, sum, lane);
        }
        // an overflowing h or sum leaves the row to the careful routine (which forms the same infinities the plain way)
        if (__any_sync(kFull, bad_bits != 0u || !(sum <= kFltMax))) return false;
        scale = __fmul_rn(sum, __uint_as_float(static_cast<unsigned>(127 - K.block_log2) << 23));     // sum / B, exact scaling
        mult = 0.0f;
    } else if (MODE == MODE_BLOCK) {
        float amax = 0.0f;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            float a, b;
            unpk2(h2[k], a, b);
            amax = fmaxf(amax, fmaxf(fabsf(a), fabsf(b)));
        }
        amax = group_max32(amax, lanes_per_block);
        if (WIDE) {                           // +Inf in place of the maximum makes every warp of the block give up
            if (__any_sync(kFull, bad_bits != 0u)) amax = __uint_as_float(0x7f800000u);
            amax = wide_exchange<false>(K, xphase, amax, lane);
        }
        // g is finite here, so h can only be +-Inf (an overflowing sum), never NaN, and the maximum shows it.  A block
        // maximum outside [2^-100, 2^100] (other than 0) also leaves the row to the careful routine, which divides.
        if (__any_sync(kFull, bad_bits != 0u || !(amax == 0.0f || in_midrange(amax)))) return false;
        scale = amax > 0.0f ? div_by_qmax(amax, hi, 1.0f / hi) : 0.0f;
        mult = amax > 0.0f ? qmax_over_midrange(hi, amax) : 0.0f;
    }

    // ---- Eq. 1 / Eq. 3: q = round_p-bit(h x s);  step 2: d, Eq. 5 ---------------------------------------------
    CodePacker<BITS == 1 ? 2 : BITS> pack;
    pack.clear();
    f32x2 en2[8];
    const f32x2 mult2 = dup2(mult), qmagic2 = dup2(qmagic), omb2 = dup2(K.omb), beta2 = dup2(K.beta);
    uint4 rnd = make_uint4(0u, 0u, 0u, 0u);                // the lane's 16 elements are one block of the Philox stream
    if (var_is_sr(VAR))
        rnd = sr_block((L.elem0 + static_cast<unsigned long long>(wrow) * kWide) >> 4, K.k_lo, K.k_hi, K.sr_keys);
    unsigned signs = 0u;                                   // sign code: bit j = 1 when element j is negative
    if (BITS == 1) {
        const unsigned mag = __float_as_uint(MODE == MODE_BLOCK ? scale : K.inv_s);     // d = q x mean|h|, or q / s = +-fl(1/s)
#pragma unroll
        for (int k = 7; k >= 0; --k) {
            const unsigned b0 = static_cast<unsigned>(h2[k]), b1 = static_cast<unsigned>(h2[k] >> 32);
            signs = __funnelshift_l(b0, __funnelshift_l(b1, signs, 1), 1);
            const f32x2 d2 = pk2(__uint_as_float(and_or(b0, 0x80000000u, mag)), __uint_as_float(and_or(b1, 0x80000000u, mag)));
            const f32x2 delta2 = fsub2(h2[k], d2);
            en2[k] = (STATE == ST_NONE) ? zero2
                     : (kSignFree ? fadd2(fmul2_pz(omb2, prev2[k]), fmul2_pz(beta2, delta2))
                                  : fadd2_after_mul(fmul2(omb2, prev2[k]), fmul2(beta2, delta2)));
        }
    }
#pragma unroll
    for (int k = (BITS == 1 ? -1 : 7); k >= 0; --k) {      // from the last pair down: the order the code packer wants
        float y0 = 0.0f, y1 = 0.0f, t0 = 0.0f, t1 = 0.0f;
        f32x2 m2;                                                                                    // kMagic + 2^(p-1) + q
        if (MODE == MODE_BLOCK && !var_is_sr(VAR)) {
            // |h| <= amax and mult = fl(qmax / amax), so |h x mult| <= qmax (1 + 2^-22): the nearest integer is inside the
            // range and the clamp of Eq. 1 has nothing to do.  The product as fma(h, mult, +0), so that the add of the
            // magic constant cannot be contracted with it (the sign of a zero product does not reach the sum).
            m2 = fadd2(fmul2_pz(h2[k], mult2), qmagic2);
        } else {
            if (var_is_sr(VAR)) {
                // floor(y + u): up with probability frac(y).  y + u is one rounded add; clamping it to [lo, hi + 1/2]
                // clamps its floor to [lo, hi]; adding the magic constant rounding DOWN leaves that floor in the mantissa
                const unsigned word = (k >> 1) == 0 ? rnd.x : ((k >> 1) == 1 ? rnd.y : ((k >> 1) == 2 ? rnd.z : rnd.w));
                const f32x2 mu2 = pk2(__uint_as_float(__byte_perm(word, 0x4B000000u, 0x7540 + 2 * (k & 1))),
                                      __uint_as_float(__byte_perm(word, 0x4B000000u, 0x7540 + 2 * (k & 1) + 1)));     // 2^23 + byte
                const f32x2 u2 = ffma2(mu2, dup2(0.00390625f), dup2(-32767.998046875f));               // byte / 256 + 1 / 512, exact
                unpk2(fadd2(fmul2_pz(h2[k], mult2), u2), t0, t1);             // the product as fma(h, s, +0): not contracted with the add
                m2 = fadd2_down(pk2(fminf(fmaxf(t0, lo), hi + 0.5f), fminf(fmaxf(t1, lo), hi + 0.5f)), qmagic2);
            } else {
                unpk2(fmul2(h2[k], mult2), y0, y1);
                t0 = y0;
                t1 = y1;
                m2 = fadd2(pk2(fminf(fmaxf(t0, lo), hi), fminf(fmaxf(t1, lo), hi)), qmagic2);
            }
        }
        const unsigned mb0 = static_cast<unsigned>(m2), mb1 = static_cast<unsigned>(m2 >> 32);
        pack.push(2 * k + 1, mb1);
        pack.push(2 * k, mb0);
        f32x2 d2;
        if (MODE == MODE_BLOCK) {
            d2 = fmul2_pz(fadd2(m2, dup2(-qmagic)), dup2(scale));          // q is never -0 and a non-zero q times a block scale never underflows
        } else if (LEAN) {
            d2 = ffma2(m2, dup2(K.dq_a), dup2(K.dq_b));
        } else {
            d2 = pk2(dec_fast(__uint_as_float(mb0), qmagic, dq_mode, K.dq_a, K.dq_b, K.s, K.inv_s),
                     dec_fast(__uint_as_float(mb1), qmagic, dq_mode, K.dq_a, K.dq_b, K.s, K.inv_s));
        }
        if (MODE != MODE_BLOCK && EXTRAS && stats) {
            if (var_is_sr(VAR)) {               // t = y + u before the floor: its floor leaves [lo, hi] iff t < lo or t >= hi + 1
                saturated += ((t0 < lo || t0 >= hi + 1.0f) ? 1u : 0u) + ((t1 < lo || t1 >= hi + 1.0f) ? 1u : 0u);
            } else {
                if (y0 >= hi + 0.5f || y0 < lo - 0.5f) saturated += 1u;
                if (y1 >= hi + 0.5f || y1 < lo - 0.5f) saturated += 1u;
            }
        }
        const f32x2 delta2 = fsub2(h2[k], d2);
        en2[k] = (STATE == ST_NONE) ? zero2
                 : (kSignFree ? fadd2(fmul2_pz(omb2, prev2[k]), fmul2_pz(beta2, delta2))
                              : fadd2_after_mul(fmul2(omb2, prev2[k]), fmul2(beta2, delta2)));
    }
    uint8_t *cdst = L.codes + static_cast<size_t>(wrow) * (kWide * BITS / 8);
    if (BITS == 4) {
        st_stream8(cdst, make_uint2(pack.word(0), pack.word(1)));
    } else if (BITS == 8) {
        st_stream16(cdst, make_uint4(pack.word(0), pack.word(1), pack.word(2), pack.word(3)));
    } else if (BITS == 2) {
        st_stream4(cdst, pack.word(0));
    } else {
        st_stream2(cdst, static_cast<uint16_t>(signs));
    }
    // the scales of wide row w: L.wire_scales / L.state_scales point at this lane's block of row 0
    if (MODE == MODE_BLOCK) {
        if (L.leader) L.wire_scales[scale_index<WIDE>(K, wrow)] = scale;
    }

    // ---- Eq. 7 ---------------------------------------------------------------------------------------------------
    if (STATE == ST_INT8) {
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        float escale = 0.0f;
        if (!K.reset) {
            float emult = K.s_e;
            if (MODE == MODE_BLOCK) {
                float amax = 0.0f;
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    float a, b;
                    unpk2(en2[k], a, b);
                    amax = fmaxf(amax, fmaxf(fabsf(a), fabsf(b)));
                }
                amax = group_max32(amax, lanes_per_block);
                if (WIDE) amax = wide_exchange<false>(K, xphase, amax, lane);
                // nothing of the state has been written yet, and the codes stored above are what the careful routine stores
                if (__any_sync(kFull, !(amax == 0.0f || in_midrange(amax)))) return false;
                escale = amax > 0.0f ? div_by_qmax(amax, 127.0f, 1.0f / 127.0f) : 0.0f;
                emult = amax > 0.0f ? qmax_over_midrange(127.0f, amax) : 0.0f;
            }
            const f32x2 emult2 = dup2(emult);
            int q[16];
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                float a, b;
                unpk2(fmul2(en2[k], emult2), a, b);
                if (MODE != MODE_BLOCK && EXTRAS && stats)      // codes that Eq. 7's 8-bit compressor clamps
                    state_saturated += ((a >= 127.5f || a < -128.5f) ? 1u : 0u) + ((b >= 127.5f || b < -128.5f) ? 1u : 0u);
                q[2 * k] = __float2int_rn(a);                   // saturates, NaN -> 0
                q[2 * k + 1] = __float2int_rn(b);
            }
            v.x = pack_sat_s8(q[0], q[1], pack_sat_s8(q[2], q[3], 0u));
            v.y = pack_sat_s8(q[4], q[5], pack_sat_s8(q[6], q[7], 0u));
            v.z = pack_sat_s8(q[8], q[9], pack_sat_s8(q[10], q[11], 0u));
            v.w = pack_sat_s8(q[12], q[13], pack_sat_s8(q[14], q[15], 0u));
        }
        st_stream16(L.state + static_cast<size_t>(wrow) * kWide, v);
        if (MODE == MODE_BLOCK) {
            if (L.leader) L.state_scales[scale_index<WIDE>(K, wrow)] = escale;
        }
    } else if (kStateF32) {
        unsigned w[16];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            w[2 * k] = K.reset ? 0u : static_cast<unsigned>(en2[k]);
            w[2 * k + 1] = K.reset ? 0u : static_cast<unsigned>(en2[k] >> 32);
        }
        uint8_t *dst = L.state + static_cast<size_t>(wrow) * (4u * kWide);   // 16-byte aligned by contract, not more
#pragma unroll
        for (int j = 0; j < 4; ++j) st_stream16(dst + 16 * j, make_uint4(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]));
    }
    return true;
}

// The lane's pointers for the wide rows of partition `part` of one bucket.
template <int STATE, int BITS>
__device__ __forceinline__ void lane_pointers(const SendBucket &Bk, uint8_t *pbase, unsigned long long part, int lane, LanePtrs &L) {
    L.lane_elem = static_cast<unsigned>(lane) * kWideLane;
    L.lane_block = 0u;
    L.leader = false;
    L.elem0 = part * Bk.lp + L.lane_elem;
    L.state = static_cast<uint8_t *>(Bk.state) + L.elem0 * (STATE == ST_INT8 ? 1u : 4u);
    L.codes = pbase + static_cast<size_t>(L.lane_elem) * BITS / 8;
    L.wire_scales = reinterpret_cast<float *>(pbase + Bk.lp * BITS / 8);
    L.state_scales = reinterpret_cast<float *>(static_cast<uint8_t *>(Bk.state) + ((Bk.n + 255ull) & ~255ull));
}

__device__ __forceinline__ void load_consts(const SendCommon &C, SendConsts &K) {
    K.s = C.s; K.s_e = C.s_e; K.beta = C.beta; K.omb = C.omb; K.inv_s = C.inv_s; K.inv_se = C.inv_se;
    K.dq_a = C.dq_a; K.dq_b = C.dq_b; K.de_a = C.de_a; K.de_b = C.de_b;
    K.dq_mode = C.dq_mode; K.de_mode = C.de_mode; K.block_log2 = C.block_log2; K.reset = C.reset; K.clip = C.clip;
    K.row_shl = C.block_log2 < 9 ? static_cast<unsigned>(9 - C.block_log2) : 0u;
    K.row_shr = C.block_log2 > 9 ? static_cast<unsigned>(C.block_log2 - 9) : 0u;
    K.group_warps = 1u;
    K.xslot = K.xgroup = 0u;
    K.bar_id = 0u;
    K.bar_threads = 32u;
    K.k_lo = C.k_lo; K.k_hi = C.k_hi; K.sr_keys = C.sr_keys;
}

// What a warp has counted goes to the bucket's status words: [0] flags, [1] saturated gradient codes, [2] saturated
// 8-bit error codes.
__device__ __forceinline__ void flush_counts(unsigned long long *status, bool collect, int lane, unsigned &saturated,
                                             unsigned &state_saturated, unsigned &nonfinite) {
    if (__any_sync(kFull, nonfinite != 0u)) {
        if (lane == 0) atomicOr(status, static_cast<unsigned long long>(kFlagNonFinite));
    }
    if (collect) {
        for (int o = 16; o > 0; o >>= 1) {
            saturated += __shfl_xor_sync(kFull, saturated, o);
            state_saturated += __shfl_xor_sync(kFull, state_saturated, o);
        }
        if (lane == 0 && saturated) atomicAdd(status + 1, static_cast<unsigned long long>(saturated));
        if (lane == 0 && state_saturated) atomicAdd(status + 2, static_cast<unsigned long long>(state_saturated));
    }
    saturated = 0u;
    state_saturated = 0u;
    nonfinite = 0u;
}

// The work of one CTA on partition `part` of one bucket: CTA `cta` of the `ctas` that share the partition.  Each warp walks
// the partition's wide rows with the stride of all warps working on that partition; the inputs of its next rows are on
// their way through the cp.async ring.  What is left of the partition (a last half-wide row, partial and padding rows;
// every block when a block is wider than a wide row) goes to the careful routine.
// `part_base()` gives where the partition's codes and scales go; it is asked again wherever the address is needed, so
// that the address does not occupy registers across the streaming loop.
template <int GRAD, int STATE, int BITS, int MODE, int VAR, typename PartBase>
__device__ __forceinline__ void send_bucket(const SendCommon &C, const SendBucket &Bk, PartBase part_base, unsigned long long part,
                                            unsigned cta, unsigned ctas) {
    using R = Ring<GRAD, STATE, MODE>;
    constexpr int D = R::kDepth;
    constexpr unsigned gbytes = (GRAD == GRAD_BF16 ? 2u : 4u) * kWide;       // gradient bytes of a wide row
    constexpr unsigned ebytes = (STATE == ST_INT8 ? 1u : 4u) * kWide;        // state bytes of a wide row
    extern __shared__ __align__(16) uint8_t ring[];
    const int lane = threadIdx.x & 31;
    const unsigned warp = cta * kWarps + (threadIdx.x >> 5);
    const unsigned nwarps = ctas * kWarps;
    const unsigned rows = static_cast<unsigned>(Bk.lp / kRow);               // 256-element rows of the partition
    const unsigned long long base = part * Bk.lp;
    // rows [0, full_rows) of this partition lie entirely below n
    unsigned full_rows = 0;
    if (Bk.n > base) {
        const unsigned long long avail = Bk.n - base;
        full_rows = avail >= Bk.lp ? rows : static_cast<unsigned>(avail / kRow);
    }
    unsigned saturated = 0u, state_saturated = 0u, nonfinite = 0u;
    auto careful = [&](unsigned long long o, int nrows) {
        const CarefulCounts N = send_careful<GRAD, STATE, BITS, MODE, var_is_sr(VAR)>(C, Bk, part_base(), part, o, nrows, lane);
        saturated += N.saturated;
        state_saturated += N.state_saturated;
        nonfinite |= N.nonfinite;
    };
    unsigned first_careful = 0u;             // first 256-element row left to the careful routine
    // a block of more than 512 elements spans G = B / 512 wide rows; the warps of a CTA hold 8 consecutive wide rows
    // at a time (warp w of every CTA takes the rows = w mod 8), so the G warps w, w + 1, ... with w a multiple of G hold
    // one block.  Only whole blocks go through the fast routine, so these warps do the same number of rows.
    constexpr bool WIDE = var_is_wide(VAR);
    const unsigned G = WIDE ? (1u << (C.block_log2 - 9)) : 1u;
    const unsigned warp_in_cta = threadIdx.x >> 5;
    __shared__ float wide_slots[WIDE ? 2 * kWarps : 1];
    if (C.fast) {
        const unsigned full_wide = (full_rows / 2) & ~(G - 1u);
        first_careful = 2 * full_wide;
        LanePtrs L;
        lane_pointers<STATE, BITS>(Bk, part_base(), part, lane, L);
        SendConsts K;
        load_consts(C, K);
        if (MODE == MODE_BLOCK) {
            // a wide row and a partition start on a block boundary (or inside the same block as the row's first element),
            // so which lane leads a block, and which block of its row a lane is in, never changes
            const unsigned lanes_per_block = C.block_log2 >= 9 ? 32u : (1u << (C.block_log2 - 4));
            L.leader = (static_cast<unsigned>(lane) & (lanes_per_block - 1u)) == 0u && (warp_in_cta & (G - 1u)) == 0u;
            L.lane_block = L.lane_elem >> C.block_log2;
            L.wire_scales += L.lane_block;
            L.state_scales += (L.elem0 >> C.block_log2);
            if (WIDE) {
                const unsigned slots = static_cast<unsigned>(__cvta_generic_to_shared(wide_slots));
                K.group_warps = G;
                K.xslot = slots + 4u * warp_in_cta;
                K.xgroup = slots + 4u * ((warp_in_cta & ~(G - 1u)) + (static_cast<unsigned>(lane) & (G - 1u)));
                K.bar_id = 1u + warp_in_cta / G;
                K.bar_threads = 32u * G;
            }
        }
        unsigned xphase = 0u;
        // staging reads: chunk `lane` of each 512-byte piece of the row
        const uint8_t *g_stage = static_cast<const uint8_t *>(Bk.grad) + base * (GRAD == GRAD_BF16 ? 2u : 4u) + lane * 16;
        const uint8_t *e_stage = static_cast<const uint8_t *>(Bk.state) + base * (STATE == ST_INT8 ? 1u : 4u) + lane * 16;
        const bool stats = C.collect_stats != 0;
        RingAddr<GRAD, STATE> A;
        ring_addresses<GRAD, STATE, MODE>(static_cast<unsigned>(__cvta_generic_to_shared(ring)), lane, threadIdx.x >> 5, A);
        // this warp's wide rows are warp + i * nwarps, i < cnt
        const unsigned cnt_all = full_wide > warp ? (full_wide - warp + nwarps - 1) / nwarps : 0u;
        const unsigned cnt = cnt_all < 32u ? cnt_all : 32u;        // the rows that stream through the fast routine
        auto stage = [&](unsigned slot_off, unsigned wrow) {
            const float *sp = L.state_scales + scale_index<WIDE>(K, wrow);                              // MODE_BLOCK only
            stage_row<GRAD, STATE, MODE>(A, slot_off, g_stage + static_cast<size_t>(wrow) * gbytes,
                                         e_stage + static_cast<size_t>(wrow) * ebytes, sp);
        };
#pragma unroll
        for (int i = 0; i < D - 1; ++i) {
            if (static_cast<unsigned>(i) < cnt) stage(i * R::kSlotStride, warp + i * nwarps);
            cp_async_commit();
        }
        unsigned slot_off = 0u, stage_off = (D - 1) * R::kSlotStride;
        unsigned wrow = warp, stage_wrow = warp + (D - 1) * nwarps;
        // Rows the fast routine hands back (a NaN, an Inf, a block maximum out of range: rare) are noted in a mask and
        // redone by the careful routine after the streaming loop: a call inside it, or between two runs of it, would
        // make the compiler keep part of the loop's registers in local memory.
        unsigned failed = 0u;
#pragma unroll 1
        for (unsigned i = 0; i < cnt; ++i) {
            cp_async_wait<D - 2>();            // every group but the newest D-2 has landed: this row is there
            __syncwarp();                      // ... for all lanes; and every lane is done reading the slot refilled next
            WideIn<GRAD, STATE> in;
            fetch_row<GRAD, STATE, MODE>(A, slot_off, in);
            if (i + (D - 1) < cnt) stage(stage_off, stage_wrow);
            cp_async_commit();                 // one group per iteration, empty near the end
            if (!send_wide_row<GRAD, STATE, BITS, MODE, VAR>(K, L, in, wrow, lane, stats, saturated, state_saturated, xphase))
                failed |= 1u << i;
            slot_off = slot_off + R::kSlotStride == R::kBytes ? 0u : slot_off + R::kSlotStride;
            stage_off = stage_off + R::kSlotStride == R::kBytes ? 0u : stage_off + R::kSlotStride;
            wrow += nwarps;
            stage_wrow += nwarps;
        }
        // every warp of a wide block noted the failure; the one that holds the block's first row redoes the block
        if ((warp_in_cta & (G - 1u)) == 0u) {
            while (failed) {
                const unsigned j = static_cast<unsigned>(__ffs(static_cast<int>(failed))) - 1u;
                failed &= failed - 1u;
                careful(static_cast<unsigned long long>(warp + j * nwarps) * kWide, static_cast<int>(2u * G));
            }
            // rows beyond what the mask can note: the host's grid leaves a warp about kRowsPerWarp rows, so there are none
            for (unsigned i = cnt; i < cnt_all; ++i)
                careful(static_cast<unsigned long long>(warp + i * nwarps) * kWide, static_cast<int>(2u * G));
        }
    }
    // the careful routine's unit: a row, or the rows of a block wider than a row
    const unsigned cu = (MODE == MODE_BLOCK && C.block_log2 > 8) ? (1u << (C.block_log2 - 8)) : 1u;
    for (unsigned u = first_careful / cu + warp; u * cu < rows; u += nwarps)
        careful(static_cast<unsigned long long>(u) * cu * kRow, static_cast<int>(cu));
    flush_counts(Bk.status, C.collect_stats != 0, lane, saturated, state_saturated, nonfinite);
}

// CTAs per SM the send kernels are compiled for: three with the global scale (80 registers per thread); the block-scaled
// form keeps a whole row's h and error in registers while the block maxima are formed and gets 120 registers (two CTAs).
template <int MODE> constexpr int kSendCtasPerSm = (MODE == MODE_BLOCK) ? 2 : 3;

// One bucket per launch: grid = (CTAs per partition, partitions).
// VAR_LEAN / VAR_LEAN_NR kernels are launched when the host proved the corresponding decompressor forms and neither
// statistics nor clipping are wanted (VAR_LEAN also for every block-scaled configuration), VAR_LEAN_X / VAR_LEAN_NR_X
// when they are; VAR_GENERAL chooses the decompressor forms at run time.
template <int GRAD, int STATE, int BITS, int MODE, int VAR>
__global__ void __launch_bounds__(kThreads, kSendCtasPerSm<MODE>) loco_send_kernel(const __grid_constant__ SendParams P) {
    const unsigned long long part = blockIdx.y;
    send_bucket<GRAD, STATE, BITS, MODE, VAR>(
        P.c, P.b, [&]() -> uint8_t * { return P.scatter ? P.part_dst[part] : P.b.comm + part * P.b.stride; }, part, blockIdx.x, gridDim.x);
}

// Several buckets per launch: grid = (most CTAs per partition any bucket wants, partitions, buckets).  The CTAs of
// bucket z do exactly what the one-bucket kernel's CTAs do; the hardware hands them to the SMs in order -- all of
// bucket 0, then bucket 1, ... -- as places become free, so an SM that streams faster than another simply receives
// more of them, no bucket boundary drains the machine, and the launch costs are paid once per call.  The table of
// buckets travels in the kernel's parameters.
template <int GRAD, int STATE, int BITS, int MODE, int VAR>
__global__ void __launch_bounds__(kThreads, kSendCtasPerSm<MODE>) loco_send_multi_kernel(const __grid_constant__ SendMultiParams P) {
    const SendBucket &Bk = P.b[blockIdx.z];
    if (blockIdx.x >= Bk.grid_x) return;
    const unsigned long long part = blockIdx.y;
    send_bucket<GRAD, STATE, BITS, MODE, VAR>(P.c, Bk, [&]() -> uint8_t * { return Bk.comm + part * Bk.stride; }, part, blockIdx.x, Bk.grid_x);
}

// ------------------------------------------------------------------------------------------
// receive: Eq. 8 on wide rows of 512 outputs, 16 per lane.

template <int BITS> struct WideCodes {                       // the 16 codes of one lane and wide row, as loaded
    static constexpr int W = BITS >= 2 ? BITS / 2 : 1;       // 32-bit words: 1 (sign code: its low half), 1, 2 or 4
    unsigned w[W];
};

template <int BITS>
__device__ __forceinline__ void load_codes(const uint8_t *src, WideCodes<BITS> &c) {
    if (BITS == 8) { const uint4 t = ld_stream16(src); c.w[0] = t.x; c.w[1 % WideCodes<BITS>::W] = t.y; c.w[2 % WideCodes<BITS>::W] = t.z; c.w[3 % WideCodes<BITS>::W] = t.w; }
    else if (BITS == 4) { const uint2 t = ld_stream8(src); c.w[0] = t.x; c.w[1 % WideCodes<BITS>::W] = t.y; }
    else if (BITS == 2) c.w[0] = ld_stream4(src);
    else c.w[0] = __ldcs(reinterpret_cast<const unsigned short *>(src));
}

// (a & b) ^ c in one instruction
__device__ __forceinline__ unsigned and_xor(unsigned a, unsigned b, unsigned c) {
    unsigned d;
    asm("lop3.b32 %0, %1, %2, %3, 0x6A;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
// Sign code: elements 2k and 2k+1 of a lane's 16 as +-mag (bit set = negative), mag >= 0 or any float whose sign
// the code may flip.
__device__ __forceinline__ f32x2 sign_pair(unsigned w, int k, unsigned mag) {
    const unsigned x0 = and_xor(w << (31 - 2 * k), 0x80000000u, mag);
    const unsigned x1 = and_xor(w << (30 - 2 * k), 0x80000000u, mag);
    return pk2(__uint_as_float(x0), __uint_as_float(x1));
}

// The magic float 2^e + (code + 2^(p-1)) of field j: the field, with its top bit already flipped in x, is masked in
// place into the mantissa of a power of two chosen so that the field's lowest bit weighs 1.  `k` receives that
// power of two plus the bias, i.e. what has to be subtracted to leave the code.
template <int BITS>
__device__ __forceinline__ float field_magic(const unsigned (&x)[WideCodes<BITS>::W], const unsigned (&xh)[WideCodes<BITS>::W], int j, float &k) {
    if (BITS == 8) {
        k = 8388608.0f + 128.0f;
        return __uint_as_float(__byte_perm(x[(j >> 2) % WideCodes<BITS>::W], 0x4B000000u, 0x7650 + (j & 3)));
    } else if (BITS == 4) {
        const int jj = j & 7;
        const int pos = jj < 5 ? jj : jj - 3;                // fields 5..7 are taken from the word shifted right by 12
        const unsigned src = jj < 5 ? x[(j >> 3) % WideCodes<BITS>::W] : xh[(j >> 3) % WideCodes<BITS>::W];
        const unsigned expo = static_cast<unsigned>(127 + 23 - 4 * pos) << 23;        // 2^(23 - 4 pos)
        k = __uint_as_float(expo) + 8.0f;
        return __uint_as_float(and_or(src, 0xFu << (4 * pos), expo));
    } else {
        const int pos = j < 11 ? j : j - 8;                  // fields 11..15 are taken from the word shifted right by 16
        const unsigned src = j < 11 ? x[0] : xh[0];
        const unsigned expo = static_cast<unsigned>(127 + 23 - 2 * pos) << 23;
        k = __uint_as_float(expo) + 2.0f;
        return __uint_as_float(and_or(src, 0x3u << (2 * pos), expo));
    }
}

__device__ __forceinline__ unsigned pack_bf16x2_rn(float a, float b) {
    // two fp32 -> two bf16 (round to nearest even), a in the low half
    unsigned r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(b), "f"(a));
    return r;
}

// 16 results of one lane to out[oi ..]; `left` = elements that exist from oi on; wide32: out + oi is 32-byte aligned.
template <int OUT>
__device__ __forceinline__ void store_out16(void *out, unsigned long long oi, const float (&res)[16], unsigned long long left, bool wide32) {
    if (left >= 16) {
        if (OUT == GRAD_BF16) {
            unsigned w[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) w[j] = pack_bf16x2_rn(res[2 * j], res[2 * j + 1]);
            uint16_t *dst = static_cast<uint16_t *>(out) + oi;
            if (wide32) {
                st_stream32(dst, w);
            } else {
                st_stream16(dst, make_uint4(w[0], w[1], w[2], w[3]));
                st_stream16(dst + 8, make_uint4(w[4], w[5], w[6], w[7]));
            }
        } else {
            unsigned w[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) w[j] = __float_as_uint(res[j]);
            float *dst = static_cast<float *>(out) + oi;
            if (wide32) {
                st_stream32(dst, w);
                st_stream32(dst + 8, w + 8);
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j) st_stream16(dst + 4 * j, make_uint4(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]));
            }
        }
    } else {
        const int cnt = static_cast<int>(left);
#pragma unroll
        for (int j = 0; j < 16; ++j) {
            if (j < cnt) {
                if (OUT == GRAD_BF16)
                    static_cast<uint16_t *>(out)[oi + j] = static_cast<uint16_t>(pack_bf16x2_rn(res[j], 0.0f) & 0xffffu);
                else
                    static_cast<float *>(out)[oi + j] = res[j];
            }
        }
    }
}

// acc / N as Eq. 8 writes it
__device__ __forceinline__ float div_workers(const ReduceCommon &C, float acc) {
    if (C.div_mode == 0) return __fmul_rn(acc, C.inv_n);
    if (C.div_mode == 1) {
        const float q0 = __fmul_rn(acc, C.inv_n);
        const float rem = __fmaf_rn(-q0, C.n_workers_f, acc);
        return __fmaf_rn(rem, C.inv_n, q0);
    }
    return __fdiv_rn(acc, C.n_workers_f);
}

// The paper's Adam-family step on the 16 averaged gradients of one lane (Algorithm 1 step 3: the update that
// consumes g~): m = (1-b1) m + b1 g; v = (1-b2) v + b2 g^2; theta -= eta / sqrt(v + delta) * m.  One IEEE fp32
// operation per written operation (scalar intrinsics: nothing is contracted), IEEE square root and division.
// The averaged gradient never goes through HBM unless the caller asks for it.
struct AdamRegs { float m[16], v[16], t[16]; };

// Start the loads of a lane's 16 moments and weights (issued before the workers' codes are summed, so that they
// are in flight meanwhile).  Only for lanes whose 16 elements all exist.
__device__ __forceinline__ void adam_load16(const ReduceCommon &C, unsigned long long oi, AdamRegs &R) {
    const float *pm = C.adam_m + oi, *pv = C.adam_v + oi, *pt = C.adam_theta + oi;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const uint4 a = ld_stream16(pm + 4 * j), b = ld_stream16(pv + 4 * j), c = ld_stream16(pt + 4 * j);
        R.m[4 * j] = __uint_as_float(a.x); R.m[4 * j + 1] = __uint_as_float(a.y); R.m[4 * j + 2] = __uint_as_float(a.z); R.m[4 * j + 3] = __uint_as_float(a.w);
        R.v[4 * j] = __uint_as_float(b.x); R.v[4 * j + 1] = __uint_as_float(b.y); R.v[4 * j + 2] = __uint_as_float(b.z); R.v[4 * j + 3] = __uint_as_float(b.w);
        R.t[4 * j] = __uint_as_float(c.x); R.t[4 * j + 1] = __uint_as_float(c.y); R.t[4 * j + 2] = __uint_as_float(c.z); R.t[4 * j + 3] = __uint_as_float(c.w);
    }
}

template <int OUT>
__device__ __forceinline__ void adam_finish16(const ReduceCommon &C, void *out, unsigned long long oi, const float (&g)[16],
                                              unsigned long long left, bool wide32, AdamRegs &R) {
    float *pm = C.adam_m + oi, *pv = C.adam_v + oi, *pt = C.adam_theta + oi;
    if (left >= 16) {                                    // R was loaded by adam_load16
#pragma unroll
        for (int j = 0; j < 16; ++j) {
            R.m[j] = __fadd_rn(__fmul_rn(C.omb1, R.m[j]), __fmul_rn(C.beta1, g[j]));
            R.v[j] = __fadd_rn(__fmul_rn(C.omb2, R.v[j]), __fmul_rn(C.beta2, __fmul_rn(g[j], g[j])));
            const float eta_k = __fdiv_rn(C.lr, __fsqrt_rn(__fadd_rn(R.v[j], C.delta)));
            R.t[j] = __fsub_rn(R.t[j], __fmul_rn(eta_k, R.m[j]));
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            st_stream16(pm + 4 * j, make_uint4(__float_as_uint(R.m[4 * j]), __float_as_uint(R.m[4 * j + 1]), __float_as_uint(R.m[4 * j + 2]), __float_as_uint(R.m[4 * j + 3])));
            st_stream16(pv + 4 * j, make_uint4(__float_as_uint(R.v[4 * j]), __float_as_uint(R.v[4 * j + 1]), __float_as_uint(R.v[4 * j + 2]), __float_as_uint(R.v[4 * j + 3])));
            st_stream16(pt + 4 * j, make_uint4(__float_as_uint(R.t[4 * j]), __float_as_uint(R.t[4 * j + 1]), __float_as_uint(R.t[4 * j + 2]), __float_as_uint(R.t[4 * j + 3])));
        }
    } else {
        const int cnt = static_cast<int>(left);
#pragma unroll
        for (int j = 0; j < 16; ++j) {
            if (j < cnt) {
                const float mk = __fadd_rn(__fmul_rn(C.omb1, pm[j]), __fmul_rn(C.beta1, g[j]));
                const float vk = __fadd_rn(__fmul_rn(C.omb2, pv[j]), __fmul_rn(C.beta2, __fmul_rn(g[j], g[j])));
                const float eta_k = __fdiv_rn(C.lr, __fsqrt_rn(__fadd_rn(vk, C.delta)));
                pm[j] = mk;
                pv[j] = vk;
                pt[j] = __fsub_rn(pt[j], __fmul_rn(eta_k, mk));
            }
        }
    }
    if (out) store_out16<OUT>(out, oi, g, left, wide32);
}

// Integer path (global power-of-two s, at most 16 workers): every dec(q; s) and every partial sum of Eq. 8
// is an integer multiple of 1/s that fp32 holds exactly, so the sum over workers does not depend on the
// order or the format it is taken in.  The codes, biased to be non-negative, are added side by side inside
// 32-bit words (8-bit lanes for 2- and 4-bit codes, 16-bit lanes for 8-bit codes); the lane sums S reach
// fp32 through the mantissa of kMagic and one fused multiply-add gives (S - bias N) / s (/ N).
// Sign code: a byte lane counts twice the negative workers of its element, 2c (a multiply spreads four wire bits to
// four bytes: bit i of a nibble times 0x00408102 lands, among others, on bit 8 i + 1, and no two bits meet), and the
// sum of the +-1 is N - 2c.
// three-input bit operations in one instruction each: a ^ b ^ c and the majority of a, b, c (a full adder on 32 positions at once)
__device__ __forceinline__ unsigned xor3(unsigned a, unsigned b, unsigned c) {
    unsigned d;
    asm("lop3.b32 %0, %1, %2, %3, 0x96;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
__device__ __forceinline__ unsigned maj3(unsigned a, unsigned b, unsigned c) {
    unsigned d;
    asm("lop3.b32 %0, %1, %2, %3, 0xE8;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}

template <int BITS>
struct WideSums {
    static constexpr int S = (BITS == 8) ? 8 : 4;
    static constexpr int P = (BITS == 1) ? 5 : 1;           // sign code: bit planes of the per-element count (at most 16 workers)
    unsigned s[S];
    unsigned p[P];
    __device__ __forceinline__ void clear() {
#pragma unroll
        for (int i = 0; i < S; ++i) s[i] = 0u;
#pragma unroll
        for (int i = 0; i < P; ++i) p[i] = 0u;
    }
    __device__ __forceinline__ void add(const WideCodes<BITS> &c) {
        if (BITS == 4) {            // s[2h] holds elements 8h + {0,2,4,6}, s[2h+1] elements 8h + {1,3,5,7}
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                s[(2 * h) % S] += xor_and(c.w[h % WideCodes<BITS>::W], 0x08080808u, 0x0F0F0F0Fu);
                s[(2 * h + 1) % S] += xor_and(c.w[h % WideCodes<BITS>::W] >> 4, 0x08080808u, 0x0F0F0F0Fu);
            }
        } else if (BITS == 8) {     // s[2h] holds elements 4h + {0,2}, s[2h+1] elements 4h + {1,3}, in 16-bit lanes
#pragma unroll
            for (int h = 0; h < 4; ++h) {
                s[(2 * h) % S] += xor_and(c.w[h % WideCodes<BITS>::W], 0x00800080u, 0x00FF00FFu);
                s[(2 * h + 1) % S] += xor_and(c.w[h % WideCodes<BITS>::W] >> 8, 0x00800080u, 0x00FF00FFu);
            }
        } else if (BITS == 2) {     // byte b of s[k] holds element 4b + k
#pragma unroll
            for (int k = 0; k < 4; ++k) s[k % S] += xor_and(c.w[0] >> (2 * k), 0x02020202u, 0x03030303u);
        } else {
            // sign code: the lane's word has one bit per element (1 = negative).  The number of negative workers of every
            // element is kept bit-sliced -- plane k holds bit k of all 16 counts -- so one worker costs a ripple of half
            // adders over the planes, eight logic instructions for 16 elements
            unsigned carry = c.w[0];
#pragma unroll
            for (int k = 0; k < P; ++k) {
                const unsigned t = p[k % P] & carry;
                p[k % P] ^= carry;
                carry = t;
            }
        }
    }
    // Sign code, four workers at once: two full adders fold them and plane 0 into a new plane 0 and two carries of weight 2,
    // a third folds those and plane 1, the rest ripples: eleven logic instructions for 64 wire bits.
    __device__ __forceinline__ void add4(const WideCodes<BITS> &a, const WideCodes<BITS> &b, const WideCodes<BITS> &c, const WideCodes<BITS> &d) {
        if (BITS != 1) {
            add(a); add(b); add(c); add(d);
        } else {
            const unsigned s1 = xor3(a.w[0], b.w[0], c.w[0]), c1 = maj3(a.w[0], b.w[0], c.w[0]);
            const unsigned c2 = maj3(s1, d.w[0], p[0]);
            p[0] = xor3(s1, d.w[0], p[0]);
            const unsigned c3 = maj3(c1, c2, p[1 % P]);
            p[1 % P] = xor3(c1, c2, p[1 % P]);
            const unsigned c4 = p[2 % P] & c3;
            p[2 % P] ^= c3;
            const unsigned c5 = p[3 % P] & c4;
            p[3 % P] ^= c4;
            p[4 % P] ^= c5;
        }
    }
    // Sign code: the planes become byte lanes once per row -- byte b of s[g] = 2 x (negative workers of element 4g + b).
    // A multiply spreads the four bits of a nibble to four bytes (bit i times 0x00408102 lands, among others, on bit
    // 8i + 1, and no two bits meet); plane k adds its spread nibble shifted by k.  `planes` = how many planes can be
    // non-zero (bit length of the worker count), the same for the whole launch.
    __device__ __forceinline__ void finalize(int planes) {
        if (BITS == 1) {
#pragma unroll
            for (int g = 0; g < 4; ++g) {
                unsigned acc = 0u;
#pragma unroll
                for (int k = 0; k < P; ++k) {
                    if (k < planes) acc += ((((p[k % P] >> (4 * g)) & 0xFu) * 0x00408102u) & 0x02020202u) << k;
                }
                s[g % S] = acc;
            }
        }
    }
    // kMagic + S_j as a float
    __device__ __forceinline__ float get(int j) const {
        if (BITS == 4) return __uint_as_float(__byte_perm(s[(2 * (j >> 3) + (j & 1)) % S], kMagicBits, 0x7650 + ((j & 7) >> 1)));
        if (BITS == 8) return __uint_as_float(__byte_perm(s[(2 * (j >> 2) + (j & 1)) % S], kMagicBits, ((j & 3) >> 1) ? 0x7632 : 0x7610));
        if (BITS == 1) return __uint_as_float(__byte_perm(s[(j >> 2) % S], kMagicBits, 0x7650 + (j & 3)));
        return __uint_as_float(__byte_perm(s[(j & 3) % S], kMagicBits, 0x7650 + (j >> 2)));
    }
};

// PATH_INT: the integer-sum path (only with the global scale); otherwise the generic path with dec(q; s) as a multiply
// (also the block-scaled form), as the Newton-Raphson division, or as the IEEE division.  Separate kernels, so that each
// path gets the registers and the occupancy it wants and no per-element choice is left.
enum : int { PATH_INT = 0, PATH_MUL = 1, PATH_NEWTON = 2, PATH_DIVIDE = 3 };

// The receive pass with the Adam-family update of the optimizer applied to the averaged gradient in the same pass.
// Its traffic is dominated by the lane's 48 optimizer words, which are loaded into registers at the start of a row;
// the codes are read with plain loads (one wide row at a time on the integer path, groups of four workers with the
// next group's loads in flight on the others).
template <int OUT, int BITS, int MODE, int PATH>
__global__ void __launch_bounds__(kThreads, 3) loco_reduce_adam_kernel(const __grid_constant__ ReduceParams P) {
    const ReduceCommon &C = P.c;
    const ReduceBucket &Bk = P.b;
    const uint8_t *const *parts = P.parts;
    constexpr unsigned kRowBytes = kWide * BITS / 8;                  // code bytes of one wide row
    const int lane = threadIdx.x & 31;
    const unsigned long long part = blockIdx.y;                       // relative to C.first
    const unsigned warp = blockIdx.x * kWarps + (threadIdx.x >> 5);
    const unsigned nwarps = gridDim.x * kWarps;
    const unsigned long long base = (C.first + part) * Bk.lp;          // first bucket element of the part
    if (base >= Bk.n) return;
    const unsigned long long avail = Bk.n - base;
    const unsigned long long valid = avail >= Bk.lp ? Bk.lp : avail;
    const unsigned rows = static_cast<unsigned>((valid + kWide - 1) / kWide);
    const unsigned long long poff = part * Bk.stride;
    const unsigned long long out0 = part * Bk.lp;                      // output index of the part's first element
    const unsigned lane_elem = static_cast<unsigned>(lane) * kWideLane;
    const unsigned lane_byte = lane_elem * BITS / 8;
    const int N = C.num_workers;
    const int count_planes = 32 - __clz(N);                            // sign code, integer path: bit length of a count of workers
    const bool wide32 = Bk.out_align32 != 0;

    if (PATH == PATH_INT) {
        // code areas below 4 GiB (checked by the host): row offsets fit 32 bits
        constexpr int kUnroll = 1;
        for (unsigned r = warp; r < rows; r += kUnroll * nwarps) {
            WideSums<BITS> sums[kUnroll];
            unsigned off[kUnroll];
            bool ok[kUnroll];
            AdamRegs AR;
            {
                const unsigned long long o = static_cast<unsigned long long>(r) * kWide + lane_elem;
                if (o + 16 <= valid) adam_load16(C, out0 + o, AR);
            }
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) {
                sums[u].clear();
                // a lane loads only if its 16 elements start below the part's valid length (they then lie inside the code area)
                ok[u] = (r + u * nwarps < rows) && (static_cast<unsigned long long>(r + u * nwarps) * kWide + lane_elem < valid);
                off[u] = (r + u * nwarps) * kRowBytes + lane_byte;
            }
#pragma unroll 4
            for (int w = 0; w < N; ++w) {
                const uint8_t *src = parts[w] + poff;
                WideCodes<BITS> cw[kUnroll];
#pragma unroll
                for (int u = 0; u < kUnroll; ++u) {
#pragma unroll
                    for (int i = 0; i < WideCodes<BITS>::W; ++i) cw[u].w[i] = 0u;
                    if (ok[u]) load_codes<BITS>(src + off[u], cw[u]);
                }
#pragma unroll
                for (int u = 0; u < kUnroll; ++u) sums[u].add(cw[u]);
            }
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) sums[u].finalize(count_planes);
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) {
                if (!ok[u]) continue;
                const unsigned long long o = static_cast<unsigned long long>(r + u * nwarps) * kWide + lane_elem;
                float res[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const float acc = __fmaf_rn(sums[u].get(j), C.ra, C.rb);
                    res[j] = C.div_mode == 0 ? acc : div_workers(C, acc);
                }
                adam_finish16<OUT>(C, Bk.out, out0 + o, res, valid - o, wide32, AR);
            }
        }
        return;
    }

    // Generic path: dec(q) and the sum in worker order, each operation rounded as Eq. 8 and Eq. 1 state them.
    // PATH_MUL: q * (1/s) equals q / s for every code (or block scales: q * scale); PATH_NEWTON: Newton-Raphson
    // division, checked on the host for every code; PATH_DIVIDE: IEEE division.
    // The workers of a row are taken four at a time; while one group is being summed, the loads of the next group
    // (of this row or of the warp's next row) are already in flight.
    constexpr int kGroup = 4;
    struct Group {
        WideCodes<BITS> c[kGroup];
        float sc[kGroup];
    };
    const int groups = (N + kGroup - 1) / kGroup;
    auto load_group = [&](unsigned row, int g, Group &G) {
        const unsigned long long o = static_cast<unsigned long long>(row) * kWide + lane_elem;
        const bool in = row < rows && o < valid;
        const unsigned long long off = static_cast<unsigned long long>(row) * kRowBytes + lane_byte;    // a part's code area may exceed 4 GiB
        const unsigned long long sidx = o >> C.block_log2;
#pragma unroll
        for (int i = 0; i < kGroup; ++i) {
            const int w = g * kGroup + i;
#pragma unroll
            for (int t = 0; t < WideCodes<BITS>::W; ++t) G.c[i].w[t] = 0u;
            G.sc[i] = C.gen_mul;
            if (in && w < N) {
                const uint8_t *wbase = parts[w] + poff;
                load_codes<BITS>(wbase + off, G.c[i]);
                if (MODE == MODE_BLOCK) G.sc[i] = __ldg(reinterpret_cast<const float *>(wbase + Bk.code_bytes) + sidx);
            }
        }
    };
    const f32x2 inv2 = dup2(C.inv_s), negs2 = dup2(-C.s);
    Group cur;
    if (warp < rows) load_group(warp, 0, cur);
    for (unsigned r = warp; r < rows; r += nwarps) {
        const unsigned long long o = static_cast<unsigned long long>(r) * kWide + lane_elem;
        f32x2 acc2[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) acc2[i] = 0ull;
        AdamRegs AR;
        if (o + 16 <= valid) adam_load16(C, out0 + o, AR);
        for (int g = 0; g < groups; ++g) {
            Group nxt;
            if (g + 1 < groups) load_group(r, g + 1, nxt);
            else load_group(r + nwarps, 0, nxt);
#pragma unroll
            for (int i = 0; i < kGroup; ++i) {
                if (g * kGroup + i >= N) break;
                if (BITS == 1) {                 // sign code: d = +-scale, exact; the sum in worker order
                    const unsigned mag = __float_as_uint(cur.sc[i]);
#pragma unroll
                    for (int k = 0; k < 8; ++k) acc2[k] = fadd2(acc2[k], sign_pair(cur.c[i].w[0], k, mag));
                } else {
                unsigned x[WideCodes<BITS>::W], xh[WideCodes<BITS>::W];
#pragma unroll
                for (int t = 0; t < WideCodes<BITS>::W; ++t) {
                    x[t] = cur.c[i].w[t] ^ (BITS == 8 ? 0x80808080u : (BITS == 4 ? 0x88888888u : 0xAAAAAAAAu));
                    xh[t] = x[t] >> (BITS == 4 ? 12 : 16);
                }
                const f32x2 sc2 = dup2(cur.sc[i]);
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    float k0, k1;
                    const float m0 = field_magic<BITS>(x, xh, 2 * k, k0);
                    const float m1 = field_magic<BITS>(x, xh, 2 * k + 1, k1);
                    const f32x2 q2 = fadd2(pk2(m0, m1), pk2(-k0, -k1));                 // the two codes, exact
                    if (PATH == PATH_MUL) {
                        acc2[k] = fadd2(acc2[k], fmul2_pz(q2, sc2));                 // product and sum rounded separately
                    } else if (PATH == PATH_NEWTON) {
                        const f32x2 q0 = fmul2(q2, inv2);
                        const f32x2 rem = ffma2(q0, negs2, q2);
                        acc2[k] = fadd2(acc2[k], ffma2(rem, inv2, q0));
                    } else {
                        float a, b, c, d;
                        unpk2(q2, a, b);
                        unpk2(acc2[k], c, d);
                        acc2[k] = pk2(__fadd_rn(c, __fdiv_rn(a, C.s)), __fadd_rn(d, __fdiv_rn(b, C.s)));
                    }
                }
                }
            }
            cur = nxt;
        }
        if (o >= valid) continue;
        float res[16];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            float a, b;
            unpk2(acc2[i], a, b);
            res[2 * i] = div_workers(C, a);                                          // the 1/N of Eq. 8
            res[2 * i + 1] = div_workers(C, b);
        }
        adam_finish16<OUT>(C, Bk.out, out0 + o, res, valid - o, wide32, AR);
    }
}

// ------------------------------------------------------------------------------------------
// The receive pass with the workers' codes travelling through a per-warp cp.async ring.
//
// The unit of the ring is a group of up to 4 entries (entry = one worker's wide row: 512 codes, and in block mode
// the scales of its blocks): with N >= 4 workers a group is 4 workers of one row (a row takes ceil(N/4) groups),
// with fewer workers it is all workers of 4/N rows, so that the bytes in flight per warp do not shrink with N.
// All copies are 16 bytes wide (the narrower forms of cp.async move fewer bytes per instruction and are slower):
// a 16-byte chunk holds the codes of 16 / (2 BITS) lanes, so one copy instruction of the warp fills 1, 2 or 4
// entries (with the sign code, 16 lanes fill the 4 entries of a group), and cp.async.wait_group followed by __syncwarp() orders every lane's reads after all lanes' copies.
// One cp.async group per ring group; the ring holds kGroups of them, kGroups - 1 are in flight while one is summed.
template <int BITS, int MODE> struct RecvRing {
    static constexpr unsigned kLaneBytes = 2u * BITS;                       // the 16 codes of one lane
    static constexpr unsigned kCodeBytes = 32u * kLaneBytes;                // one worker's wide row
    static constexpr unsigned kEntry = kCodeBytes + (MODE == MODE_BLOCK ? 64u : 0u);   // + up to 16 block scales
    static constexpr unsigned kGroupBytes = 4u * kEntry;
    static constexpr unsigned kWarpBytes = 8192u;
    static constexpr int kGroups = (kWarpBytes / kGroupBytes) > 8u ? 8 : static_cast<int>(kWarpBytes / kGroupBytes);
    static constexpr unsigned kCtaBytes = kWarps * kGroups * kGroupBytes;
    static constexpr int kLanesPerEntry = static_cast<int>(kCodeBytes / 16u);   // 16-byte chunks of an entry: 4 (sign code), 8, 16, 32
    static constexpr int kEntriesPerCopy = 32 / kLanesPerEntry > 4 ? 4 : 32 / kLanesPerEntry;   // entries one copy instruction fills: 4 (half the lanes idle), 4, 2, 1
    static constexpr int kCopies = 4 / kEntriesPerCopy;                     // copy instructions per group: 1, 1, 2, 4
    static constexpr unsigned kChunkElems = 128u / BITS;                    // codes in a 16-byte chunk
    static_assert(kGroups >= 3, "the ring must hold at least three groups");
};

// The work of one CTA on part `part` (relative to C.first) of one bucket: CTA `cta` of the `ctas` that share the part.
template <int OUT, int BITS, int MODE, int PATH>
__device__ __forceinline__ void reduce_bucket(const ReduceCommon &C, const ReduceBucket &Bk, const uint8_t *const *parts,
                                              unsigned long long part, unsigned cta, unsigned ctas) {
    using R = RecvRing<BITS, MODE>;
    constexpr int G = R::kGroups;
    constexpr unsigned kRowBytes = kWide * BITS / 8;                  // code bytes of one wide row
    extern __shared__ __align__(16) uint8_t ring[];
    const int lane = threadIdx.x & 31;
    const unsigned warp = cta * kWarps + (threadIdx.x >> 5);
    const unsigned nwarps = ctas * kWarps;
    const unsigned long long base = (C.first + part) * Bk.lp;          // first bucket element of the part
    if (base >= Bk.n) return;
    const unsigned long long avail = Bk.n - base;
    const unsigned long long valid = avail >= Bk.lp ? Bk.lp : avail;
    const unsigned rows = static_cast<unsigned>((valid + kWide - 1) / kWide);
    const unsigned long long poff = part * Bk.stride;
    const unsigned long long out0 = part * Bk.lp;                      // output index of the part's first element
    const unsigned lane_elem = static_cast<unsigned>(lane) * kWideLane;
    const unsigned lane_byte = static_cast<unsigned>(lane) * R::kLaneBytes;
    const int N = C.num_workers;
    const int count_planes = 32 - __clz(N);                            // sign code, integer path: bit length of a count of workers
    const bool wide32 = Bk.out_align32 != 0;
    const int WG = N < 4 ? N : 4;                                      // workers per group
    const int group_entries = (4 / WG) * WG;                            // 4, 4, 3, 4: (rows per group) x C
    const unsigned row_step = static_cast<unsigned>(4 / WG) * nwarps;  // a group's rows are r, r + nwarps, ...
    const unsigned my_ring = static_cast<unsigned>(__cvta_generic_to_shared(ring)) +
                             (threadIdx.x >> 5) * (G * R::kGroupBytes);

    // What this lane copies for a group: in copy instruction i it serves entry j = i * kEntriesPerCopy + lane / kLanesPerEntry
    // (entry j = worker j % C of the group's row j / C) with the 16-byte chunk lane % kLanesPerEntry of that entry's codes.
    // Per copy the lane keeps: where it goes in the ring group, which worker of the group it reads, the two limits that
    // decide whether there is anything to copy (w0 < cp_lim: the worker exists; p_row < cp_rowlim: the chunk lies below the
    // part's valid length), and the running byte offset of the chunk inside a worker's part.
    const unsigned full_rows = static_cast<unsigned>(valid / kWide);  // rows all of whose 512 elements exist
    const unsigned tail = static_cast<unsigned>(valid - static_cast<unsigned long long>(full_rows) * kWide);   // elements of the partial row
    unsigned cp_dst[R::kCopies], cp_rowlim[R::kCopies];
    int cp_w[R::kCopies], cp_lim[R::kCopies];
    unsigned long long cp_off[R::kCopies];
#pragma unroll
    for (int i = 0; i < R::kCopies; ++i) {
        const int j = i * R::kEntriesPerCopy + lane / R::kLanesPerEntry;
        const unsigned chunk = static_cast<unsigned>(lane % R::kLanesPerEntry);
        const int rr = WG == 1 ? j : (WG == 2 ? (j >> 1) : 0);
        const unsigned row_off = static_cast<unsigned>(rr) * nwarps;
        const unsigned lim_row = full_rows + (chunk * R::kChunkElems < tail ? 1u : 0u);
        cp_w[i] = j - rr * WG;
        cp_lim[i] = j < group_entries ? N - cp_w[i] : 0;
        cp_rowlim[i] = lim_row > row_off ? lim_row - row_off : 0u;
        cp_dst[i] = static_cast<unsigned>(j) * R::kEntry + chunk * 16u;
        cp_off[i] = poff + static_cast<unsigned long long>(warp + row_off) * kRowBytes + chunk * 16u;
    }
    // block mode: copy instruction i (of 2) brings the scales of entries 2i and 2i+1, lane % 16 = block within the row
    // (a block wider than a wide row has one scale that all its rows fetch: the scale's index comes from the row's
    // first element each time, not from a running offset)
    int sc_w[2], sc_lim[2];
    unsigned sc_rowlim[2], sc_dst[2], sc_row[2];
    unsigned long long sc_base[2];
    if (MODE == MODE_BLOCK) {
        const unsigned bpr = static_cast<unsigned>(kWide) >> C.block_log2;
        const unsigned blocks_per_row = bpr ? bpr : 1u;
        const unsigned idx = static_cast<unsigned>(lane & 15);
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const int j = 2 * i + (lane >> 4);
            const int rr = WG == 1 ? j : (WG == 2 ? (j >> 1) : 0);
            const unsigned row_off = static_cast<unsigned>(rr) * nwarps;
            const unsigned lim_row = full_rows + ((idx << C.block_log2) < tail ? 1u : 0u);
            sc_w[i] = j - rr * WG;
            sc_lim[i] = (j < group_entries && idx < blocks_per_row) ? N - sc_w[i] : 0;
            sc_rowlim[i] = lim_row > row_off ? lim_row - row_off : 0u;
            sc_dst[i] = static_cast<unsigned>(j) * R::kEntry + R::kCodeBytes + 4u * idx;
            sc_row[i] = warp + row_off;
            sc_base[i] = poff + Bk.code_bytes + 4ull * idx;
        }
    }
    const unsigned long long code_step = static_cast<unsigned long long>(row_step) * kRowBytes;             // per advance of p_row

    // producer: this warp's groups in order -- rows warp, warp + row_step, ...; within a row its chunks of C workers
    unsigned p_row = warp, p_slot = 0u, c_slot = 0u;
    int p_w0 = 0;                                                      // first worker of the producer's chunk
    auto produce = [&]() {                     // one cp.async group per call, empty past the end
        const unsigned dst = my_ring + p_slot * R::kGroupBytes;
#pragma unroll
        for (int i = 0; i < R::kCopies; ++i)
            if (p_w0 < cp_lim[i] && p_row < cp_rowlim[i]) cp_async16(dst + cp_dst[i], parts[p_w0 + cp_w[i]] + cp_off[i]);
        if (MODE == MODE_BLOCK) {
#pragma unroll
            for (int i = 0; i < 2; ++i)
                if (p_w0 < sc_lim[i] && p_row < sc_rowlim[i])
                    cp_async4(dst + sc_dst[i], parts[p_w0 + sc_w[i]] + sc_base[i] +
                                                   4ull * ((static_cast<unsigned long long>(sc_row[i]) * kWide) >> C.block_log2));
        }
        cp_async_commit();
        p_w0 += WG;
        if (p_w0 >= N) {
            p_w0 = 0;
            p_row += row_step;
#pragma unroll
            for (int i = 0; i < R::kCopies; ++i) cp_off[i] += code_step;
            if (MODE == MODE_BLOCK) {
#pragma unroll
                for (int i = 0; i < 2; ++i) sc_row[i] += row_step;
            }
        }
        p_slot = p_slot + 1 == static_cast<unsigned>(G) ? 0u : p_slot + 1;
    };

    WideSums<BITS> sums;                                              // PATH_INT
    f32x2 acc2[8];                                                    // the other paths
    const f32x2 inv2 = dup2(C.inv_s), negs2 = dup2(-C.s);
    const unsigned scale_off = R::kCodeBytes + 4u * (lane_elem >> C.block_log2);      // this lane's scale within an entry

    auto begin_row = [&]() {
        if (PATH == PATH_INT) sums.clear();
        else {
#pragma unroll
            for (int i = 0; i < 8; ++i) acc2[i] = 0ull;
        }
    };
    auto fetch = [&](unsigned entry, WideCodes<BITS> &cw, float &scale) {             // this lane's codes (and scale) of an entry
        if (BITS == 8) { const uint4 t = lds16(entry + lane_byte); cw.w[0] = t.x; cw.w[1 % WideCodes<BITS>::W] = t.y; cw.w[2 % WideCodes<BITS>::W] = t.z; cw.w[3 % WideCodes<BITS>::W] = t.w; }
        else if (BITS == 4) { const uint2 t = lds8(entry + lane_byte); cw.w[0] = t.x; cw.w[1 % WideCodes<BITS>::W] = t.y; }
        else if (BITS == 2) cw.w[0] = lds4(entry + lane_byte);
        else cw.w[0] = lds2(entry + lane_byte);
        scale = (PATH != PATH_INT && MODE == MODE_BLOCK) ? __uint_as_float(lds4(entry + scale_off)) : C.gen_mul;
    };
    auto accumulate = [&](const WideCodes<BITS> &cw, float scale) {                   // one worker's codes into the row's sums
        if (PATH == PATH_INT) {
            sums.add(cw);
        } else if (BITS == 1) {
            // sign code: d = +-scale (the global magnitude fl(1/s), or the worker's block scale); exact, then the sum in worker order
            const unsigned mag = __float_as_uint(scale);
#pragma unroll
            for (int k = 0; k < 8; ++k) acc2[k] = fadd2(acc2[k], sign_pair(cw.w[0], k, mag));
        } else {
            unsigned x[WideCodes<BITS>::W], xh[WideCodes<BITS>::W];
#pragma unroll
            for (int t = 0; t < WideCodes<BITS>::W; ++t) {
                x[t] = cw.w[t] ^ (BITS == 8 ? 0x80808080u : (BITS == 4 ? 0x88888888u : 0xAAAAAAAAu));
                xh[t] = x[t] >> (BITS == 4 ? 12 : 16);
            }
            const f32x2 sc2 = dup2(scale);
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                float k0, k1;
                const float m0 = field_magic<BITS>(x, xh, 2 * k, k0);
                const float m1 = field_magic<BITS>(x, xh, 2 * k + 1, k1);
                const f32x2 q2 = fadd2(pk2(m0, m1), pk2(-k0, -k1));                 // the two codes, exact
                if (PATH == PATH_MUL) {
                    acc2[k] = fadd2(acc2[k], fmul2_pz(q2, sc2));                 // product and sum rounded separately
                } else if (PATH == PATH_NEWTON) {
                    const f32x2 q0 = fmul2(q2, inv2);
                    const f32x2 rem = ffma2(q0, negs2, q2);
                    acc2[k] = fadd2(acc2[k], ffma2(rem, inv2, q0));
                } else {
                    float a, b, cc, d;
                    unpk2(q2, a, b);
                    unpk2(acc2[k], cc, d);
                    acc2[k] = pk2(__fadd_rn(cc, __fdiv_rn(a, C.s)), __fadd_rn(d, __fdiv_rn(b, C.s)));
                }
            }
        }
    };
    auto finish_row = [&](unsigned long long o) {                                    // the 1/N of Eq. 8 and the store
        if (o >= valid) return;
        float res[16];
        if (PATH == PATH_INT) {
            sums.finalize(count_planes);
#pragma unroll
            for (int i = 0; i < 16; ++i) res[i] = __fmaf_rn(sums.get(i), C.ra, C.rb);
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) unpk2(acc2[i], res[2 * i], res[2 * i + 1]);
        }
        // one branch per row, not per element: which form the division by N takes is the same for the whole launch
        if (PATH != PATH_INT && C.div_mode == 0) {
#pragma unroll
            for (int i = 0; i < 16; ++i) res[i] = __fmul_rn(res[i], C.inv_n);
        } else if (C.div_mode == 1) {
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const float q0 = __fmul_rn(res[i], C.inv_n);
                const float rem = __fmaf_rn(-q0, C.n_workers_f, res[i]);
                res[i] = __fmaf_rn(rem, C.inv_n, q0);
            }
        } else if (C.div_mode == 2) {
#pragma unroll
            for (int i = 0; i < 16; ++i) res[i] = __fdiv_rn(res[i], C.n_workers_f);
        }
        store_out16<OUT>(Bk.out, out0 + o, res, valid - o, wide32);
    };

    auto next_group = [&]() -> unsigned {      // wait for the oldest group, refill the slot summed last, return the group's ring address
        cp_async_wait<G - 2>();                // all groups but the newest G-2 have landed
        __syncwarp();                          // ... for all lanes; and all lanes are done with the slot that is refilled now
        produce();
        const unsigned src = my_ring + c_slot * R::kGroupBytes;
        c_slot = c_slot + 1 == static_cast<unsigned>(G) ? 0u : c_slot + 1;
        return src;
    };
#pragma unroll 1
    for (int i = 0; i < G - 1; ++i) produce();

    if (N >= 4) {
        // a group = 4 workers (fewer in a row's last group) of one row
#pragma unroll 1
        for (unsigned row = warp; row < rows; row += nwarps) {
            const unsigned long long o = static_cast<unsigned long long>(row) * kWide + lane_elem;
            begin_row();
#pragma unroll 1
            for (int left = N; left > 0; left -= 4) {
                const unsigned src = next_group();
                if (left >= 4) {
                    WideCodes<BITS> cw[4];
                    float sc[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) fetch(src + e * R::kEntry, cw[e], sc[e]);
                    if (PATH == PATH_INT && BITS == 1) {
                        sums.add4(cw[0], cw[1], cw[2], cw[3]);
                    } else {
#pragma unroll
                        for (int e = 0; e < 4; ++e) accumulate(cw[e], sc[e]);
                    }
                } else {
#pragma unroll 1
                    for (int e = 0; e < left; ++e) {
                        WideCodes<BITS> cw;
                        float sc;
                        fetch(src + e * R::kEntry, cw, sc);
                        accumulate(cw, sc);
                    }
                }
            }
            finish_row(o);
        }
    } else {
        // a group = all N workers of 4 / N rows
#pragma unroll 1
        for (unsigned r0 = warp; r0 < rows; r0 += row_step) {
            unsigned src = next_group();
#pragma unroll 1
            for (unsigned row = r0; row < rows && row < r0 + row_step; row += nwarps) {
                const unsigned long long o = static_cast<unsigned long long>(row) * kWide + lane_elem;
                begin_row();
#pragma unroll 1
                for (int e = 0; e < N; ++e) {
                    WideCodes<BITS> cw;
                    float sc;
                    fetch(src, cw, sc);
                    accumulate(cw, sc);
                    src += R::kEntry;
                }
                finish_row(o);
            }
        }
    }
    cp_async_wait<0>();
}

// One bucket per launch: grid = (CTAs per part, parts).
template <int OUT, int BITS, int MODE, int PATH>
__global__ void __launch_bounds__(kThreads, 3) loco_reduce_kernel(const __grid_constant__ ReduceParams P) {
    reduce_bucket<OUT, BITS, MODE, PATH>(P.c, P.b, P.parts, blockIdx.y, blockIdx.x, gridDim.x);
}

// Several buckets per launch: grid = (most CTAs per part any bucket wants, parts, buckets); see loco_send_multi_kernel.
template <int OUT, int BITS, int MODE, int PATH>
__global__ void __launch_bounds__(kThreads, 3) loco_reduce_multi_kernel(const __grid_constant__ ReduceMultiParams P) {
    const ReduceBucket &Bk = P.b[blockIdx.z];
    if (blockIdx.x >= Bk.grid_x) return;
    reduce_bucket<OUT, BITS, MODE, PATH>(P.c, Bk, P.parts + blockIdx.z * P.c.num_workers, blockIdx.y, blockIdx.x, Bk.grid_x);
}

}  // namespace loco
