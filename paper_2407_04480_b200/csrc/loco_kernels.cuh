// LoCo send / receive kernels for sm_100a.
//
// Both passes are elementwise streams over HBM (no contraction, no tensor cores).
// Work unit: a "row" of 256 consecutive elements handled by one warp, 8 consecutive
// elements per lane, so that the widest stream (the gradient) moves as one 128-bit
// access per lane and every warp-wide access covers one contiguous span of memory.
// A warp takes ROWS rows per trip and issues all their loads before the arithmetic.
//
// Rounding discipline: every floating-point step of Algorithm 1 is one IEEE fp32
// operation rounded to nearest even, written with the __f*_rn intrinsics so that the
// compiler can never contract a multiply and an add into an FMA.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace loco {

enum : int { GRAD_F32 = 0, GRAD_BF16 = 1 };
enum : int { ST_INT8 = 0, ST_FP32 = 1, ST_NONE = 2, ST_Q8COMP = 3 };
// MODE_FIXED_RCP: global scales whose reciprocals reproduce Eq. 1's division bit for bit
// on every possible code (checked on the host); MODE_FIXED_DIV: IEEE division;
// MODE_BLOCK: per-block absmax scales.
enum : int { MODE_FIXED_RCP = 0, MODE_FIXED_DIV = 1, MODE_BLOCK = 2 };

constexpr int kRow = 256;          // elements per warp row
constexpr int kLaneElems = 8;      // elements per lane per row
constexpr int kThreads = 256;      // threads per CTA
constexpr int kWarps = kThreads / 32;
constexpr float kMagic = 12582912.0f;   // 1.5 * 2^23: adding it rounds to an integer, ties to even
constexpr float kFltMax = 3.402823466e+38f;
constexpr unsigned kFlagNonFinite = 1u;

struct SendParams {
    const void *grad;
    void *state;
    uint8_t *comm;
    unsigned long long n;            // bucket elements
    unsigned long long lp;           // elements per partition (multiple of 256 and of B)
    unsigned long long stride;       // bytes per partition
    unsigned long long code_bytes;   // bytes of the code area of a partition
    unsigned long long state_scale_off;   // byte offset of the state scales (BLOCK + INT8)
    float s, inv_s, s_e, inv_se, beta, omb;
    int block_log2;                  // log2(B), BLOCK mode
    int reset;                       // k % T_c == 0
    int collect_stats;
    unsigned long long *status;      // [0] flags, [1] saturated codes
};

struct ReduceParams {
    const uint8_t *parts[64];        // partition `first` of each worker
    void *out;
    unsigned long long n, lp, stride, code_bytes;
    unsigned long long first;        // first partition
    int num_workers;
    int block_log2;
    float s, inv_s, n_workers_f, inv_n;
    int inv_n_exact;                 // multiplying by inv_n equals dividing by N for all sums
};

// ------------------------------------------------------------------------------------------
// small helpers

template <int BITS> struct QRange {
    static constexpr float lo = -float(1 << (BITS - 1));
    static constexpr float hi = float((1 << (BITS - 1)) - 1);
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

__device__ __forceinline__ float warp_group_max(float v, int lanes) {
    // max over aligned groups of `lanes` lanes (power of two, <= 32)
    for (int o = 1; o < lanes; o <<= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

template <int GRAD>
__device__ __forceinline__ void load_grad8(const void *grad, unsigned long long i, float (&g)[8]) {
    if (GRAD == GRAD_BF16) {
        const uint4 v = __ldg(reinterpret_cast<const uint4 *>(static_cast<const uint16_t *>(grad) + i));
        const unsigned w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            g[2 * j] = __uint_as_float(w[j] << 16);
            g[2 * j + 1] = __uint_as_float(w[j] & 0xffff0000u);
        }
    } else {
        const float4 a = __ldg(reinterpret_cast<const float4 *>(static_cast<const float *>(grad) + i));
        const float4 b = __ldg(reinterpret_cast<const float4 *>(static_cast<const float *>(grad) + i) + 1);
        g[0] = a.x; g[1] = a.y; g[2] = a.z; g[3] = a.w;
        g[4] = b.x; g[5] = b.y; g[6] = b.z; g[7] = b.w;
    }
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

// ------------------------------------------------------------------------------------------
// send: Algorithm 1 steps 1-2 on 8 elements held by one lane.
//
//  g      gradient values (already fp32)
//  prev   e~_k as Eq. 5 sees it;  c  what is added to g (dec(e_k), e~_k, or dec(comp(e~_k)))
//  valid  number of leading elements that exist (8 on the fast path)
//  Outputs: code bits (low byte of each word = code), e_new = e~_{k+1}, scale of the block.
template <int STATE, int BITS, int MODE>
__device__ __forceinline__ void send_core(const SendParams &P, const float (&g)[8], const float (&c)[8],
                                          const float (&prev)[8], int valid, int lanes_per_block,
                                          unsigned (&code)[8], float (&e_new)[8], float &scale,
                                          unsigned &nonfinite, unsigned &saturated) {
    constexpr float lo = QRange<BITS>::lo, hi = QRange<BITS>::hi;
    float h[8];
    bool fin[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        h[j] = __fadd_rn(g[j], c[j]);                       // step 1 / Eq. 2
        fin[j] = fabsf(h[j]) <= kFltMax;                    // false for NaN and +-Inf
        if (!fin[j] && j < valid) nonfinite = 1u;
    }
    float mult = P.s;
    scale = 0.0f;
    if (MODE == MODE_BLOCK) {
        float amax = 0.0f;
#pragma unroll
        for (int j = 0; j < 8; ++j) amax = fmaxf(amax, fin[j] ? fabsf(h[j]) : 0.0f);
        amax = warp_group_max(amax, lanes_per_block);
        scale = amax > 0.0f ? __fdiv_rn(amax, hi) : 0.0f;
        mult = amax > 0.0f ? __fdiv_rn(hi, amax) : 0.0f;
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const float hq = (h[j] != h[j]) ? 0.0f : h[j];      // NaN is sent as code 0
        float y = __fmul_rn(hq, mult);                      // h x s of Eq. 1
        if (!fin[j]) y = hq;                                // +-Inf saturates whatever the scale
        const float r = round_clamp(y, lo, hi, code[j]);    // round_p-bit
        float d;                                            // step 2: dec(q; s)
        if (MODE == MODE_FIXED_RCP) d = __fmul_rn(r, P.inv_s);
        else if (MODE == MODE_FIXED_DIV) d = __fdiv_rn(r, P.s);
        else d = __fmul_rn(r, scale);
        const float delta = fin[j] ? __fsub_rn(h[j], d) : 0.0f;
        e_new[j] = __fadd_rn(__fmul_rn(P.omb, prev[j]), __fmul_rn(P.beta, delta));   // Eq. 5
        if (MODE != MODE_BLOCK && P.collect_stats) {
            // nearest integer outside the range: y >= hi + 1/2 (hi is odd, the tie goes up and out)
            // or y < lo - 1/2 (lo is even, the tie stays in)
            if (fin[j] && j < valid && (y >= hi + 0.5f || y < lo - 0.5f)) saturated += 1u;
        }
    }
}

// Eq. 7 for 8 elements in the int8 format: codes of e~_{k+1} (or zeros at a reset).
template <int MODE>
__device__ __forceinline__ void state_compress8(const SendParams &P, const float (&e_new)[8], int lanes_per_block,
                                                unsigned (&ebits)[8], float &escale) {
    float mult = P.s_e;
    escale = 0.0f;
    if (MODE == MODE_BLOCK) {
        float amax = 0.0f;
#pragma unroll
        for (int j = 0; j < 8; ++j) amax = fmaxf(amax, fabsf(e_new[j]));
        amax = warp_group_max(amax, lanes_per_block);
        escale = amax > 0.0f ? __fdiv_rn(amax, 127.0f) : 0.0f;
        mult = amax > 0.0f ? __fdiv_rn(127.0f, amax) : 0.0f;
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        (void)round_clamp(__fmul_rn(e_new[j], mult), -128.0f, 127.0f, ebits[j]);
    }
}

__device__ __forceinline__ unsigned pack4_bytes(unsigned a, unsigned b, unsigned c, unsigned d) {
    // low bytes of a, b, c, d -> one word, a lowest
    return __byte_perm(__byte_perm(a, b, 0x0040), __byte_perm(c, d, 0x0040), 0x5410);
}

// Compensation value and Eq. 5's previous error for 8 elements, from the stored state.
template <int STATE, int MODE>
__device__ __forceinline__ void decode_state8(const SendParams &P, uint2 e8, const float (&ef)[8], float sscale,
                                              float (&c)[8], float (&prev)[8]) {
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        if (STATE == ST_INT8) {
            const float ei = byte_to_float(j < 4 ? e8.x : e8.y, j & 3);
            if (MODE == MODE_FIXED_RCP) c[j] = __fmul_rn(ei, P.inv_se);       // dec(e_k; s_e), Eq. 2
            else if (MODE == MODE_FIXED_DIV) c[j] = __fdiv_rn(ei, P.s_e);
            else c[j] = __fmul_rn(ei, sscale);
            prev[j] = c[j];
        } else if (STATE == ST_FP32) {
            c[j] = ef[j];
            prev[j] = ef[j];
        } else if (STATE == ST_Q8COMP) {
            prev[j] = ef[j];
            unsigned bits;
            const float r = round_clamp(__fmul_rn(ef[j], P.s_e), -128.0f, 127.0f, bits);
            c[j] = (MODE == MODE_FIXED_RCP) ? __fmul_rn(r, P.inv_se) : __fdiv_rn(r, P.s_e);
        } else {
            c[j] = 0.0f;
            prev[j] = 0.0f;
        }
    }
}

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
    } else {
        unsigned w = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) w |= (code[j] & 0x3u) << (2 * j);
        *reinterpret_cast<uint16_t *>(dst) = static_cast<uint16_t>(w);
    }
}

// One warp row (256 elements starting at partition-local offset `o`, bucket element i0 = part*lp + o).
// FULL: all 256 elements exist; otherwise elements >= n are treated as absent (code 0, no state).
template <int GRAD, int STATE, int BITS, int MODE, bool FULL>
__device__ __forceinline__ void send_row(const SendParams &P, unsigned long long part, unsigned long long o,
                                         int lane, unsigned &nonfinite, unsigned &saturated) {
    const unsigned long long i0 = part * P.lp + o + static_cast<unsigned long long>(lane) * kLaneElems;
    int valid = 8;
    if (!FULL) {
        valid = i0 >= P.n ? 0 : (P.n - i0 >= 8 ? 8 : static_cast<int>(P.n - i0));
    }
    const int lanes_per_block = (MODE == MODE_BLOCK) ? (P.block_log2 >= 8 ? 32 : (1 << (P.block_log2 - 3))) : 1;
    const unsigned long long blk = (MODE == MODE_BLOCK) ? (i0 >> P.block_log2) : 0;

    float g[8], ef[8], c[8], prev[8];
    uint2 e8 = make_uint2(0u, 0u);
    float sscale = 0.0f;
    int8_t *st8 = static_cast<int8_t *>(P.state);
    float *stf = static_cast<float *>(P.state);
    float *st_scales = reinterpret_cast<float *>(static_cast<uint8_t *>(P.state) + P.state_scale_off);

    if (FULL) {
        load_grad8<GRAD>(P.grad, i0, g);
        if (STATE == ST_INT8) e8 = *reinterpret_cast<const uint2 *>(st8 + i0);
        if (STATE == ST_FP32 || STATE == ST_Q8COMP) {
            const float4 a = *reinterpret_cast<const float4 *>(stf + i0);
            const float4 b = *(reinterpret_cast<const float4 *>(stf + i0) + 1);
            ef[0] = a.x; ef[1] = a.y; ef[2] = a.z; ef[3] = a.w;
            ef[4] = b.x; ef[5] = b.y; ef[6] = b.z; ef[7] = b.w;
        }
    } else {
        unsigned lo_w = 0, hi_w = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            g[j] = 0.0f;
            ef[j] = 0.0f;
            if (j < valid) {
                g[j] = load_grad1<GRAD>(P.grad, i0 + j);
                if (STATE == ST_INT8) {
                    const unsigned b = static_cast<uint8_t>(st8[i0 + j]);
                    if (j < 4) lo_w |= b << (8 * j); else hi_w |= b << (8 * (j - 4));
                }
                if (STATE == ST_FP32 || STATE == ST_Q8COMP) ef[j] = stf[i0 + j];
            }
        }
        e8 = make_uint2(lo_w, hi_w);
    }
    if (STATE == ST_INT8 && MODE == MODE_BLOCK) sscale = (FULL || valid > 0) ? st_scales[blk] : 0.0f;

    decode_state8<STATE, MODE>(P, e8, ef, sscale, c, prev);

    unsigned code[8];
    float e_new[8], scale;
    send_core<STATE, BITS, MODE>(P, g, c, prev, valid, lanes_per_block, code, e_new, scale, nonfinite, saturated);

    // codes (and the block's scale) into the partition's areas of the communication buffer
    uint8_t *pbase = P.comm + part * P.stride;
    const unsigned long long ol = o + static_cast<unsigned long long>(lane) * kLaneElems;
    store_codes8<BITS>(pbase + ol * BITS / 8, code);
    if (MODE == MODE_BLOCK) {
        if ((lane & (lanes_per_block - 1)) == 0 && ((ol & ((1ull << P.block_log2) - 1)) == 0))
            *reinterpret_cast<float *>(pbase + P.code_bytes + (ol >> P.block_log2) * 4) = scale;
    }

    // Eq. 7: reset, or keep / compress the new error
    if (STATE == ST_NONE) return;
    if (STATE == ST_INT8) {
        unsigned ebits[8];
        float escale = 0.0f;
        if (P.reset) {
#pragma unroll
            for (int j = 0; j < 8; ++j) ebits[j] = 0u;
        } else {
            state_compress8<MODE>(P, e_new, lanes_per_block, ebits, escale);
        }
        if (FULL) {
            uint2 v;
            v.x = pack4_bytes(ebits[0], ebits[1], ebits[2], ebits[3]);
            v.y = pack4_bytes(ebits[4], ebits[5], ebits[6], ebits[7]);
            *reinterpret_cast<uint2 *>(st8 + i0) = v;
        } else {
#pragma unroll
            for (int j = 0; j < 8; ++j)
                if (j < valid) st8[i0 + j] = static_cast<int8_t>(ebits[j] & 0xffu);
        }
        if (MODE == MODE_BLOCK) {
            if ((lane & (lanes_per_block - 1)) == 0 && (i0 & ((1ull << P.block_log2) - 1)) == 0 && (FULL || valid > 0))
                st_scales[blk] = escale;
        }
    } else {
        if (P.reset) {
#pragma unroll
            for (int j = 0; j < 8; ++j) e_new[j] = 0.0f;
        }
        if (FULL) {
            *reinterpret_cast<float4 *>(stf + i0) = make_float4(e_new[0], e_new[1], e_new[2], e_new[3]);
            *(reinterpret_cast<float4 *>(stf + i0) + 1) = make_float4(e_new[4], e_new[5], e_new[6], e_new[7]);
        } else {
#pragma unroll
            for (int j = 0; j < 8; ++j)
                if (j < valid) stf[i0 + j] = e_new[j];
        }
    }
}

// grid = (ctas per partition, partitions).  Each warp walks the partition's rows with the
// stride of all warps working on that partition.
template <int GRAD, int STATE, int BITS, int MODE>
__global__ void __launch_bounds__(kThreads) loco_send_kernel(const SendParams P) {
    const int lane = threadIdx.x & 31;
    const unsigned long long part = blockIdx.y;
    const unsigned long long warp = static_cast<unsigned long long>(blockIdx.x) * kWarps + (threadIdx.x >> 5);
    const unsigned long long nwarps = static_cast<unsigned long long>(gridDim.x) * kWarps;
    const unsigned long long rows = P.lp / kRow;
    const unsigned long long base = part * P.lp;
    // rows [0, full_rows) of this partition lie entirely below n
    unsigned long long full_rows = 0;
    if (P.n > base) {
        const unsigned long long avail = P.n - base;
        full_rows = avail >= P.lp ? rows : avail / kRow;
    }
    unsigned nonfinite = 0u, saturated = 0u;
    for (unsigned long long r = warp; r < rows; r += nwarps) {
        if (r < full_rows) send_row<GRAD, STATE, BITS, MODE, true>(P, part, r * kRow, lane, nonfinite, saturated);
        else send_row<GRAD, STATE, BITS, MODE, false>(P, part, r * kRow, lane, nonfinite, saturated);
    }
    if (__any_sync(0xffffffffu, nonfinite != 0u)) {
        if (lane == 0) atomicOr(P.status, static_cast<unsigned long long>(kFlagNonFinite));
    }
    if (P.collect_stats) {
        for (int o = 16; o > 0; o >>= 1) saturated += __shfl_xor_sync(0xffffffffu, saturated, o);
        if (lane == 0 && saturated) atomicAdd(P.status + 1, static_cast<unsigned long long>(saturated));
    }
}

// ------------------------------------------------------------------------------------------
// receive: Eq. 8 on one warp row of 256 outputs, 8 per lane.

template <int BITS>
__device__ __forceinline__ void load_codes8(const uint8_t *src, float (&q)[8]) {
    if (BITS == 8) {
        const uint2 v = __ldg(reinterpret_cast<const uint2 *>(src));
#pragma unroll
        for (int j = 0; j < 8; ++j) q[j] = byte_to_float(j < 4 ? v.x : v.y, j & 3);
    } else if (BITS == 4) {
        const unsigned w = __ldg(reinterpret_cast<const unsigned *>(src));
#pragma unroll
        for (int j = 0; j < 8; ++j) q[j] = __int2float_rn(static_cast<int>(w << (28 - 4 * j)) >> 28);
    } else {
        const unsigned w = __ldg(reinterpret_cast<const uint16_t *>(src));
#pragma unroll
        for (int j = 0; j < 8; ++j) q[j] = __int2float_rn(static_cast<int>(w << (30 - 2 * j)) >> 30);
    }
}

__device__ __forceinline__ unsigned pack_bf16x2_rn(float a, float b) {
    // two fp32 -> two bf16 (round to nearest even), a in the low half
    unsigned r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(b), "f"(a));
    return r;
}

template <int OUT, int BITS, int MODE>
__global__ void __launch_bounds__(kThreads) loco_reduce_kernel(const ReduceParams P) {
    const int lane = threadIdx.x & 31;
    const unsigned long long part = blockIdx.y;                       // relative to P.first
    const unsigned long long warp = static_cast<unsigned long long>(blockIdx.x) * kWarps + (threadIdx.x >> 5);
    const unsigned long long nwarps = static_cast<unsigned long long>(gridDim.x) * kWarps;
    const unsigned long long base = (P.first + part) * P.lp;          // first bucket element of the part
    if (base >= P.n) return;
    const unsigned long long avail = P.n - base;
    const unsigned long long valid = avail >= P.lp ? P.lp : avail;
    const unsigned long long rows = (valid + kRow - 1) / kRow;
    const unsigned long long poff = part * P.stride;
    const unsigned long long out0 = part * P.lp;                      // output index of the part's first element

    for (unsigned long long r = warp; r < rows; r += nwarps) {
        const unsigned long long o = r * kRow + static_cast<unsigned long long>(lane) * kLaneElems;
        if (o >= valid) continue;
        float acc[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[j] = 0.0f;
#pragma unroll 4
        for (int w = 0; w < P.num_workers; ++w) {
            const uint8_t *src = P.parts[w] + poff;
            float q[8];
            load_codes8<BITS>(src + o * BITS / 8, q);
            float sc = 0.0f;
            if (MODE == MODE_BLOCK)
                sc = __ldg(reinterpret_cast<const float *>(src + P.code_bytes) + (o >> P.block_log2));
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                float d;                                               // dec(q; s), Eq. 1
                if (MODE == MODE_FIXED_RCP) d = __fmul_rn(q[j], P.inv_s);
                else if (MODE == MODE_FIXED_DIV) d = __fdiv_rn(q[j], P.s);
                else d = __fmul_rn(q[j], sc);
                acc[j] = __fadd_rn(acc[j], d);
            }
        }
        float res[8];
#pragma unroll
        for (int j = 0; j < 8; ++j)                                    // the 1/N of Eq. 8
            res[j] = P.inv_n_exact ? __fmul_rn(acc[j], P.inv_n) : __fdiv_rn(acc[j], P.n_workers_f);
        const unsigned long long oi = out0 + o;
        if (valid - o >= 8) {
            if (OUT == GRAD_BF16) {
                uint4 v;
                v.x = pack_bf16x2_rn(res[0], res[1]);
                v.y = pack_bf16x2_rn(res[2], res[3]);
                v.z = pack_bf16x2_rn(res[4], res[5]);
                v.w = pack_bf16x2_rn(res[6], res[7]);
                *reinterpret_cast<uint4 *>(static_cast<uint16_t *>(P.out) + oi) = v;
            } else {
                float4 *dst = reinterpret_cast<float4 *>(static_cast<float *>(P.out) + oi);
                dst[0] = make_float4(res[0], res[1], res[2], res[3]);
                dst[1] = make_float4(res[4], res[5], res[6], res[7]);
            }
        } else {
            const int cnt = static_cast<int>(valid - o);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                if (j < cnt) {
                    if (OUT == GRAD_BF16)
                        static_cast<uint16_t *>(P.out)[oi + j] = static_cast<uint16_t>(pack_bf16x2_rn(res[j], 0.0f) & 0xffffu);
                    else
                        static_cast<float *>(P.out)[oi + j] = res[j];
                }
            }
        }
    }
}

}  // namespace loco
