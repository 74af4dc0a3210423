// C ABI of the LoCo hot-path library: argument checks, layout arithmetic, kernel dispatch.
// See include/loco.h for the contract of every entry point.
#include "../../include/loco.h"

#include <atomic>
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>

#include "loco_dispatch.h"

namespace loco {

// mismatch[0]: amax / c, mismatch[1]: c / amax, over all positive finite floats, for c = 1, 7, 127
__global__ void loco_division_selfcheck_kernel(unsigned long long *mismatch) {
    const float cs[3] = {1.0f, 7.0f, 127.0f};
    unsigned long long bad0 = 0, bad1 = 0;
    for (unsigned long long b = blockIdx.x * static_cast<unsigned long long>(blockDim.x) + threadIdx.x + 1; b <= 0x7f7fffffull;
         b += static_cast<unsigned long long>(gridDim.x) * blockDim.x) {
        const float a = __uint_as_float(static_cast<unsigned>(b));
#pragma unroll
        for (int i = 0; i < 3; ++i) {
            const float c = cs[i];
            if (__float_as_uint(div_by_qmax(a, c, __frcp_rn(c))) != __float_as_uint(__fdiv_rn(a, c))) ++bad0;
            if (__float_as_uint(qmax_over(c, a)) != __float_as_uint(__fdiv_rn(c, a))) ++bad1;
            if (in_midrange(a) && __float_as_uint(qmax_over_midrange(c, a)) != __float_as_uint(__fdiv_rn(c, a))) ++bad1;
        }
    }
    if (bad0) atomicAdd(mismatch, bad0);
    if (bad1) atomicAdd(mismatch + 1, bad1);
}

}  // namespace loco

namespace {

using namespace loco;

std::atomic<uint64_t> g_launches{0};

inline uint64_t round_up(uint64_t x, uint64_t m) { return (x + m - 1) / m * m; }
inline bool is_pow2(uint64_t x) { return x && !(x & (x - 1)); }
inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline int ilog2(uint32_t x) { int l = 0; while ((1u << l) < x) ++l; return l; }
constexpr size_t kStatusBytes = 32;      // device status words of a handle: flags, saturated codes, saturated error codes, spare

int check_config(const loco_config_t *c) {
    if (!c) return LOCO_ERR_ARG;
    if (c->bits != 1 && c->bits != 2 && c->bits != 4 && c->bits != 8) return LOCO_ERR_ARG;
    if (c->scale_mode != LOCO_SCALE_FIXED && c->scale_mode != LOCO_SCALE_BLOCK_ABSMAX) return LOCO_ERR_ARG;
    if (c->state_fmt < LOCO_STATE_INT8 || c->state_fmt > LOCO_STATE_FP32_Q8COMP) return LOCO_ERR_ARG;
    if (c->scale_mode == LOCO_SCALE_BLOCK_ABSMAX) {
        const int b = c->block_size;
        if (b < 32 || b > 4096 || !is_pow2(static_cast<uint64_t>(b))) return LOCO_ERR_ARG;
        if (c->state_fmt == LOCO_STATE_FP32_Q8COMP) return LOCO_ERR_ARG;
    } else {
        if (!(c->s > 0.0f) || !std::isfinite(c->s)) return LOCO_ERR_ARG;
        if (c->state_fmt == LOCO_STATE_INT8 || c->state_fmt == LOCO_STATE_FP32_Q8COMP)
            if (!(c->s_e > 0.0f) || !std::isfinite(c->s_e)) return LOCO_ERR_ARG;
    }
    if (c->state_fmt != LOCO_STATE_NONE && !(c->beta >= 0.0f && c->beta <= 1.0f)) return LOCO_ERR_ARG;
    if (c->reset_period < 0) return LOCO_ERR_ARG;
    if (c->grad_dtype != LOCO_F32 && c->grad_dtype != LOCO_BF16) return LOCO_ERR_ARG;
    if (c->out_dtype != LOCO_F32 && c->out_dtype != LOCO_BF16) return LOCO_ERR_ARG;
    if (c->num_partitions < 1 || c->num_partitions > 65535) return LOCO_ERR_ARG;
    if (!(c->clip >= 0.0f) || !std::isfinite(c->clip)) return LOCO_ERR_ARG;
    if (c->rounding != LOCO_ROUND_NEAREST && c->rounding != LOCO_ROUND_STOCHASTIC) return LOCO_ERR_ARG;
    if (c->bits == 1 && c->rounding != LOCO_ROUND_NEAREST) return LOCO_ERR_ARG;      // a sign code has nothing to round
    return LOCO_OK;
}

// Layout arithmetic accepts every well-formed configuration, also those the kernels do not cover.
bool layout_ok(const loco_config_t *c) {
    const int rc = check_config(c);
    return rc == LOCO_OK || rc == LOCO_ERR_UNSUPPORTED;
}

struct Layout {
    uint64_t lp, code_bytes, scale_bytes, stride;
};

Layout make_layout(const loco_config_t *c, uint64_t n) {
    Layout L{0, 0, 0, 0};
    if (n == 0) return L;
    uint64_t unit = kRow;
    if (c->scale_mode == LOCO_SCALE_BLOCK_ABSMAX && static_cast<uint64_t>(c->block_size) > unit)
        unit = static_cast<uint64_t>(c->block_size);
    const uint64_t per = (n + static_cast<uint64_t>(c->num_partitions) - 1) / static_cast<uint64_t>(c->num_partitions);
    L.lp = round_up(per, unit);
    L.code_bytes = L.lp * static_cast<uint64_t>(c->bits) / 8;
    L.scale_bytes = c->scale_mode == LOCO_SCALE_BLOCK_ABSMAX ? (L.lp / static_cast<uint64_t>(c->block_size)) * 4 : 0;
    L.stride = round_up(L.code_bytes + L.scale_bytes, 128);
    return L;
}

uint64_t state_bytes(const loco_config_t *c, uint64_t n) {
    if (n == 0) return 0;
    switch (c->state_fmt) {
    case LOCO_STATE_NONE: return 0;
    case LOCO_STATE_INT8: {
        uint64_t b = round_up(n, 256);
        if (c->scale_mode == LOCO_SCALE_BLOCK_ABSMAX)
            b += round_up(((n + static_cast<uint64_t>(c->block_size) - 1) / static_cast<uint64_t>(c->block_size)) * 4, 256);
        return b;
    }
    default: return round_up(n * 4, 256);
    }
}

inline bool same_bits(float a, float b) { return std::memcmp(&a, &b, 4) == 0; }

// The kernels replace Eq. 1's division  code / scale  by cheaper sequences, but only when the sequence
// gives the bits of the IEEE division for EVERY code it can meet; these routines run that check.
// `bias` is what the kernel adds to the code inside the magic float: m = kMagic + bias + code.
struct DecChoice { int mode; float a, b, inv; };

DecChoice choose_dec(float scale, int lo, int hi, int bias) {
    DecChoice c{DEC_DIVIDE, 0.0f, 0.0f, 0.0f};
    const volatile float vinv = 1.0f / scale;
    const float inv = vinv;
    c.inv = inv;
    if (!std::isfinite(inv) || inv == 0.0f) return c;
    const float base = kMagic + static_cast<float>(bias);           // exact: an integer below 2^24
    const volatile float vb = -base * inv;
    const float a = inv, b = vb;
    bool fma_ok = std::isfinite(b), nr_ok = true;
    for (int q = lo; q <= hi; ++q) {
        const volatile float vwant = static_cast<float>(q) / scale;
        const float want = vwant;
        const float m = base + static_cast<float>(q);                // exact
        if (fma_ok && !same_bits(std::fmaf(m, a, b), want)) fma_ok = false;
        if (nr_ok) {
            const float cq = m - base;                               // exact
            const volatile float vq0 = cq * inv;
            const float q0 = vq0;
            const float rem = std::fmaf(-q0, scale, cq);
            if (!same_bits(std::fmaf(rem, inv, q0), want)) nr_ok = false;
        }
    }
    if (fma_ok) { c.mode = DEC_FMA; c.a = a; c.b = b; }
    else if (nr_ok) c.mode = DEC_NEWTON;
    return c;
}

// A multiplier m with fl(q * m) == fl(q / scale) for every integer q in [lo, hi]: fl(1/scale) or one of its
// neighbours (for a handful of small codes such an m very often exists even when 1/scale itself rounds badly).
bool exact_multiplier(float scale, int lo, int hi, float *mul) {
    const volatile float vinv = 1.0f / scale;
    const float inv = vinv;
    if (!std::isfinite(inv) || inv <= 0.0f) return false;
    uint32_t bits;
    std::memcpy(&bits, &inv, 4);
    for (int step = 0; step <= 8; ++step) {
        for (int sign = -1; sign <= 1; sign += 2) {
            if (step == 0 && sign > 0) continue;
            const uint32_t cand_bits = bits + static_cast<uint32_t>(sign * step);
            float cand;
            std::memcpy(&cand, &cand_bits, 4);
            if (!std::isfinite(cand) || cand <= 0.0f) continue;
            bool ok = true;
            for (int q = lo; q <= hi && ok; ++q) {
                const volatile float a = static_cast<float>(q) * cand;
                const volatile float b = static_cast<float>(q) / scale;
                ok = same_bits(a, b);
            }
            if (ok) { *mul = cand; return true; }
        }
    }
    return false;
}

bool is_pow2_float(float x) {
    uint32_t u;
    std::memcpy(&u, &x, 4);
    const uint32_t expo = (u >> 23) & 0xffu;
    return (u >> 31) == 0 && (u & 0x7fffffu) == 0 && expo >= 27 && expo <= 227;    // 2^-100 .. 2^100
}

int kernel_mode(const loco_config_t *c) {
    return c->scale_mode == LOCO_SCALE_BLOCK_ABSMAX ? MODE_BLOCK : MODE_FIXED;
}

// SMs of the current device (asked for once per device)
int num_sms() {
    static std::atomic<int> sms[64];
    int dev = 0, v = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0) { cudaGetLastError(); return 148; }
    if (dev < 64 && (v = sms[dev].load(std::memory_order_relaxed)) > 0) return v;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) { cudaGetLastError(); return 148; }
    if (dev < 64) sms[dev].store(v, std::memory_order_relaxed);
    return v;
}

SendKernel pick_send(const loco_config_t *c, int mode, int var) {
    const bool bf = c->grad_dtype == LOCO_BF16;
    switch (c->state_fmt) {
    case LOCO_STATE_INT8: return bf ? pick_send_g1_s0(c->bits, mode, var) : pick_send_g0_s0(c->bits, mode, var);
    case LOCO_STATE_FP32: return bf ? pick_send_g1_s1(c->bits, mode, var) : pick_send_g0_s1(c->bits, mode, var);
    case LOCO_STATE_NONE: return bf ? pick_send_g1_s2(c->bits, mode, var) : pick_send_g0_s2(c->bits, mode, var);
    default: return bf ? pick_send_g1_s3(c->bits, mode, var) : pick_send_g0_s3(c->bits, mode, var);
    }
}

ReduceKernel pick_reduce(const loco_config_t *c, int mode, int path, bool adam) {
    if (c->out_dtype == LOCO_BF16) return adam ? pick_reduce_o1_a1(c->bits, mode, path) : pick_reduce_o1_a0(c->bits, mode, path);
    return adam ? pick_reduce_o0_a1(c->bits, mode, path) : pick_reduce_o0_a0(c->bits, mode, path);
}

// CTAs per partition.  A bucket that fits one resident wave gets exactly that: every CTA resident at once, each warp a
// handful of wide rows.  A larger bucket gets more CTAs than are resident, each with about kRowsPerWarp wide rows per
// warp: the hardware then hands them out as SMs become free, which evens out the different speeds at which the SMs
// stream under a saturated memory system (with one wave and a fixed split, the fast SMs would idle until the slowest
// is done), at the price of one ring fill per CTA.
constexpr uint64_t kRowsPerWarp = 16;
unsigned grid_x_for(uint64_t wide_rows_per_partition, int partitions, int ctas_per_sm) {
    const uint64_t want = (wide_rows_per_partition + kWarps - 1) / kWarps;        // one wide row per warp
    uint64_t budget = static_cast<uint64_t>(num_sms()) * static_cast<uint64_t>(ctas_per_sm);
    uint64_t per_part = budget / static_cast<uint64_t>(partitions);
    if (per_part < 1) per_part = 1;
    uint64_t gx = want < per_part ? want : per_part;
    const uint64_t many = (wide_rows_per_partition + kWarps * kRowsPerWarp - 1) / (kWarps * kRowsPerWarp);
    if (many > gx) gx = many;
    if (gx < 1) gx = 1;
    if (gx > 0x7fffffffull) gx = 0x7fffffffull;
    return static_cast<unsigned>(gx);
}

}  // namespace

struct loco_state {
    loco_config_t cfg;
    uint64_t n;
    void *d_state;
    uint64_t state_bytes;
    unsigned long long *d_status;   // 2 words on the device
    int device;
    int mode;
    SendFn send_fn;
    SendMultiFn send_multi_fn;      // the same kernel walking several buckets per launch
    int send_var;
    int send_smem_bytes;            // dynamic shared memory of the send kernel (its cp.async ring)
    int send_ctas_per_sm;
    Layout layout;
    DecChoice dq, de;               // how the kernels evaluate dec(q; s) and dec(e; s_e)
    int fast;                       // the fast routine may be used
};

extern "C" {

const char *loco_status_string(int status) {
    switch (status) {
    case LOCO_OK: return "LOCO_OK";
    case LOCO_ERR_ARG: return "LOCO_ERR_ARG";
    case LOCO_ERR_ALIGN: return "LOCO_ERR_ALIGN";
    case LOCO_ERR_SIZE: return "LOCO_ERR_SIZE";
    case LOCO_ERR_CUDA: return "LOCO_ERR_CUDA";
    case LOCO_ERR_UNSUPPORTED: return "LOCO_ERR_UNSUPPORTED";
    default: return "LOCO_ERR_UNKNOWN";
    }
}

uint64_t loco_launch_count(void) { return g_launches.load(); }

int loco_config_check(const loco_config_t *cfg) { return check_config(cfg); }

uint64_t loco_state_bytes(const loco_config_t *cfg, uint64_t n) {
    return layout_ok(cfg) ? state_bytes(cfg, n) : 0;
}
uint64_t loco_partition_capacity(const loco_config_t *cfg, uint64_t n) {
    return layout_ok(cfg) ? make_layout(cfg, n).lp : 0;
}
uint64_t loco_partition_bytes(const loco_config_t *cfg, uint64_t n) {
    return layout_ok(cfg) ? make_layout(cfg, n).stride : 0;
}
uint64_t loco_packed_bytes(const loco_config_t *cfg, uint64_t n) {
    return layout_ok(cfg) ? make_layout(cfg, n).stride * static_cast<uint64_t>(cfg->num_partitions) : 0;
}
uint64_t loco_partition_elems(const loco_config_t *cfg, uint64_t n, int32_t j) {
    if (!layout_ok(cfg) || j < 0 || j >= cfg->num_partitions) return 0;
    const uint64_t lp = make_layout(cfg, n).lp;
    const uint64_t lo = static_cast<uint64_t>(j) * lp;
    if (lp == 0 || lo >= n) return 0;
    return (n - lo < lp) ? n - lo : lp;
}

int loco_state_init(loco_state_t **out, const loco_config_t *cfg, uint64_t n, void *d_state,
                    uint64_t d_state_bytes, void *stream) {
    if (!out) return LOCO_ERR_ARG;
    *out = nullptr;
    const int rc = check_config(cfg);
    if (rc != LOCO_OK) return rc;
    const uint64_t need = state_bytes(cfg, n);
    if (need > 0) {
        if (!d_state) return LOCO_ERR_ARG;
        if (!aligned16(d_state)) return LOCO_ERR_ALIGN;
        if (d_state_bytes < need) return LOCO_ERR_SIZE;
    }
    loco_state *st = new (std::nothrow) loco_state;
    if (!st) return LOCO_ERR_ARG;
    st->cfg = *cfg;
    st->n = n;
    st->d_state = d_state;
    st->state_bytes = need;
    st->d_status = nullptr;
    st->layout = make_layout(cfg, n);
    st->mode = kernel_mode(cfg);
    st->dq = DecChoice{DEC_FMA, 0.0f, 0.0f, 0.0f};
    st->de = st->dq;
    st->fast = 1;
    if (st->mode == MODE_FIXED) {
        if (cfg->bits == 1) {
            // sign code: d = +-fl(1/s), nothing to prove; the magnitude must be a usable number
            const volatile float vinv = 1.0f / cfg->s;
            st->dq = DecChoice{(std::isfinite(vinv) && vinv != 0.0f) ? DEC_FMA : DEC_DIVIDE, 0.0f, 0.0f, vinv};
        } else {
            const int half = 1 << (cfg->bits - 1);
            st->dq = choose_dec(cfg->s, -half, half - 1, half);
        }
        if (cfg->state_fmt == LOCO_STATE_INT8 || cfg->state_fmt == LOCO_STATE_FP32_Q8COMP)
            st->de = choose_dec(cfg->s_e, -128, 127, 128);
        st->fast = (st->dq.mode != DEC_DIVIDE && st->de.mode != DEC_DIVIDE) ? 1 : 0;
        // the fast routine tests only g for NaN / Inf when the state is 8-bit: dec(e) must be too small to push a
        // finite g to infinity (|e / s_e| <= 128 / s_e < 2^100)
        if (cfg->state_fmt == LOCO_STATE_INT8 && !(cfg->s_e > 1e-28f)) st->fast = 0;
    }
    {
        int var = VAR_GENERAL;
        if (cfg->rounding == LOCO_ROUND_STOCHASTIC) {
            var = VAR_STOCHASTIC;
            if (st->mode == MODE_BLOCK) st->fast = 0;        // block scales with stochastic rounding: careful routine only
            else if (st->dq.mode == DEC_FMA && st->de.mode == DEC_FMA) var = VAR_LEAN_SR;
        } else if (st->mode == MODE_BLOCK) {
            var = cfg->clip > 0.0f ? VAR_GENERAL : VAR_LEAN;      // the plain lean variants carry no clipping
            if (cfg->block_size > kWide) var |= VAR_WIDE_BLOCKS;   // the rows of a block on neighbouring warps
        } else {
            const bool extras = cfg->collect_stats || cfg->clip > 0.0f;
            if (st->dq.mode == DEC_FMA && st->de.mode == DEC_FMA) var = extras ? VAR_LEAN_X : VAR_LEAN;
            else if (st->dq.mode == DEC_FMA && st->de.mode == DEC_NEWTON) var = extras ? VAR_LEAN_NR_X : VAR_LEAN_NR;
        }
        const SendKernel k = pick_send(cfg, st->mode, var);
        st->send_fn = k.fn;
        st->send_multi_fn = k.multi_fn;
        st->send_var = var;
        st->send_smem_bytes = k.smem_bytes;
    }
    st->send_ctas_per_sm = 1;
    if (!st->send_fn) { delete st; return LOCO_ERR_UNSUPPORTED; }
    if (cudaGetDevice(&st->device) != cudaSuccess) { delete st; return LOCO_ERR_CUDA; }
    int occ = 0;
    // the ring wants most of the SM's shared memory (3 CTAs x up to 72 KB)
    for (const void *fn : {reinterpret_cast<const void *>(st->send_fn), reinterpret_cast<const void *>(st->send_multi_fn)}) {
        if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, st->send_smem_bytes) != cudaSuccess ||
            cudaFuncSetAttribute(fn, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared) != cudaSuccess) {
            cudaGetLastError();
            delete st;
            return LOCO_ERR_CUDA;
        }
    }
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, st->send_fn, kThreads, static_cast<size_t>(st->send_smem_bytes)) != cudaSuccess || occ < 1) {
        cudaGetLastError();
        delete st;
        return LOCO_ERR_CUDA;
    }
    st->send_ctas_per_sm = occ;
    if (cudaMalloc(reinterpret_cast<void **>(&st->d_status), kStatusBytes) != cudaSuccess) {
        cudaGetLastError();
        delete st;
        return LOCO_ERR_CUDA;
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemsetAsync(st->d_status, 0, kStatusBytes, s);
    if (e == cudaSuccess && need > 0) e = cudaMemsetAsync(d_state, 0, need, s);   // e~_0 = 0
    if (e != cudaSuccess) {
        cudaGetLastError();
        cudaFree(st->d_status);
        delete st;
        return LOCO_ERR_CUDA;
    }
    *out = st;
    return LOCO_OK;
}

int loco_state_reset(loco_state_t *st, void *stream) {
    if (!st) return LOCO_ERR_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemsetAsync(st->d_status, 0, kStatusBytes, s);
    if (e == cudaSuccess && st->state_bytes > 0) e = cudaMemsetAsync(st->d_state, 0, st->state_bytes, s);
    if (e != cudaSuccess) { cudaGetLastError(); return LOCO_ERR_CUDA; }
    return LOCO_OK;
}

int loco_state_destroy(loco_state_t *st) {
    if (!st) return LOCO_ERR_ARG;
    int rc = LOCO_OK;
    if (st->d_status && cudaFree(st->d_status) != cudaSuccess) { cudaGetLastError(); rc = LOCO_ERR_CUDA; }
    delete st;
    return rc;
}

}  // extern "C"

namespace {

// Algorithm 1's scalars for iteration step_k, as the kernels take them.
void fill_common(const loco_state_t *st, int64_t step_k, SendCommon &C) {
    const loco_config_t &c = st->cfg;
    std::memset(&C, 0, sizeof(C));
    C.s = c.s;
    C.s_e = c.s_e;
    C.beta = c.beta;
    {
        const volatile float omb = 1.0f - c.beta;    // (1 - beta), rounded once to fp32
        C.omb = omb;
    }
    C.inv_s = st->dq.inv;
    C.inv_se = st->de.inv;
    C.dq_a = st->dq.a; C.dq_b = st->dq.b; C.dq_mode = st->dq.mode;
    C.de_a = st->de.a; C.de_b = st->de.b; C.de_mode = st->de.mode;
    C.fast = st->fast;
    C.block_log2 = c.scale_mode == LOCO_SCALE_BLOCK_ABSMAX ? ilog2(static_cast<uint32_t>(c.block_size)) : 0;
    C.reset = (c.reset_period > 0 && (step_k % static_cast<int64_t>(c.reset_period)) == 0) ? 1 : 0;
    C.collect_stats = c.collect_stats ? 1 : 0;
    C.clip = c.clip;
    C.stochastic = c.rounding == LOCO_ROUND_STOCHASTIC ? 1 : 0;
    C.seed_lo = c.seed_lo; C.seed_hi = c.seed_hi;
    for (uint32_t r = 0; r < 10; ++r) {                  // Philox round keys: the Weyl sequence of the key
        C.sr_keys[2 * r] = c.seed_lo + r * 0x9E3779B9u;
        C.sr_keys[2 * r + 1] = c.seed_hi + r * 0xBB67AE85u;
    }
    C.k_lo = static_cast<unsigned>(static_cast<uint64_t>(step_k));
    C.k_hi = static_cast<unsigned>(static_cast<uint64_t>(step_k) >> 32);
}

void fill_bucket(const loco_state_t *st, const void *d_grad, void *d_comm, SendBucket &B) {
    B.grad = d_grad;
    B.state = st->d_state;
    B.comm = static_cast<uint8_t *>(d_comm);
    B.status = st->d_status;
    B.n = st->n;
    B.lp = st->layout.lp;
    B.stride = st->layout.stride;
    B.grid_x = 0;
    B.reserved = 0;
}

// The handle's kernels were prepared (shared-memory size, occupancy) on the device that was current at
// loco_state_init, and its buffers live there: a call with another device current is refused.
int check_device(const loco_state_t *st) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return LOCO_ERR_CUDA; }
    return dev == st->device ? LOCO_OK : LOCO_ERR_ARG;
}

// The send pass.  Its partitions go to d_comm + j * stride, or, with d_part_dst, to d_part_dst[j].
int send_launch(loco_state_t *st, const void *d_grad, void *d_comm, void *const *d_part_dst, int64_t step_k,
                void *stream) {
    if (!st || step_k < 0) return LOCO_ERR_ARG;
    const loco_config_t &c = st->cfg;
    if (d_part_dst && c.num_partitions > kMaxScatter) return LOCO_ERR_UNSUPPORTED;
    if (st->n == 0) return LOCO_OK;
    if (!d_grad || (!d_comm && !d_part_dst)) return LOCO_ERR_ARG;
    if (!aligned16(d_grad) || !aligned16(d_comm)) return LOCO_ERR_ALIGN;
    const int rc = check_device(st);
    if (rc != LOCO_OK) return rc;
    SendParams P;
    std::memset(&P, 0, sizeof(P));
    if (d_part_dst) {
        for (int j = 0; j < c.num_partitions; ++j) {
            if (!d_part_dst[j]) return LOCO_ERR_ARG;
            if (!aligned16(d_part_dst[j])) return LOCO_ERR_ALIGN;
            P.part_dst[j] = static_cast<uint8_t *>(d_part_dst[j]);
        }
        P.scatter = 1;
    }
    fill_common(st, step_k, P.c);
    fill_bucket(st, d_grad, d_comm, P.b);
    const uint64_t rows = (P.b.lp + kWide - 1) / kWide;
    dim3 grid(grid_x_for(rows, c.num_partitions, st->send_ctas_per_sm), static_cast<unsigned>(c.num_partitions), 1);
    st->send_fn<<<grid, kThreads, static_cast<size_t>(st->send_smem_bytes), static_cast<cudaStream_t>(stream)>>>(P);
    if (cudaGetLastError() != cudaSuccess) return LOCO_ERR_CUDA;
    g_launches.fetch_add(1);
    return LOCO_OK;
}

bool same_send_setup(const loco_state_t *a, const loco_state_t *b) {
    return std::memcmp(&a->cfg, &b->cfg, sizeof(loco_config_t)) == 0 && a->send_multi_fn == b->send_multi_fn &&
           a->device == b->device && a->fast == b->fast;
}

// Buckets [lo, hi) of a multi-bucket call, all of one configuration, in one launch: grid.z = buckets.
int send_multi_launch(loco_state_t *const *states, const void *const *d_grads, void *const *d_comms, int lo, int hi,
                      int64_t step_k, void *stream) {
    static thread_local SendMultiParams P;             // 29 KB: not on the stack
    const loco_state_t *first = states[lo];
    fill_common(first, step_k, P.c);
    P.count = 0;
    unsigned gx = 1;
    for (int i = lo; i < hi; ++i) {
        const loco_state_t *st = states[i];
        if (st->n == 0) continue;
        SendBucket &B = P.b[P.count++];
        fill_bucket(st, d_grads[i], d_comms[i], B);
        B.grid_x = grid_x_for((st->layout.lp + kWide - 1) / kWide, st->cfg.num_partitions, st->send_ctas_per_sm);
        if (B.grid_x > gx) gx = B.grid_x;
    }
    if (P.count == 0) return LOCO_OK;
    dim3 grid(gx, static_cast<unsigned>(first->cfg.num_partitions), static_cast<unsigned>(P.count));
    first->send_multi_fn<<<grid, kThreads, static_cast<size_t>(first->send_smem_bytes), static_cast<cudaStream_t>(stream)>>>(P);
    if (cudaGetLastError() != cudaSuccess) return LOCO_ERR_CUDA;
    g_launches.fetch_add(1);
    return LOCO_OK;
}

}  // namespace

extern "C" {

int loco_compensate_quantize_pack(loco_state_t *st, const void *d_grad, void *d_comm, int64_t step_k,
                                  void *stream) {
    if (st && st->n != 0 && !d_comm) return LOCO_ERR_ARG;
    return send_launch(st, d_grad, d_comm, nullptr, step_k, stream);
}

int loco_compensate_quantize_pack_scatter(loco_state_t *st, const void *d_grad, void *const *d_part_dst,
                                          int64_t step_k, void *stream) {
    if (!d_part_dst) return LOCO_ERR_ARG;
    return send_launch(st, d_grad, nullptr, d_part_dst, step_k, stream);
}

}  // extern "C"

namespace {

// What Eq. 8 needs that does not depend on the bucket: the forms of dec(q; s) and of the division by N that the host
// can prove equal to the IEEE divisions, and with them the kernel (`path`).  `max_code_bytes`: the largest code area of
// a part among the call's buckets (the integer path keeps 32-bit byte offsets).
int reduce_common(const loco_config_t *cfg, int32_t num_workers, int32_t first_partition, uint64_t max_code_bytes,
                  const loco_adam_t *ad, float *d_m, float *d_v, float *d_theta, ReduceCommon &C, int &mode, int &path) {
    std::memset(&C, 0, sizeof(C));
    C.first = static_cast<unsigned long long>(first_partition);
    C.num_workers = num_workers;
    C.block_log2 = cfg->scale_mode == LOCO_SCALE_BLOCK_ABSMAX ? ilog2(static_cast<uint32_t>(cfg->block_size)) : 0;
    C.s = cfg->s;
    C.n_workers_f = static_cast<float>(num_workers);
    {
        const volatile float inv_n = 1.0f / static_cast<float>(num_workers);
        C.inv_n = inv_n;
    }
    mode = kernel_mode(cfg);
    const bool n_pow2 = is_pow2(static_cast<uint64_t>(num_workers));
    C.div_mode = n_pow2 ? 0 : 2;          // a multiply by 1/N is the division only for powers of two
    C.gen_mul = 0.0f;
    C.gen_mode = 2;
    C.inv_s = 0.0f;
    C.int_path = 0;
    if (mode == MODE_FIXED && cfg->bits == 1) {
        // sign code: d = +-fl(1/s), which is (+-1) / s exactly as the division gives it
        const volatile float vinv = 1.0f / cfg->s;
        C.inv_s = vinv;
        C.gen_mul = vinv;
        C.gen_mode = 0;
        // Integer path: with s a power of two every partial sum of the +-1/s is exact, so the negative workers of an
        // element can be counted; the kernel's byte lanes hold 2c <= 32 and the sum is (N - 2c) / s (/ N)
        if (num_workers <= 16 && is_pow2_float(cfg->s) && max_code_bytes < (1ull << 32)) {
            C.int_path = 1;
            const float inv_s = 1.0f / cfg->s;                                    // exact
            float r = inv_s;
            if (n_pow2) r = inv_s * C.inv_n;                                      // exact: both powers of two
            C.ra = -r;
            C.rb = (kMagic + static_cast<float>(num_workers)) * r;                // exact: integer < 2^24 times 2^k
            if (!n_pow2) {
                bool nr_ok = true;
                for (int c2 = 0; c2 <= num_workers && nr_ok; ++c2) {
                    const float acc = static_cast<float>(num_workers - 2 * c2) * inv_s;
                    const volatile float want = acc / C.n_workers_f;
                    const volatile float q0 = acc * C.inv_n;
                    const float rem = std::fmaf(-q0, C.n_workers_f, acc);
                    nr_ok = same_bits(std::fmaf(rem, C.inv_n, q0), want);
                }
                C.div_mode = nr_ok ? 1 : 2;
            }
        }
    } else if (mode == MODE_FIXED) {
        const int half = 1 << (cfg->bits - 1);
        {
            const volatile float vinv = 1.0f / cfg->s;
            const float inv = vinv;
            C.inv_s = inv;
            float mul = 0.0f;
            if (exact_multiplier(cfg->s, -half, half - 1, &mul)) {
                C.gen_mul = mul;
                C.gen_mode = 0;
            } else if (std::isfinite(inv) && inv != 0.0f) {
                bool nr_ok = true;
                for (int q = -half; q < half && nr_ok; ++q) {
                    const float fq = static_cast<float>(q);
                    const volatile float want = fq / cfg->s;
                    const volatile float q0 = fq * inv;
                    const float rem = std::fmaf(q0, -cfg->s, fq);
                    nr_ok = same_bits(std::fmaf(rem, inv, q0), want);
                }
                if (nr_ok) C.gen_mode = 1;
            }
        }
        // Integer path: with s a power of two every partial sum of Eq. 8 is exact in fp32, so the codes can be
        // added as integers.  The lane sums are bounded by (2^p - 1) * N, which 8- and 16-bit lanes hold for N <= 16.
        if (num_workers <= 16 && is_pow2_float(cfg->s) && max_code_bytes < (1ull << 32)) {
            C.int_path = 1;
            const float inv_s = 1.0f / cfg->s;                                    // exact
            float ra = inv_s;
            if (n_pow2) ra = inv_s * C.inv_n;                                     // exact: both powers of two
            C.ra = ra;
            C.rb = -(kMagic + static_cast<float>(half * num_workers)) * ra;       // exact: integer < 2^24 times 2^k
            if (!n_pow2) {
                // acc takes the values t / s, t in [-half N, (half-1) N]: check the short division on all of them
                bool nr_ok = true;
                for (int t = -half * num_workers; t <= (half - 1) * num_workers && nr_ok; ++t) {
                    const float acc = static_cast<float>(t) * inv_s;
                    const volatile float want = acc / C.n_workers_f;
                    const volatile float q0 = acc * C.inv_n;
                    const float rem = std::fmaf(-q0, C.n_workers_f, acc);
                    nr_ok = same_bits(std::fmaf(rem, C.inv_n, q0), want);
                }
                C.div_mode = nr_ok ? 1 : 2;
            }
        }
    }
    path = mode == MODE_BLOCK ? PATH_MUL
           : (C.int_path ? PATH_INT : (cfg->bits == 1 || C.gen_mode == 0 ? PATH_MUL : (C.gen_mode == 1 ? PATH_NEWTON : PATH_DIVIDE)));
    if (ad) {
        C.adam_m = d_m; C.adam_v = d_v; C.adam_theta = d_theta;
        C.lr = ad->lr; C.beta1 = ad->beta1; C.beta2 = ad->beta2; C.delta = ad->delta;
        const volatile float o1 = 1.0f - ad->beta1, o2 = 1.0f - ad->beta2;       // rounded once to fp32
        C.omb1 = o1; C.omb2 = o2;
    }
    return LOCO_OK;
}

// Per device and kernel, once: the shared-memory attributes of the kernels and the CTAs of one that fit an SM.
int reduce_occupancy(const loco_config_t *cfg, int mode, int path, bool adam, const ReduceKernel &rk, int &occ) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
        cudaGetLastError();
        return LOCO_ERR_CUDA;
    }
    static int occ_cache[64][2][4][2][4][2] = {};
    static std::mutex occ_mu;
    std::lock_guard<std::mutex> lock(occ_mu);
    int &slot = occ_cache[dev][cfg->out_dtype == LOCO_BF16][cfg->bits == 1 ? 0 : (cfg->bits == 2 ? 1 : (cfg->bits == 4 ? 2 : 3))][mode][path][adam];
    if (slot == 0) {
        int v = 0;
        if (rk.smem_bytes > 0) {
            for (const void *fn : {reinterpret_cast<const void *>(rk.fn), reinterpret_cast<const void *>(rk.multi_fn)}) {
                if (!fn) continue;
                if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, rk.smem_bytes) != cudaSuccess ||
                    cudaFuncSetAttribute(fn, cudaFuncAttributePreferredSharedMemoryCarveout, 100) != cudaSuccess) {
                    cudaGetLastError();
                    return LOCO_ERR_CUDA;
                }
            }
        }
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&v, rk.fn, kThreads, rk.smem_bytes) != cudaSuccess || v < 1) {
            cudaGetLastError();
            return LOCO_ERR_CUDA;
        }
        slot = v;
    }
    occ = slot;
    return LOCO_OK;
}

void fill_reduce_bucket(const Layout &L, uint64_t n, void *d_out, ReduceBucket &B) {
    B.out = d_out;
    B.n = n;
    B.lp = L.lp;
    B.stride = L.stride;
    B.code_bytes = L.code_bytes;
    B.grid_x = 0;
    B.out_align32 = (reinterpret_cast<uintptr_t>(d_out) & 31u) == 0 ? 1 : 0;
}

int check_reduce_args(const loco_config_t *cfg, int32_t num_workers, int32_t first_partition, int32_t partition_count,
                      const loco_adam_t *ad) {
    const int rc = check_config(cfg);
    if (rc != LOCO_OK) return rc;
    if (num_workers < 1 || first_partition < 0 || partition_count < 0 ||
        first_partition + partition_count > cfg->num_partitions) return LOCO_ERR_ARG;
    if (num_workers > 64) return LOCO_ERR_UNSUPPORTED;
    if (ad && !(std::isfinite(ad->lr) && ad->beta1 >= 0.0f && ad->beta1 <= 1.0f && ad->beta2 >= 0.0f && ad->beta2 <= 1.0f &&
                ad->delta >= 0.0f && std::isfinite(ad->delta))) return LOCO_ERR_ARG;
    return LOCO_OK;
}

// The receive pass; with `ad` the Adam-family step is applied to the averaged gradient in the same kernel and d_out
// (the gradient itself) becomes optional.
int reduce_launch(const loco_config_t *cfg, const void *const *d_packed, int32_t num_workers, uint64_t n,
                  int32_t first_partition, int32_t partition_count, void *d_out, const loco_adam_t *ad, float *d_m,
                  float *d_v, float *d_theta, void *stream) {
    const int rc = check_reduce_args(cfg, num_workers, first_partition, partition_count, ad);
    if (rc != LOCO_OK) return rc;
    if (n == 0 || partition_count == 0) return LOCO_OK;
    const Layout L = make_layout(cfg, n);
    if (static_cast<uint64_t>(first_partition) * L.lp >= n) return LOCO_OK;      // nothing valid there
    if (!d_packed || (!ad && !d_out)) return LOCO_ERR_ARG;
    if (ad && (!d_m || !d_v || !d_theta)) return LOCO_ERR_ARG;
    if (!aligned16(d_out)) return LOCO_ERR_ALIGN;
    if (ad && (!aligned16(d_m) || !aligned16(d_v) || !aligned16(d_theta))) return LOCO_ERR_ALIGN;
    ReduceParams P;
    std::memset(&P, 0, sizeof(P));
    for (int w = 0; w < num_workers; ++w) {
        if (!d_packed[w]) return LOCO_ERR_ARG;
        if (!aligned16(d_packed[w])) return LOCO_ERR_ALIGN;
        P.parts[w] = static_cast<const uint8_t *>(d_packed[w]);
    }
    int mode = 0, path = 0;
    reduce_common(cfg, num_workers, first_partition, L.code_bytes, ad, d_m, d_v, d_theta, P.c, mode, path);
    fill_reduce_bucket(L, n, d_out, P.b);
    const ReduceKernel rk = pick_reduce(cfg, mode, path, ad != nullptr);
    int occ = 0;
    const int ro = reduce_occupancy(cfg, mode, path, ad != nullptr, rk, occ);
    if (ro != LOCO_OK) return ro;
    const uint64_t rows = (L.lp + kWide - 1) / kWide;
    dim3 grid(grid_x_for(rows, partition_count, occ), static_cast<unsigned>(partition_count), 1);
    rk.fn<<<grid, kThreads, static_cast<size_t>(rk.smem_bytes), static_cast<cudaStream_t>(stream)>>>(P);
    if (cudaGetLastError() != cudaSuccess) return LOCO_ERR_CUDA;
    g_launches.fetch_add(1);
    return LOCO_OK;
}

}  // namespace

extern "C" {

int loco_unpack_dequant_reduce(const loco_config_t *cfg, const void *const *d_packed, int32_t num_workers,
                               uint64_t n, int32_t first_partition, int32_t partition_count, void *d_out,
                               void *stream) {
    return reduce_launch(cfg, d_packed, num_workers, n, first_partition, partition_count, d_out, nullptr, nullptr, nullptr,
                         nullptr, stream);
}

int loco_unpack_dequant_reduce_adam(const loco_config_t *cfg, const void *const *d_packed, int32_t num_workers,
                                    uint64_t n, int32_t first_partition, int32_t partition_count, const loco_adam_t *adam,
                                    float *d_m, float *d_v, float *d_theta, void *d_grad_out, void *stream) {
    if (!adam) return LOCO_ERR_ARG;
    return reduce_launch(cfg, d_packed, num_workers, n, first_partition, partition_count, d_grad_out, adam, d_m, d_v,
                         d_theta, stream);
}

}  // extern "C"

namespace {

}  // namespace

extern "C" {

int loco_compensate_quantize_pack_multi(loco_state_t *const *states, const void *const *d_grads, void *const *d_comms,
                                        int32_t count, int64_t step_k, void *stream) {
    if (count < 0 || step_k < 0 || (count > 0 && (!states || !d_grads || !d_comms))) return LOCO_ERR_ARG;
    if (count == 0) return LOCO_OK;
    // every argument is checked before anything is launched
    for (int32_t i = 0; i < count; ++i) {
        if (!states[i]) return LOCO_ERR_ARG;
        if (states[i]->n == 0) continue;
        if (!d_grads[i] || !d_comms[i]) return LOCO_ERR_ARG;
        if (!aligned16(d_grads[i]) || !aligned16(d_comms[i])) return LOCO_ERR_ALIGN;
        const int rc = check_device(states[i]);
        if (rc != LOCO_OK) return rc;
    }
    // consecutive buckets of one configuration share a launch, as many as the kernel's table holds
    int rc = LOCO_OK;
    int32_t lo = 0;
    while (lo < count) {
        int32_t hi = lo + 1;
        while (hi < count && hi - lo < kMaxMulti && same_send_setup(states[lo], states[hi])) ++hi;
        const int r = send_multi_launch(states, d_grads, d_comms, lo, hi, step_k, stream);
        if (r != LOCO_OK && rc == LOCO_OK) rc = r;
        lo = hi;
    }
    return rc;
}

int loco_unpack_dequant_reduce_multi(const loco_config_t *cfg, const void *const *const *d_packed, int32_t num_workers,
                                     const uint64_t *n, void *const *d_outs, int32_t count, void *stream) {
    if (count < 0 || (count > 0 && (!cfg || !d_packed || !n || !d_outs))) return LOCO_ERR_ARG;
    if (count == 0) return LOCO_OK;
    const int rc0 = check_reduce_args(cfg, num_workers, 0, cfg ? cfg->num_partitions : 0, nullptr);
    if (rc0 != LOCO_OK) return rc0;
    // every argument is checked before anything is launched
    uint64_t max_code_bytes = 0;
    for (int32_t i = 0; i < count; ++i) {
        if (n[i] == 0) continue;
        if (!d_packed[i] || !d_outs[i]) return LOCO_ERR_ARG;
        if (!aligned16(d_outs[i])) return LOCO_ERR_ALIGN;
        for (int w = 0; w < num_workers; ++w) {
            if (!d_packed[i][w]) return LOCO_ERR_ARG;
            if (!aligned16(d_packed[i][w])) return LOCO_ERR_ALIGN;
        }
        const uint64_t cb = make_layout(cfg, n[i]).code_bytes;
        if (cb > max_code_bytes) max_code_bytes = cb;
    }
    static thread_local ReduceMultiParams P;           // 32 KB: not on the stack
    int mode = 0, path = 0;
    reduce_common(cfg, num_workers, 0, max_code_bytes, nullptr, nullptr, nullptr, nullptr, P.c, mode, path);
    const ReduceKernel rk = pick_reduce(cfg, mode, path, false);
    int occ = 0;
    const int ro = reduce_occupancy(cfg, mode, path, false, rk, occ);
    if (ro != LOCO_OK) return ro;
    // as many buckets per launch as the kernel's tables hold
    const int per_launch_ptrs = kMaxReducePtrs / num_workers;
    const int per_launch = per_launch_ptrs < kMaxReduceBuckets ? per_launch_ptrs : kMaxReduceBuckets;
    int rc = LOCO_OK;
    int32_t i = 0;
    while (i < count) {
        P.count = 0;
        unsigned gx = 1;
        for (; i < count && P.count < per_launch; ++i) {
            if (n[i] == 0) continue;
            const Layout L = make_layout(cfg, n[i]);
            ReduceBucket &B = P.b[P.count];
            fill_reduce_bucket(L, n[i], d_outs[i], B);
            B.grid_x = grid_x_for((L.lp + kWide - 1) / kWide, cfg->num_partitions, occ);
            if (B.grid_x > gx) gx = B.grid_x;
            for (int w = 0; w < num_workers; ++w)
                P.parts[P.count * num_workers + w] = static_cast<const uint8_t *>(d_packed[i][w]);
            ++P.count;
        }
        if (P.count == 0) break;
        dim3 grid(gx, static_cast<unsigned>(cfg->num_partitions), static_cast<unsigned>(P.count));
        rk.multi_fn<<<grid, kThreads, static_cast<size_t>(rk.smem_bytes), static_cast<cudaStream_t>(stream)>>>(P);
        if (cudaGetLastError() != cudaSuccess) { if (rc == LOCO_OK) rc = LOCO_ERR_CUDA; }
        else g_launches.fetch_add(1);
    }
    return rc;
}

uint64_t loco_send_host_workspace_bytes(const loco_config_t *cfg, uint64_t n) {
    if (!layout_ok(cfg) || n == 0) return 0;
    const uint64_t gbytes = round_up(n * (cfg->grad_dtype == LOCO_BF16 ? 2u : 4u), 256);
    return gbytes + make_layout(cfg, n).stride * static_cast<uint64_t>(cfg->num_partitions);
}

uint64_t loco_reduce_host_workspace_bytes(const loco_config_t *cfg, uint64_t n, int32_t num_workers,
                                          int32_t partition_count) {
    if (!layout_ok(cfg) || n == 0 || num_workers < 1 || partition_count < 1) return 0;
    const Layout L = make_layout(cfg, n);
    const uint64_t in = static_cast<uint64_t>(num_workers) * static_cast<uint64_t>(partition_count) * L.stride;
    const uint64_t out = round_up(static_cast<uint64_t>(partition_count) * L.lp * (cfg->out_dtype == LOCO_BF16 ? 2u : 4u), 256);
    return in + out;
}

int loco_compensate_quantize_pack_host(loco_state_t *st, const void *h_grad, void *h_comm, void *d_work,
                                       uint64_t d_work_bytes, int64_t step_k, void *stream) {
    if (!st || step_k < 0) return LOCO_ERR_ARG;
    if (st->n == 0) return LOCO_OK;
    if (!h_grad || !h_comm || !d_work) return LOCO_ERR_ARG;
    if (!aligned16(d_work)) return LOCO_ERR_ALIGN;
    if (d_work_bytes < loco_send_host_workspace_bytes(&st->cfg, st->n)) return LOCO_ERR_SIZE;
    const uint64_t gbytes_exact = st->n * (st->cfg.grad_dtype == LOCO_BF16 ? 2u : 4u);
    const uint64_t gbytes = round_up(gbytes_exact, 256);
    const uint64_t pbytes = st->layout.stride * static_cast<uint64_t>(st->cfg.num_partitions);
    uint8_t *d_grad = static_cast<uint8_t *>(d_work);
    uint8_t *d_comm = d_grad + gbytes;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(d_grad, h_grad, gbytes_exact, cudaMemcpyHostToDevice, s) != cudaSuccess) {
        cudaGetLastError();
        return LOCO_ERR_CUDA;
    }
    const int rc = loco_compensate_quantize_pack(st, d_grad, d_comm, step_k, stream);
    if (rc != LOCO_OK) return rc;
    if (cudaMemcpyAsync(h_comm, d_comm, pbytes, cudaMemcpyDeviceToHost, s) != cudaSuccess) {
        cudaGetLastError();
        return LOCO_ERR_CUDA;
    }
    return LOCO_OK;
}

int loco_unpack_dequant_reduce_host(const loco_config_t *cfg, const void *const *h_packed, int32_t num_workers,
                                    uint64_t n, int32_t first_partition, int32_t partition_count, void *h_out,
                                    void *d_work, uint64_t d_work_bytes, void *stream) {
    const int rc0 = check_config(cfg);
    if (rc0 != LOCO_OK) return rc0;
    if (num_workers < 1 || first_partition < 0 || partition_count < 0 ||
        first_partition + partition_count > cfg->num_partitions) return LOCO_ERR_ARG;
    if (num_workers > 64) return LOCO_ERR_UNSUPPORTED;
    if (n == 0 || partition_count == 0) return LOCO_OK;
    if (!h_packed || !h_out || !d_work) return LOCO_ERR_ARG;
    if (!aligned16(d_work)) return LOCO_ERR_ALIGN;
    if (d_work_bytes < loco_reduce_host_workspace_bytes(cfg, n, num_workers, partition_count)) return LOCO_ERR_SIZE;
    const Layout L = make_layout(cfg, n);
    const uint64_t per_worker = static_cast<uint64_t>(partition_count) * L.stride;
    uint8_t *base = static_cast<uint8_t *>(d_work);
    const void *d_ptrs[64];
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    for (int w = 0; w < num_workers; ++w) {
        if (!h_packed[w]) return LOCO_ERR_ARG;
        d_ptrs[w] = base + static_cast<uint64_t>(w) * per_worker;
        if (cudaMemcpyAsync(const_cast<void *>(d_ptrs[w]), h_packed[w], per_worker, cudaMemcpyHostToDevice, s) != cudaSuccess) {
            cudaGetLastError();
            return LOCO_ERR_CUDA;
        }
    }
    uint8_t *d_out = base + static_cast<uint64_t>(num_workers) * per_worker;
    const int rc = loco_unpack_dequant_reduce(cfg, d_ptrs, num_workers, n, first_partition, partition_count, d_out, stream);
    if (rc != LOCO_OK) return rc;
    uint64_t n_out = 0;
    for (int j = first_partition; j < first_partition + partition_count; ++j) n_out += loco_partition_elems(cfg, n, j);
    if (n_out == 0) return LOCO_OK;
    if (cudaMemcpyAsync(h_out, d_out, n_out * (cfg->out_dtype == LOCO_BF16 ? 2u : 4u), cudaMemcpyDeviceToHost, s) != cudaSuccess) {
        cudaGetLastError();
        return LOCO_ERR_CUDA;
    }
    return LOCO_OK;
}

// ---- receive pass for host buffers with a built-in staging area -------------------------------

}  // extern "C"

namespace {

// Staging area of loco_unpack_dequant_reduce_host_noalloc: part of the library image, present on
// every device that loads it, never allocated or freed.
static __device__ __align__(256) unsigned char g_noalloc_scratch[LOCO_NOALLOC_SCRATCH_BYTES];

// Device address of g_noalloc_scratch on the current device.  In host code the array's name only
// identifies the symbol to the runtime; it is not an address a copy or a kernel could use, so the
// address is asked for once per device (with that device current) and remembered.
int noalloc_scratch_address(void **out) {
    constexpr int kCached = 64;
    static std::mutex mu;
    static void *cached[kCached] = {};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0) { cudaGetLastError(); return LOCO_ERR_CUDA; }
    std::lock_guard<std::mutex> lock(mu);
    if (dev < kCached && cached[dev]) { *out = cached[dev]; return LOCO_OK; }
    void *p = nullptr;
    if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) { cudaGetLastError(); return LOCO_ERR_CUDA; }
    if (dev < kCached) cached[dev] = p;
    *out = p;
    return LOCO_OK;
}

}  // namespace

extern "C" {

int loco_unpack_dequant_reduce_host_noalloc(const loco_config_t *cfg, const void *const *h_packed,
                                            int32_t num_workers, uint64_t n, int32_t first_partition,
                                            int32_t partition_count, void *h_out, void *stream) {
    const int rc0 = check_config(cfg);
    if (rc0 != LOCO_OK) return rc0;
    if (num_workers < 1 || first_partition < 0 || partition_count < 0 ||
        first_partition + partition_count > cfg->num_partitions) return LOCO_ERR_ARG;
    if (num_workers > 64) return LOCO_ERR_UNSUPPORTED;
    if (n == 0 || partition_count == 0) return LOCO_OK;
    // the request must fit the fixed array: refuse it before anything is enqueued
    if (loco_reduce_host_workspace_bytes(cfg, n, num_workers, partition_count) > LOCO_NOALLOC_SCRATCH_BYTES)
        return LOCO_ERR_SIZE;
    void *d_scratch = nullptr;
    const int rc1 = noalloc_scratch_address(&d_scratch);
    if (rc1 != LOCO_OK) return rc1;
    return loco_unpack_dequant_reduce_host(cfg, h_packed, num_workers, n, first_partition, partition_count, h_out,
                                           d_scratch, LOCO_NOALLOC_SCRATCH_BYTES, stream);
}

int loco_selfcheck_block_division(uint64_t *mismatches) {
    if (!mismatches) return LOCO_ERR_ARG;
    unsigned long long *d = nullptr;
    if (cudaMalloc(reinterpret_cast<void **>(&d), 16) != cudaSuccess) { cudaGetLastError(); return LOCO_ERR_CUDA; }
    unsigned long long h[2] = {0, 0};
    cudaError_t e = cudaMemset(d, 0, 16);
    if (e == cudaSuccess) {
        loco_division_selfcheck_kernel<<<num_sms() * 8, 256>>>(d);
        e = cudaGetLastError();
    }
    if (e == cudaSuccess) e = cudaMemcpy(h, d, 16, cudaMemcpyDeviceToHost);
    cudaFree(d);
    if (e != cudaSuccess) { cudaGetLastError(); return LOCO_ERR_CUDA; }
    g_launches.fetch_add(1);
    mismatches[0] = h[0];
    mismatches[1] = h[1];
    return LOCO_OK;
}

int loco_status_counters(loco_state_t *st, uint32_t *flags, uint64_t *n_saturated, uint64_t *n_saturated_state,
                         void *stream) {
    if (!st) return LOCO_ERR_ARG;
    unsigned long long host[4] = {0, 0, 0, 0};
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(host, st->d_status, kStatusBytes, cudaMemcpyDeviceToHost, s) != cudaSuccess ||
        cudaStreamSynchronize(s) != cudaSuccess) {
        cudaGetLastError();
        return LOCO_ERR_CUDA;
    }
    if (flags) *flags = static_cast<uint32_t>(host[0]);
    if (n_saturated) *n_saturated = host[1];
    if (n_saturated_state) *n_saturated_state = host[2];
    return LOCO_OK;
}

int loco_last_status(loco_state_t *st, uint32_t *flags, uint64_t *n_saturated, void *stream) {
    return loco_status_counters(st, flags, n_saturated, nullptr, stream);
}

}  // extern "C"
