// Shared device-side definitions of the CO3 kernels: workspace layout, derived per-segment
// tables, the bit-exact converter and small block primitives.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "co3.h"

namespace co3 {

constexpr int kC = CO3_CHUNK_SYMS;                           // symbols per chunk
constexpr int kS = CO3_SUB_SYMS;                             // symbols per sub-chunk offset
constexpr int kSubs = kC / kS;                               // 16
constexpr int kSlotWords = kC * CO3_MAX_CODE_LEN / 32;       // worst-case words of one chunk
constexpr int kDecBits = 12;                                 // decode LUT is indexed by 12 stream bits
constexpr int kDecLut = 1 << kDecBits;
constexpr int kSubBits = CO3_MAX_CODE_LEN - kDecBits;        // second-level tables are indexed by the next 4 bits
constexpr int kSubLut = 256 << kSubBits;                     // at most 256 second-level tables per segment
constexpr uint32_t kEncMissing = 0x80000000u;                // encode table entry of a symbol without codeword
constexpr uint32_t kDecLong = 0x8000u;                       // decode table entry: look in a second-level table
constexpr uint32_t kDecInvalid = 0x01ffu;                    // decode table entry: no codeword; consumes one bit and
                                                             // yields 0xff, which is a symbol of no format
constexpr int kRangeChunks = 4096;                            // chunks summed by one block in the two-level scan
constexpr uint32_t kMagic = 0x53334F43u;                     // 'C','O','3','S'
constexpr uint32_t kHeaderBytes = 64;
constexpr int kThreads = 256;

// Call-wide state in the workspace, cleared at the start of every call.
struct Ctrl {
    uint32_t abort;     // set when descriptor validation failed: later kernels return at once
    uint32_t n_chunks;  // chunks per client
    uint32_t n_tiles;   // decode tiles per client
    uint32_t pad;
    uint64_t chunk_off, sub_off, payload_off;  // byte offsets of the container sections
};

// Where a chunk lives: written by the prepare kernel, read by every kernel that works per chunk.
struct ChunkDesc {
    uint32_t seg;    // segment (layer) of the chunk
    uint32_t cnt;    // symbols in the chunk (kC except for the last chunk of a segment)
    uint64_t elem0;  // index of its first element inside a client's vector
    uint32_t cis;    // the chunk's index inside its segment: its first element is at place cis * kC of the layer
    uint32_t pad;
};

// A decode tile: up to `tile_chunks` consecutive chunks of one segment.
struct TileDesc {
    uint32_t seg;
    uint32_t chunk0;
    uint32_t n_chunks;
    uint32_t pad;
};

// Converter constants of one segment, derived from co3_fmt by the prepare kernel.  (16-byte alignment: a thread
// fetches its copy from shared memory with a few wide loads.)
struct alignas(16) FmtDev {
    uint32_t mant_bits;        // M
    uint32_t mag_bits;         // E + M
    uint32_t fast;             // 1: M >= 1 and sub-normal levels kept, the branch-free converter applies
    uint32_t drop;             // 23 - M: fp32 mantissa bits below the format's
    uint32_t min_normal_bits;  // fp32 pattern of 2^emin
    uint32_t code_bias;        // (emin + 126) << M : fp32 (exp|mant>>drop) minus this is the magnitude code
    uint32_t max_code;         // largest magnitude code
    uint32_t top_bits;         // fp32 pattern of the largest level
    uint32_t sign_shift;       // 31 - (E + M): moves the fp32 sign bit to the symbol's sign bit
    uint32_t flush;            // 1: no sub-normal levels
    uint32_t half_min_bits;    // fp32 pattern of 2^(emin-1)
    float magic;               // 2^(emin - M + 23): adding it rounds to a multiple of the sub-normal step
    float scale, inv_scale;
    uint32_t pad[2];           // 64 bytes: the table is addressed in whole 16-byte units
};
static_assert(sizeof(FmtDev) == 64, "FmtDev is a whole number of 16-byte units");

// Workspace sections (device pointers), computed on the host from sizes only.
struct Ws {
    Ctrl* ctrl;
    uint32_t* first_chunk;  // [n_seg + 1]
    ChunkDesc* chunk_desc;  // [n_chunks_max]
    TileDesc* tile_desc;    // [n_chunks_max]
    FmtDev* fmt;            // [n_seg]
    uint32_t* enc_lut;      // [n_seg][256]   bits << 8 | len ; kEncMissing for a symbol without codeword
    uint16_t* dec_lut;      // [n_seg][4096]  len << 8 | sym ; kDecInvalid where no codeword matches;
                            //                kDecLong | index of a second-level table for longer codewords
    uint16_t* dec_sub;      // [n_seg][256][16]  len << 8 | sym for codewords of 13..16 bits, by their bits 13..16
    float* val_lut;         // [n_seg][256]   reconstructed value of each symbol
    uint32_t* client_fail;  // [n_clients]
    uint32_t* chunk_bits;   // [n_clients][n_chunks_max]
    uint64_t* bit_prefix;   // [n_clients][n_chunks_max + 1]
    uint64_t* range_tot;    // [n_clients][n_ranges_max][2]  words and bits of each range of kRangeChunks chunks
                            //                               (long inputs only), then their exclusive prefixes
    uint64_t* totals;       // [n_clients][2]                payload words and bits of the client (long inputs)
    uint32_t* slots;        // [n_clients][n_chunks_max][kSlotWords]
    uint32_t n_chunks_max;
};

__host__ __device__ inline uint64_t align16(uint64_t x) { return (x + 15u) & ~(uint64_t)15u; }

// First error wins, except that the soft "non-finite input" status yields to any other error.
__device__ inline void set_status(co3_result* r, int code) {
    const int old = atomicCAS(&r->status, CO3_OK, code);
    if (old == CO3_ERR_NONFINITE && code != CO3_ERR_NONFINITE) atomicCAS(&r->status, CO3_ERR_NONFINITE, code);
}

// Index of the segment that owns item `x`: largest k with first[k] <= x (empty segments are skipped).
__device__ inline uint32_t find_seg(const uint32_t* __restrict__ first, uint32_t n_seg, uint32_t x) {
    uint32_t lo = 0, hi = n_seg;  // invariant: first[lo] <= x < first[hi]
    while (hi - lo > 1) {
        const uint32_t mid = (lo + hi) >> 1;
        if (first[mid] <= x) lo = mid; else hi = mid;
    }
    return lo;
}

// One element of Algorithm 1's client update:
//   v = g + gamma*m (one FMA); t = v*scale; nearest level by integer work on the fp32 pattern
//   (ties to the even code); ghat = level*inv_scale; returns m_new = v - ghat and the symbol.
// flags: bit 0 = finite input beyond the largest level, bit 1 = NaN/Inf input.
__device__ __forceinline__ float convert_one(float g, float m, float decay, const FmtDev& f,
                                             uint32_t& sym, uint32_t& flags) {
    const float v = __fmaf_rn(decay, m, g);
    const uint32_t vb = __float_as_uint(v) & 0x7fffffffu;
    const float t = __fmul_rn(v, f.scale);
    const uint32_t tb = __float_as_uint(t);
    const uint32_t a = tb & 0x7fffffffu;
    uint32_t code;
    float qmag;
    if (a >= f.min_normal_bits) {
        const uint32_t drop = 23u - f.mant_bits;
        const uint32_t r = a + ((1u << (drop - 1u)) - 1u) + ((a >> drop) & 1u);  // round half to even
        code = (r >> drop) - f.code_bias;
        flags |= (a > f.top_bits) ? 1u : 0u;  // beyond the boundary, even if it would round back onto it
        code = min(code, f.max_code);
        qmag = __uint_as_float((code + f.code_bias) << drop);
    } else if (!f.flush) {
        const float s = __fadd_rn(__uint_as_float(a), f.magic);  // rounds |t| to the sub-normal step, ties to even
        code = __float_as_uint(s) - __float_as_uint(f.magic);
        qmag = __fsub_rn(s, f.magic);
    } else {
        code = (a > f.half_min_bits) ? (1u << f.mant_bits) : 0u;  // zero or the smallest normal level; tie to zero
        qmag = code ? __uint_as_float(f.min_normal_bits) : 0.0f;
    }
    uint32_t sign = (code != 0u) ? (tb >> 31) : 0u;
    float ghat = __fmul_rn(sign ? -qmag : qmag, f.inv_scale);
    float m_new = __fsub_rn(v, ghat);
    if (vb >= 0x7f800000u) {  // NaN is sent as zero, +-Inf as the boundary level; their memory restarts
        flags = (flags & ~1u) | 2u;
        m_new = 0.0f;
        if (vb > 0x7f800000u) { code = 0u; sign = 0u; }
    }
    sym = (sign << f.mag_bits) | code;
    return m_new;
}

// The same update without branches, for formats with M >= 1 that keep the sub-normal levels.
// Rounding by one fp32 addition: with ae the (clamped) exponent of |t|, |t| + 2^(ae + 23 - M) is rounded by
// the adder to a multiple of the format's step in that binade, ties to the even multiple, which has the
// even code when M >= 1.  Inputs beyond the largest level and non-finite ones are clamped to it here and
// reported in `beyond` (a NaN fails the comparison too): for a finite input that is already the right level
// and memory (saturation, Sec. V-B boundary) and the caller only counts it; a group that holds a NaN or an
// infinity is repeated with convert_one.  Inputs that land on the largest level from inside the range (common
// in the narrow formats) need no second look.
__device__ __forceinline__ float convert_fast(float g, float m, float decay, const FmtDev& f, uint32_t& sym,
                                              bool& beyond) {
    const float v = __fmaf_rn(decay, m, g);
    const float t = __fmul_rn(v, f.scale);
    const float top = __uint_as_float(f.top_bits);
    beyond |= !(fabsf(t) <= top);
    const float at = fminf(fabsf(t), top);  // NaN -> largest level
    const uint32_t ac = __float_as_uint(at);
    const uint32_t ae = max(ac & 0x7f800000u, f.min_normal_bits);
    const uint32_t mg = ae + (f.drop << 23);
    const float s = __fadd_rn(at, __uint_as_float(mg));
    const uint32_t code = ((ae - f.min_normal_bits) >> f.drop) + (__float_as_uint(s) - mg);
    const float qmag = __fsub_rn(s, __uint_as_float(mg));
    const uint32_t sgn = code ? (__float_as_uint(t) & 0x80000000u) : 0u;
    sym = code | (sgn >> f.sign_shift);
    const float ghat = __fmul_rn(__uint_as_float(__float_as_uint(qmag) | sgn), f.inv_scale);
    return __fsub_rn(v, ghat);
}

// First statement of a kernel that is launched right behind another kernel of the same call with programmatic
// stream serialization: its blocks may be set up while that kernel still runs, and wait here until it has completed
// and its writes are visible.  Without that launch attribute the instruction does nothing.
__device__ __forceinline__ void wait_for_previous_kernel() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Philox-4x32 with 10 rounds (Salmon, Moraes, Dror, Shaw, SC 2011): a block of four 32-bit words from a counter
// and a key.  Each round multiplies two counter words by fixed constants, crosses the halves of the products with
// the other two words and the key, and the key advances by Weyl constants between rounds.
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint32_t k0, uint32_t k1) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        if (r > 0) { k0 += 0x9E3779B9u; k1 += 0xBB67AE85u; }
        const uint32_t lo0 = 0xD2511F53u * c.x, hi0 = __umulhi(0xD2511F53u, c.x);
        const uint32_t lo1 = 0xCD9E8D57u * c.z, hi1 = __umulhi(0xCD9E8D57u, c.z);
        c = make_uint4(hi1 ^ c.y ^ k0, lo1, hi0 ^ c.w ^ k1, lo0);
    }
    return c;
}

// convert_one with the nearest-level rule replaced by the dithered one (Sec. II-B (ii): the quantizer as a stochastic
// mapping): with R the element's 24-bit draw the upper of the two levels around |t| is taken iff
// R < (|t| - lower) / (upper - lower) * 2^24.  From the smallest normal level up that fraction is the part of
// the fp32 mantissa below the format's, so adding what the draw leaves of the dropped bits' range and cutting does
// it; below, |t| is brought to a fixed-point count of 2^-24 steps by one exact multiplication.
__device__ __forceinline__ float convert_one_dither(float g, float m, float decay, const FmtDev& f, uint32_t R,
                                                    uint32_t& sym, uint32_t& flags) {
    const float v = __fmaf_rn(decay, m, g);
    const uint32_t vb = __float_as_uint(v) & 0x7fffffffu;
    const float t = __fmul_rn(v, f.scale);
    const uint32_t tb = __float_as_uint(t);
    const uint32_t a = tb & 0x7fffffffu;
    uint32_t code;
    float qmag;
    if (a >= f.top_bits) {  // the largest level or beyond it (also +-Inf and NaN patterns, sorted out below)
        flags |= (a > f.top_bits) ? 1u : 0u;
        code = f.max_code;
        qmag = __uint_as_float(f.top_bits);
    } else if (a >= f.min_normal_bits) {
        const uint32_t mask = (1u << f.drop) - 1u;
        const uint32_t r = R >> (f.mant_bits + 1u);  // the draw on the grid of the dropped bits
        code = ((a + (mask - r)) >> f.drop) - f.code_bias;  // one more iff the dropped bits exceed r
        qmag = __uint_as_float((code + f.code_bias) << f.drop);
    } else {
        // |t| in units of 2^-24 of the step below the smallest normal level (2^(emin - M), or 2^emin without
        // sub-normal levels): an exact product with a power of two, below 2^(24 + M)
        const uint32_t step_exp = (f.min_normal_bits >> 23) - (f.flush ? 0u : f.mant_bits);  // biased exponent of the step
        const float w = __fmul_rn(__uint_as_float(a), __uint_as_float((24u + 254u - step_exp) << 23));
        const uint32_t wi = __float2uint_rz(w);
        const uint32_t frac = (wi & 0xffffffu) + (__uint2float_rn(wi) != w ? 1u : 0u);
        const uint32_t n = (wi >> 24) + (R < frac ? 1u : 0u);  // steps
        code = f.flush ? n << f.mant_bits : n;
        qmag = __fmul_rn(__uint2float_rn(n), __uint_as_float(step_exp << 23));
    }
    uint32_t sign = (code != 0u) ? (tb >> 31) : 0u;
    float ghat = __fmul_rn(sign ? -qmag : qmag, f.inv_scale);
    float m_new = __fsub_rn(v, ghat);
    if (vb >= 0x7f800000u) {  // NaN is sent as zero, +-Inf as the boundary level; their memory restarts
        flags = (flags & ~1u) | 2u;
        m_new = 0.0f;
        if (vb > 0x7f800000u) { code = 0u; sign = 0u; }
    }
    sym = (sign << f.mag_bits) | code;
    return m_new;
}

// ------------------------------------------------------------------------------------------------
// Bulk asynchronous copies (TMA, untiled form) into shared memory, completed on an mbarrier.
// Source and destination must be 16-byte aligned and the size a multiple of 16 bytes.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t arrivals) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(arrivals) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

// Orders earlier ordinary shared-memory accesses before later bulk copies into the same bytes.
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(smem_addr(bar)), "r"(parity)
        : "memory");
    return done != 0;
}

__device__ __forceinline__ uint64_t global_timer_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Waits for the phase with the given parity, for at most about half a second of wall time.
// Returns false on give-up.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = global_timer_ns();
    for (;;) {
        for (int i = 0; i < 64; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (global_timer_ns() - t0 > 500000000ull) return false;
    }
}

__device__ __forceinline__ void bulk_copy_g2s(void* dst_smem, const void* src_gmem, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_addr(dst_smem)),
                 "l"(src_gmem), "r"(bytes), "r"(smem_addr(bar))
                 : "memory");
}

// Exclusive prefix sum over the 256 threads of a block; *total receives the block sum.
// scratch: 8 words of shared memory.  Contains two __syncthreads().
__device__ __forceinline__ uint32_t block_exclusive_scan_256(uint32_t x, uint32_t* scratch, uint32_t* total) {
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    uint32_t inc = x;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t y = __shfl_up_sync(0xffffffffu, inc, d);
        if (lane >= (uint32_t)d) inc += y;
    }
    if (lane == 31u) scratch[warp] = inc;
    __syncthreads();
    uint32_t base = 0, sum = 0;
#pragma unroll
    for (int w = 0; w < 8; ++w) {
        const uint32_t s = scratch[w];
        if ((uint32_t)w < warp) base += s;
        sum += s;
    }
    __syncthreads();
    *total = sum;
    return base + inc - x;
}

}  // namespace co3
