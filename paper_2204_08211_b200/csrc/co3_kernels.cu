// CUDA kernels of the CO3 uplink pipeline and its parameter-server inverse (sm_100a).
//
//   prepare_kernel        descriptor validation + derived tables (chunk map, encode/decode LUTs);
//                         for decode calls also header / table validation of every stream
//   convert_kernel        v = g + gamma*m, ghat = Q_fp(v), m = v - ghat, symbols, histogram
//   pack_kernel           (convert +) codeword lookup, block scan of lengths, bit packing of one chunk
//   scan_kernel           chunk word offsets, header and tables of one client's container
//   compact_kernel        chunk payloads from their worst-case slots to their final place
//   decode_kernel         chunk-indexed prefix-code decoder fused with the ordered cross-client sum
#include <cuda_runtime.h>
#include <stddef.h>

#include <algorithm>
#include <utility>
#include <stdint.h>

#include "co3.h"
#include "co3_device.cuh"

namespace co3 {

// ------------------------------------------------------------------------------------------------
// prepare: one block per segment validates that segment's descriptors, finds its place by a block
// reduction over the segments before it, writes its chunk and tile descriptors and builds its tables.
// ------------------------------------------------------------------------------------------------
struct PrepArgs {
    const co3_fmt* fmts;    // nullable (encode from symbols)
    const co3_code* codes;  // nullable (convert only)
    const co3_seg* segs;
    uint32_t n_seg;
    uint64_t n_elem;
    uint32_t tile_chunks;  // chunks per decode tile
    co3_result* res;
    uint32_t n_res;
    uint32_t want_dec;     // build the decode tables (decode calls only)
    // decode calls: the streams to validate against the layout (n_streams = 0 otherwise)
    const uint8_t* const* streams;  // device array of pointers, or null:
    const uint8_t* single;          // the one stream
    size_t stream_bytes;
    uint32_t n_streams;
    Ws ws;
};

__device__ __forceinline__ const uint8_t* prep_stream(const PrepArgs& a, uint32_t u) {
    return a.streams ? a.streams[u] : a.single;
}

// A stream failed validation: the decode kernel must not run.
__device__ void fail_corrupt(const PrepArgs& a) {
    a.ws.ctrl->abort = 1u;
    set_status(&a.res[0], CO3_ERR_CORRUPT);
}

// Header of stream u against the layout (n_chunks chunks, payload at payload_off).  One thread per stream.
__device__ bool header_ok(const PrepArgs& a, uint32_t u, uint64_t n_chunks, uint64_t chunk_off, uint64_t payload_off) {
    const uint8_t* stream = prep_stream(a, u);
    if (stream == nullptr || (reinterpret_cast<uintptr_t>(stream) & 15u) || a.stream_bytes < payload_off) return false;
    const uint32_t* h32 = reinterpret_cast<const uint32_t*>(stream);
    const uint64_t* h64 = reinterpret_cast<const uint64_t*>(stream);
    const uint64_t cap_words = (a.stream_bytes - payload_off) / 4;
    if (h32[0] != kMagic || h32[1] != 1u || h32[2] != a.n_seg || h32[3] != (uint32_t)kC || h32[4] != (uint32_t)kS ||
        h64[3] != a.n_elem || h64[4] != n_chunks || h64[5] > cap_words || h64[7] > a.stream_bytes ||
        h64[7] != align16(payload_off + 4ull * h64[5]))
        return false;
    if (reinterpret_cast<const uint64_t*>(stream + chunk_off)[n_chunks] != h64[5]) return false;
    atomicAdd(reinterpret_cast<unsigned long long*>(&a.res[0].payload_bits), (unsigned long long)h64[6]);
    atomicAdd(reinterpret_cast<unsigned long long*>(&a.res[0].container_bytes), (unsigned long long)h64[7]);
    return true;
}

__device__ void fail_all(const PrepArgs& a, int code) {
    a.ws.ctrl->abort = 1u;
    for (uint32_t u = 0; u < a.n_res; ++u) set_status(&a.res[u], code);
}

__device__ __forceinline__ uint64_t block_sum_u64(uint64_t x, uint64_t* scratch /* [8] */) {
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) x += __shfl_xor_sync(0xffffffffu, x, d);
    __syncthreads();
    if ((threadIdx.x & 31u) == 0) scratch[threadIdx.x >> 5] = x;
    __syncthreads();
    uint64_t sum = 0;
#pragma unroll
    for (int w = 0; w < kThreads / 32; ++w) sum += scratch[w];
    return sum;
}

// Block sums of three 64-bit values at once (two barriers); every thread receives them in x[].
__device__ __forceinline__ void block_sum3_u64(uint64_t (&x)[3], uint64_t* scratch /* [3 * 8] */) {
#pragma unroll
    for (int q = 0; q < 3; ++q) {
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) x[q] += __shfl_xor_sync(0xffffffffu, x[q], d);
    }
    __syncthreads();
    if ((threadIdx.x & 31u) == 0) {
#pragma unroll
        for (int q = 0; q < 3; ++q) scratch[q * 8 + (threadIdx.x >> 5)] = x[q];
    }
    __syncthreads();
#pragma unroll
    for (int q = 0; q < 3; ++q) {
        uint64_t sum = 0;
#pragma unroll
        for (int w = 0; w < kThreads / 32; ++w) sum += scratch[q * 8 + w];
        x[q] = sum;
    }
}

// Zeroes up to three word ranges: the state a call starts from (control block and failure marks, results, and where a
// call has them its histogram or completion counters), in one launch.
struct ClearArgs {
    uint32_t* p[3];
    uint64_t words[3];
};

__global__ void __launch_bounds__(kThreads) clear_kernel(ClearArgs a) {
    wait_for_previous_kernel();  // the kernels of the call before may still read what is cleared here
    const uint64_t step = (uint64_t)gridDim.x * kThreads;
#pragma unroll
    for (int r = 0; r < 3; ++r)
        for (uint64_t i = (uint64_t)blockIdx.x * kThreads + threadIdx.x; i < a.words[r]; i += step) a.p[r][i] = 0u;
}

__global__ void __launch_bounds__(kThreads) prepare_kernel(PrepArgs a) {
    wait_for_previous_kernel();
    __shared__ uint64_t s_red[3 * 8];
    __shared__ uint32_t s_kraft;
    __shared__ uint32_t s_scan[8];
    const uint32_t tid = threadIdx.x;
    const uint32_t k = blockIdx.x;
    const uint32_t G = a.tile_chunks;

    // this segment's descriptors, requested before the sums below need their first round trip to memory
    co3_seg sg{};
    co3_fmt f{};
    uint32_t len = 0, bits = 0;
    if (a.n_seg) {
        sg = a.segs[k];
        if (a.fmts && blockIdx.y == 0) f = a.fmts[k];
        if (a.codes && blockIdx.y == 0) {
            len = a.codes[k].len[tid];
            bits = a.codes[k].bits[tid];
        }
    }

    if (k == 0 && blockIdx.y == 0)
        for (uint32_t u = tid; u < a.n_res; u += kThreads) a.res[u].first_bad_chunk = 0xffffffffu;

    // ---- layout: elements, chunks and tiles of the segments before this one
    uint64_t before[3] = {0, 0, 0};  // elements, chunks, tiles
    bool bad = false;
    for (uint32_t i = tid; i < k && i < a.n_seg; i += kThreads) {
        const uint64_t n = a.segs[i].n_elem;
        if (n > a.n_elem) bad = true;
        const uint64_t c = (n + kC - 1) / kC;
        before[0] += n;
        before[1] += c;
        before[2] += (c + G - 1) / G;
    }
    block_sum3_u64(before, s_red);
    const uint64_t e_before = before[0], c_before = before[1], t_before = before[2];
    bad = __syncthreads_or(bad);
    if (a.n_seg == 0) {
        if (tid == 0) {
            Ctrl* c = a.ws.ctrl;
            c->n_chunks = 0;
            c->n_tiles = 0;
            c->chunk_off = align16(kHeaderBytes);
            c->sub_off = align16(c->chunk_off + 8ull);
            c->payload_off = c->sub_off;
            a.ws.first_chunk[0] = 0;
            if (a.n_elem != 0) fail_all(a, CO3_ERR_INVALID_ARG);
            else
                for (uint32_t u = 0; u < a.n_streams; ++u)
                    if (!header_ok(a, u, 0, c->chunk_off, c->payload_off)) fail_corrupt(a);
        }
        return;
    }
    const uint64_t my_chunks = sg.n_elem <= a.n_elem ? (sg.n_elem + kC - 1) / kC : 0;
    const uint64_t my_tiles = (my_chunks + G - 1) / G;
    if (sg.n_elem > a.n_elem || sg.elem_off != e_before || c_before + my_chunks > a.ws.n_chunks_max) bad = true;
    if (k == a.n_seg - 1 && e_before + sg.n_elem != a.n_elem) bad = true;
    if (bad) {
        if (tid == 0) fail_all(a, CO3_ERR_INVALID_ARG);
        return;
    }
    if (tid == 0 && blockIdx.y == 0) {
        a.ws.first_chunk[k] = (uint32_t)c_before;
        if (k == a.n_seg - 1) {
            const uint64_t nc = c_before + my_chunks;
            a.ws.first_chunk[a.n_seg] = (uint32_t)nc;
            Ctrl* c = a.ws.ctrl;
            c->n_chunks = (uint32_t)nc;
            c->n_tiles = (uint32_t)(t_before + my_tiles);
            c->chunk_off = align16(kHeaderBytes + 24ull * a.n_seg);
            c->sub_off = align16(c->chunk_off + 8ull * (nc + 1ull));
            c->payload_off = align16(c->sub_off + 2ull * nc * kSubs);
        }
    }
    // decode calls: every stream must describe exactly this layout (this block checks its segment's entry, the
    // last segment's block the headers)
    if (blockIdx.y == 0 && a.n_streams) {
        bool corrupt = false;
        for (uint32_t u = tid; u < a.n_streams; u += kThreads) {
            const uint8_t* stream = prep_stream(a, u);
            if (stream == nullptr || (reinterpret_cast<uintptr_t>(stream) & 15u) ||
                a.stream_bytes < kHeaderBytes + 24ull * (k + 1ull)) {
                corrupt = true;
                continue;
            }
            const uint64_t* e = reinterpret_cast<const uint64_t*>(stream + kHeaderBytes + 24ull * k);
            if (e[0] != sg.n_elem || e[1] != c_before) corrupt = true;
            if (k == a.n_seg - 1) {
                const uint64_t nc = c_before + my_chunks;
                const uint64_t chunk_off = align16(kHeaderBytes + 24ull * a.n_seg);
                const uint64_t payload_off = align16(align16(chunk_off + 8ull * (nc + 1ull)) + 2ull * nc * kSubs);
                if (!header_ok(a, u, nc, chunk_off, payload_off)) corrupt = true;
            }
        }
        if (corrupt) fail_corrupt(a);
    }
    // descriptors: blockIdx.y strides over them, so that one long segment is laid out by many blocks
    for (uint64_t c = (uint64_t)blockIdx.y * kThreads + tid; c < my_chunks; c += (uint64_t)gridDim.y * kThreads) {
        ChunkDesc d;
        d.seg = k;
        d.cnt = (uint32_t)min((uint64_t)kC, sg.n_elem - c * kC);
        d.elem0 = sg.elem_off + c * kC;
        d.cis = (uint32_t)c;
        d.pad = 0;
        a.ws.chunk_desc[c_before + c] = d;
    }
    for (uint64_t t = (uint64_t)blockIdx.y * kThreads + tid; t < my_tiles; t += (uint64_t)gridDim.y * kThreads) {
        TileDesc d;
        d.seg = k;
        d.chunk0 = (uint32_t)(c_before + t * G);
        d.n_chunks = (uint32_t)min((uint64_t)G, my_chunks - t * G);
        d.pad = 0;
        a.ws.tile_desc[t_before + t] = d;
    }
    if (blockIdx.y != 0) return;  // helper blocks only lay out descriptors

    // ---- format constants and value table
    bool fmt_ok = true;
    FmtDev fd{};
    if (a.fmts) {
        const uint32_t E = f.exp_bits, M = f.mant_bits;
        fmt_ok = E >= 2 && 1 + E + M <= 8 && (f.flags & ~CO3_FMT_FLUSH_SUBNORMALS) == 0 && f.scale > 0.0f &&
                 f.inv_scale > 0.0f && !isinf(f.scale) && !isinf(f.inv_scale);
        const int emin = fmt_ok ? -((1 << (E - 1)) - 2) : 0;
        if (fmt_ok) {
            fd.mant_bits = M;
            fd.mag_bits = E + M;
            fd.drop = 23u - M;
            fd.sign_shift = 31u - (E + M);
            fd.min_normal_bits = (uint32_t)(emin + 127) << 23;
            fd.code_bias = (uint32_t)(emin + 126) << M;
            fd.max_code = (((1u << E) - 2u) << M) | ((1u << M) - 1u);
            fd.top_bits = (fd.max_code + fd.code_bias) << (23u - M);
            fd.flush = (f.flags & CO3_FMT_FLUSH_SUBNORMALS) ? 1u : 0u;
            fd.fast = (M >= 1 && !fd.flush) ? 1u : 0u;
            fd.half_min_bits = (uint32_t)(emin - 1 + 127) << 23;
            fd.magic = __uint_as_float((uint32_t)(emin - (int)M + 23 + 127) << 23);
            fd.scale = f.scale;
            fd.inv_scale = f.inv_scale;
            const float top = __fmul_rn(__uint_as_float(fd.top_bits), f.inv_scale);
            if (isinf(top)) fmt_ok = false;
        }
        if (fmt_ok) {
            if (tid == 0) a.ws.fmt[k] = fd;
            // reconstructed value of symbol `tid`
            const uint32_t sym = tid, nb = fd.mag_bits;
            float val = 0.0f;
            if (sym < (2u << nb)) {
                const uint32_t sign = sym >> nb, code = sym & ((1u << nb) - 1u);
                const uint32_t efield = code >> M, mfield = code & ((1u << M) - 1u);
                float q = 0.0f;
                bool valid = efield != (1u << E) - 1u && !(sign && code == 0);
                if (efield == 0) {
                    if (fd.flush && mfield) valid = false;
                    q = __fmul_rn((float)mfield, __uint_as_float((uint32_t)(emin - (int)M + 127) << 23));
                } else {
                    q = __uint_as_float((code + fd.code_bias) << (23u - M));
                }
                if (valid) val = __fmul_rn(sign ? -q : q, f.inv_scale);
            }
            a.ws.val_lut[k * 256 + tid] = val;
        }
    }

    // ---- code tables
    bool code_ok = true;
    if (a.codes) {
        __shared__ uint32_t s_code[256];  // bits << 8 | len of every symbol
        // one bit per node of the binary code tree down to depth CO3_MAX_CODE_LEN: node (1 << len) + bits is the
        // codeword `bits` of `len` bits, its ancestors are its proper prefixes
        __shared__ uint32_t s_tree[(2u << CO3_MAX_CODE_LEN) / 32];
        if (tid == 0) s_kraft = 0;
        for (uint32_t i = tid; i < (2u << CO3_MAX_CODE_LEN) / 32; i += kThreads) s_tree[i] = 0;
        __syncthreads();
        if (len > CO3_MAX_CODE_LEN || (len && (bits >> len))) code_ok = false;
        if (tid == 255 && len) code_ok = false;  // 0xff is a symbol of no format: the decoder uses it as its error mark
        if (code_ok && len) atomicAdd(&s_kraft, 1u << (CO3_MAX_CODE_LEN - len));
        s_code[tid] = code_ok ? ((bits << 8) | len) : 0u;
        a.ws.enc_lut[k * 256 + tid] = (code_ok && len) ? ((bits << 8) | len) : kEncMissing;
        uint16_t* lut = a.ws.dec_lut + (size_t)k * kDecLut;
        uint16_t* sub = a.ws.dec_sub + (size_t)k * kSubLut;
        if (a.want_dec) {
            for (uint32_t i = tid; i < (uint32_t)kDecLut / 2; i += kThreads)
                reinterpret_cast<uint32_t*>(lut)[i] = kDecInvalid | (kDecInvalid << 16);
            for (uint32_t i = tid; i < (uint32_t)kSubLut / 2; i += kThreads)
                reinterpret_cast<uint32_t*>(sub)[i] = kDecInvalid | (kDecInvalid << 16);
        }
        __syncthreads();
        if (s_kraft > (1u << CO3_MAX_CODE_LEN)) code_ok = false;  // over-subscribed: cannot be prefix-free
        // no codeword may start with another one (equal codewords included): every thread marks its node, then
        // looks for a mark on the way up to the root
        const uint32_t node = (1u << len) + bits;
        if (code_ok && len) {
            const uint32_t old = atomicOr(&s_tree[node >> 5], 1u << (node & 31u));
            if (old & (1u << (node & 31u))) code_ok = false;
        }
        __syncthreads();
        if (code_ok && len) {
            for (uint32_t up = 1; up < len; ++up) {
                const uint32_t anc = node >> up;
                if (s_tree[anc >> 5] & (1u << (anc & 31u))) code_ok = false;
            }
        }
        code_ok = __syncthreads_and(code_ok);
        if (code_ok && a.want_dec) {
            // short codewords fill every table entry they prefix: one warp per symbol, lanes over the span
            for (uint32_t sym = tid >> 5; sym < 256; sym += kThreads / 32) {
                const uint32_t l = s_code[sym] & 0xffu, b = s_code[sym] >> 8;
                if (l == 0 || l > (uint32_t)kDecBits) continue;
                const uint32_t span = 1u << (kDecBits - l), first = b << (kDecBits - l);
                for (uint32_t i = tid & 31u; i < span; i += 32) lut[first + i] = (uint16_t)((l << 8) | sym);
            }
            // longer codewords: mark their 12-bit prefix, number the marked prefixes, fill one 16-entry
            // second-level table per prefix
            const bool is_long = len > (uint32_t)kDecBits;
            const uint32_t prefix = is_long ? (bits >> (len - kDecBits)) : 0u;
            if (is_long) lut[prefix] = (uint16_t)kDecLong;
            __syncthreads();
            const uint32_t per = kDecLut / kThreads;
            uint32_t marked = 0;
            for (uint32_t i = 0; i < per; ++i) marked += (lut[tid * per + i] == kDecLong) ? 1u : 0u;
            uint32_t total;
            uint32_t idx = block_exclusive_scan_256(marked, s_scan, &total);
            for (uint32_t i = 0; i < per; ++i)
                if (lut[tid * per + i] == kDecLong) lut[tid * per + i] = (uint16_t)(kDecLong | (idx++ & 0xffu));
            __syncthreads();
            if (is_long) {
                const uint32_t t = lut[prefix] & 0xffu;
                const uint32_t rest = len - kDecBits;  // 1..4 bits beyond the prefix
                const uint32_t first = (bits & ((1u << rest) - 1u)) << (kSubBits - rest);
                for (uint32_t i = 0; i < (1u << (kSubBits - rest)); ++i)
                    sub[t * (1u << kSubBits) + first + i] = (uint16_t)((len << 8) | tid);
            }
        }
    }
    if ((!fmt_ok || !code_ok) && tid == 0) fail_all(a, CO3_ERR_INVALID_ARG);
}

// ------------------------------------------------------------------------------------------------
// Element access for one thread.  In the client kernels thread t owns two groups of four consecutive elements of a
// chunk, half a chunk apart: elements 4t .. 4t+3 and kC/2 + 4t .. kC/2 + 4t+3 (register j holds element
// 4t + (j & 3) + (j >> 2) * kC/2).  A warp's 16-byte accesses are then contiguous, in the shared-memory ring (no bank
// conflicts) and in global memory (whole lines per store).  The moment sums keep eight consecutive elements.
// ------------------------------------------------------------------------------------------------
constexpr uint32_t kHalf = kC / 2;
static_assert(kC == 8 * kThreads, "eight elements of a chunk per thread");

// The helpers below take the distance kQ between the two groups (kHalf in the 256-thread kernels; the packer's
// 128 threads own two such pairs each, kQuarter apart) and q0, the place of the first group in the chunk.
constexpr uint32_t kQuarter = kC / 4;

// Bit j set: register j holds an element of a chunk of `cnt` elements.
template <uint32_t kQ>
__device__ __forceinline__ uint32_t quads_valid(uint32_t cnt, uint32_t q0) {
    const uint32_t na = cnt > q0 ? min(4u, cnt - q0) : 0u;
    const uint32_t nb = cnt > q0 + kQ ? min(4u, cnt - q0 - kQ) : 0u;
    return ((1u << na) - 1u) | (((1u << nb) - 1u) << 4);
}

// p: the chunk's first element + q0
template <uint32_t kQ>
__device__ __forceinline__ void store_quads_vec(float* __restrict__ p, const float (&x)[8]) {
    *reinterpret_cast<float4*>(p) = make_float4(x[0], x[1], x[2], x[3]);
    *reinterpret_cast<float4*>(p + kQ) = make_float4(x[4], x[5], x[6], x[7]);
}

template <uint32_t kQ>
__device__ __forceinline__ void load_quads_any(const float* __restrict__ p, uint32_t valid, float (&x)[8]) {
#pragma unroll
    for (int j = 0; j < 8; ++j) x[j] = ((valid >> j) & 1u) ? p[(j & 3) + (j >> 2) * kQ] : 0.0f;
}

template <uint32_t kQ>
__device__ __forceinline__ void store_quads_any(float* __restrict__ p, uint32_t valid, const float (&x)[8]) {
#pragma unroll
    for (int j = 0; j < 8; ++j)
        if ((valid >> j) & 1u) p[(j & 3) + (j >> 2) * kQ] = x[j];
}

__device__ __forceinline__ void load8_vec(const float* __restrict__ p, float (&x)[8]) {
    const float4 a = __ldg(reinterpret_cast<const float4*>(p));
    const float4 b = __ldg(reinterpret_cast<const float4*>(p) + 1);
    x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w;
    x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
}

__device__ __forceinline__ void load8_any(const float* __restrict__ p, uint32_t n_valid, float (&x)[8]) {
#pragma unroll
    for (int j = 0; j < 8; ++j) x[j] = (uint32_t)j < n_valid ? p[j] : 0.0f;
}

__device__ __forceinline__ uint2 pack_sym8(const uint32_t (&s)[8]) {
    uint2 w;
    w.x = __byte_perm(__byte_perm(s[0], s[1], 0x0040), __byte_perm(s[2], s[3], 0x0040), 0x5410);
    w.y = __byte_perm(__byte_perm(s[4], s[5], 0x0040), __byte_perm(s[6], s[7], 0x0040), 0x5410);
    return w;
}

// Adds the saturated / non-finite counts of a warp to the client's result.
__device__ __forceinline__ void add_counts(co3_result* r, uint32_t n_sat, uint32_t n_nf) {
    if (__any_sync(0xffffffffu, (n_sat | n_nf) != 0)) {
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) {
            n_sat += __shfl_xor_sync(0xffffffffu, n_sat, d);
            n_nf += __shfl_xor_sync(0xffffffffu, n_nf, d);
        }
        if ((threadIdx.x & 31u) == 0) {
            if (n_sat) atomicAdd(reinterpret_cast<unsigned long long*>(&r->n_saturated), (unsigned long long)n_sat);
            if (n_nf) {
                atomicAdd(reinterpret_cast<unsigned long long*>(&r->n_nonfinite), (unsigned long long)n_nf);
                set_status(r, CO3_ERR_NONFINITE);
            }
        }
    }
}

// Where a thread's eight elements lie, for the draws of a dithered conversion: the call's seed, client, layer, and
// the place of the first of them inside the layer (a multiple of 4; the second group of four lies kQ further on).
struct Place {
    uint32_t seed, client, layer;
    uint64_t first;
};

// Correct + convert + memory update of 8 elements held in registers (Algorithm 1, client side).
// kWhole: all eight are valid, so the branch-free converter may be used; otherwise bit j of `valid` says whether
// register j holds an element.  Symbols land in s[], the new memory in mo[]; counters accumulate in n_sat / n_nf.
// kDither: the instance of the dithered entry points: one draw per element (four per block of the draw stream)
// decides between the two levels around its value.
// ring_g / ring_m (kWhole only): the thread's first gradient and memory value in the shared-memory ring, from which
// the rare second look at a group reads them again, so that the registers holding them are free once the first
// look is done.
template <bool kWhole, bool kDither, uint32_t kQ>
__device__ __forceinline__ void convert8(const float (&g)[8], const float (&m)[8], uint32_t valid, float decay,
                                         const FmtDev& f, const Place& at, float (&mo)[8], uint32_t (&s)[8],
                                         uint32_t& n_sat, uint32_t& n_nf, const float* ring_g = nullptr,
                                         const float* ring_m = nullptr) {
    if (kDither) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const uint64_t b = (at.first >> 2) + (uint32_t)h * (kQ / 4u);
            const uint4 r = philox4x32_10(make_uint4((uint32_t)b, (uint32_t)(b >> 32), at.client, at.layer), at.seed, 0u);
            const uint32_t R[4] = {r.x >> 8, r.y >> 8, r.z >> 8, r.w >> 8};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int j = 4 * h + q;
                uint32_t fl = 0;
                mo[j] = convert_one_dither(g[j], m[j], decay, f, R[q], s[j], fl);
                if ((valid >> j) & 1u) { n_sat += fl & 1u; n_nf += fl >> 1; }
            }
        }
        return;
    }
    if (kWhole && f.fast) {
        bool beyond = false;
#pragma unroll
        for (int j = 0; j < 8; ++j) mo[j] = convert_fast(g[j], m[j], decay, f, s[j], beyond);
        if (beyond) {  // a saturating or non-finite input: the clamp above already gave a finite one its level and
                       // memory, it only has to be counted; a NaN or an infinity sends the group through convert_one
            const float top = __uint_as_float(f.top_bits);
            float g2[8], m2[8];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const float4 x = *reinterpret_cast<const float4*>(ring_g + h * kQ);
                const float4 y = *reinterpret_cast<const float4*>(ring_m + h * kQ);
                g2[4 * h] = x.x; g2[4 * h + 1] = x.y; g2[4 * h + 2] = x.z; g2[4 * h + 3] = x.w;
                m2[4 * h] = y.x; m2[4 * h + 1] = y.y; m2[4 * h + 2] = y.z; m2[4 * h + 3] = y.w;
            }
            uint32_t sat = 0;
            bool again = false;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const float v = __fmaf_rn(decay, m2[j], g2[j]);
                again |= !(fabsf(v) < __uint_as_float(0x7f800000u));
                sat += (fabsf(__fmul_rn(v, f.scale)) > top) ? 1u : 0u;
            }
            if (!again) {
                n_sat += sat;
            } else {
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    uint32_t fl = 0;
                    mo[j] = convert_one(g2[j], m2[j], decay, f, s[j], fl);
                    n_sat += fl & 1u;
                    n_nf += fl >> 1;
                }
            }
        }
        return;
    }
    const bool redo = true;
    if (redo) {  // generic formats, ragged groups, and groups that hold a non-finite input
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            uint32_t fl = 0;
            mo[j] = convert_one(g[j], m[j], decay, f, s[j], fl);
            if ((valid >> j) & 1u) { n_sat += fl & 1u; n_nf += fl >> 1; }
        }
    }
}

// ------------------------------------------------------------------------------------------------
// Work feed of the persistent client kernels.  A work item is one chunk of one client; block b takes
// items b, b + gridDim.x, ...  Thread 0 runs one item ahead: while the block works on item k it has
// already started two bulk copies (gradient and memory of item k + 1, 8 KB each) into the other half
// of a two-stage shared-memory ring, completed on that stage's mbarrier.  Chunks that are short or not
// 16-byte aligned are not copied; their threads load from global memory directly.
// ------------------------------------------------------------------------------------------------
struct alignas(16) FeedItem {
    ChunkDesc d;
    uint64_t base;    // index of the chunk's first element from the batch base pointer
    uint32_t client;
    uint32_t tma;     // 1: gradient and memory arrive in the ring
    uint32_t valid;   // 0: no more work
    uint32_t chunk;   // chunk index inside the client
};

// Thread 0's position in the item sequence.  Items are numbered client-major (item = client * n_chunks + chunk)
// and handed out in groups of `group` consecutive items: block b takes groups b, b + gridDim.x, ...  Consecutive
// chunks mostly belong to one layer, so a block changes tables (and flushes its private histograms) rarely.  The
// cursor moves by one item inside a group and by the distance to the block's next group at its end, both as
// (whole clients, chunks) pairs worked out once: no 64-bit division per item.
struct FeedCursor {
    uint32_t client, chunk;            // the item to publish next
    uint32_t jump_client, jump_chunk;  // from the last item of a group to the first of the block's next group
    uint32_t group, j;                 // items per group; place of the next item inside its group
    __device__ __forceinline__ void init(uint32_t n_chunks, uint32_t grp) {
        const uint64_t first = (uint64_t)blockIdx.x * grp, jump = (uint64_t)(gridDim.x - 1u) * grp + 1u;
        client = (uint32_t)(first / n_chunks);
        chunk = (uint32_t)(first % n_chunks);
        jump_client = (uint32_t)(jump / n_chunks);
        jump_chunk = (uint32_t)(jump % n_chunks);
        group = grp;
        j = 0;
    }
    __device__ __forceinline__ void advance(uint32_t n_chunks) {
        if (++j < group) {
            ++chunk;
        } else {
            j = 0;
            client += jump_client;
            chunk += jump_chunk;
        }
        if (chunk >= n_chunks) { chunk -= n_chunks; ++client; }
    }
};

struct alignas(16) Feed {
    float g[2][kC];
    float m[2][kC];
    uint64_t bar[2];
    FeedItem item[2];
    FmtDev fmt[2];    // converter constants of the item in each slot
    FeedCursor cur;   // thread 0's place in the item sequence (kept here to spare every thread the registers)
    uint32_t fail;    // set by any thread whose wait for a copy gave up; the block leaves its item loop at the next barrier
};

static_assert(sizeof(Feed) % 16 == 0, "what follows a Feed in shared memory is accessed 16 bytes at a time");

struct FeedArgs {
    const float* grad;
    const float* mem;
    uint64_t client_stride;
    uint32_t n_clients;
};

// Thread 0 only: publishes the cursor's item in ring slot `slot` and starts its copies.  `next` holds the chunk
// descriptor fetched one call earlier for exactly this item; the cursor moves on and `next` is refilled.
__device__ __forceinline__ void feed_issue(Feed& fd, const FeedArgs& fa, const Ws& ws, uint32_t n_chunks, uint32_t slot,
                                           ChunkDesc& next, bool use_tma) {
    FeedCursor cur = fd.cur;
    FeedItem it;
    it.valid = cur.client < fa.n_clients ? 1u : 0u;
    it.d = next;
    it.client = cur.client;
    it.chunk = cur.chunk;
    it.base = 0;
    it.tma = 0;
    if (it.valid) {
        it.base = (uint64_t)it.client * fa.client_stride + it.d.elem0;
        const uintptr_t pg = reinterpret_cast<uintptr_t>(fa.grad + it.base), pm = reinterpret_cast<uintptr_t>(fa.mem + it.base);
        it.tma = (use_tma && it.d.cnt == (uint32_t)kC && ((pg | pm) & 15u) == 0) ? 1u : 0u;
    }
    fd.item[slot] = it;
    if (it.tma) {
        fence_async_smem();
        mbar_arrive_expect_tx(&fd.bar[slot], 2u * kC * 4u);
        bulk_copy_g2s(fd.g[slot], fa.grad + it.base, kC * 4u, &fd.bar[slot]);
        bulk_copy_g2s(fd.m[slot], fa.mem + it.base, kC * 4u, &fd.bar[slot]);
    }
    cur.advance(n_chunks);
    fd.cur = cur;
    if (cur.client < fa.n_clients) next = ws.chunk_desc[cur.chunk];
}

// The first threads of warp 0 copy the converter constants of the item in ring slot `slot` next to it; visible to the
// block after its next barrier.
__device__ __forceinline__ void feed_fetch_fmt(Feed& fd, const Ws& ws, uint32_t slot) {
    static_assert(sizeof(FmtDev) % 4 == 0 && sizeof(FmtDev) / 4 <= 32, "FmtDev is copied word by word by one warp");
    __syncwarp();  // the publishing thread 0 shares a warp with the copying threads
    if (threadIdx.x < sizeof(FmtDev) / 4 && fd.item[slot].valid)
        reinterpret_cast<uint32_t*>(&fd.fmt[slot])[threadIdx.x] =
            reinterpret_cast<const uint32_t*>(&ws.fmt[fd.item[slot].d.seg])[threadIdx.x];
}

// All threads: waits for the current item's copies, if it has any.  Returns false if they never arrived (never
// expected).  `parity` holds, per ring slot, the phase parity of the next copy to wait for.
__device__ __forceinline__ bool feed_wait(Feed& fd, const FeedItem& it, uint32_t k, uint32_t& parity) {
    if (!it.tma) return true;
    const uint32_t slot = k & 1u;
    const bool ok = mbar_wait(&fd.bar[slot], (parity >> slot) & 1u);
    parity ^= 1u << slot;
    if (!ok) fd.fail = 1u;
    return ok;
}

// All threads, after feed_wait: the gradient and memory values of the current item that lie in the thread's two groups
// at q0 and q0 + kQ (`valid` as quads_valid gives it).
template <uint32_t kQ>
__device__ __forceinline__ void feed_get(const Feed& fd, const FeedArgs& fa, const FeedItem& it, uint32_t k, uint32_t q0,
                                         uint32_t valid, float (&g)[8], float (&m)[8]) {
    if (it.tma) {
        const uint32_t slot = k & 1u;
        const float4 a = *reinterpret_cast<const float4*>(&fd.g[slot][q0]);
        const float4 b = *reinterpret_cast<const float4*>(&fd.g[slot][q0 + kQ]);
        const float4 c = *reinterpret_cast<const float4*>(&fd.m[slot][q0]);
        const float4 d = *reinterpret_cast<const float4*>(&fd.m[slot][q0 + kQ]);
        g[0] = a.x; g[1] = a.y; g[2] = a.z; g[3] = a.w; g[4] = b.x; g[5] = b.y; g[6] = b.z; g[7] = b.w;
        m[0] = c.x; m[1] = c.y; m[2] = c.z; m[3] = c.w; m[4] = d.x; m[5] = d.y; m[6] = d.z; m[7] = d.w;
    } else {
        load_quads_any<kQ>(fa.grad + it.base + q0, valid, g);
        load_quads_any<kQ>(fa.mem + it.base + q0, valid, m);
    }
}

// A wait gave up and the block has left its item loop after item k: thread 0 still waits (bounded again) for the
// copies it had started for item k + 1, so that nothing is in flight into this block's shared memory when it exits.
__device__ __forceinline__ void feed_drain(Feed& fd, uint32_t k, uint32_t parity) {
    const uint32_t slot = (k + 1u) & 1u;
    if (threadIdx.x == 0 && fd.item[slot].valid && fd.item[slot].tma) mbar_wait(&fd.bar[slot], (parity >> slot) & 1u);
}

// ------------------------------------------------------------------------------------------------
// convert: persistent blocks over (chunk, client) items
// ------------------------------------------------------------------------------------------------
struct ConvertArgs {
    const float* grad;
    float* mem;
    float decay;
    uint64_t client_stride;
    uint32_t n_clients;
    uint8_t* sym_out;    // nullable
    uint64_t* hist_out;  // nullable
    co3_result* res;
    uint32_t group;      // consecutive items a block takes at a time
    uint32_t seed;       // key of the draw stream (dithered entry points)
    Ws ws;
};

constexpr int kHistCopies = 8;    // private histograms per block, spread over the lanes
constexpr int kHistStride = 260;  // words between copies: shifts each copy by four banks

// One thread's part of one work item once its inputs are in registers: conversion, new memory, symbols, counts.
// kWhole: the chunk is complete and came through the ring (every register holds an element, 16-byte accesses).
// q0, kQ: the thread's two groups of four lie at q0 and q0 + kQ in the chunk.
template <bool kSym, bool kHist, bool kMem, bool kDither, bool kWhole, uint32_t kQ>
__device__ __forceinline__ void convert_item(const ConvertArgs& a, Feed& fd, const FeedItem& it, uint64_t k, const FmtDev& f,
                                             uint32_t q0, uint32_t valid, const float (&g)[8], const float (&m)[8],
                                             uint32_t* s_hist, uint32_t& n_sat, uint32_t& n_nf) {
    const uint64_t e = it.base + q0;
    const Place at{a.seed, it.client, it.d.seg, (uint64_t)it.d.cis * kC + q0};
    float mo[8];
    uint32_t s[8];
    if (kWhole) {
        convert8<true, kDither, kQ>(g, m, 0xffu, a.decay, f, at, mo, s, n_sat, n_nf, &fd.g[k & 1u][q0], &fd.m[k & 1u][q0]);
        if (kMem) store_quads_vec<kQ>(a.mem + e, mo);
    } else {
        convert8<false, kDither, kQ>(g, m, valid, a.decay, f, at, mo, s, n_sat, n_nf);
        if (kMem) store_quads_any<kQ>(a.mem + e, valid, mo);
    }
    if (kSym) {
        if (kWhole && (reinterpret_cast<uintptr_t>(a.sym_out + e) & 3u) == 0) {
            const uint2 w = pack_sym8(s);
            *reinterpret_cast<uint32_t*>(a.sym_out + e) = w.x;
            *reinterpret_cast<uint32_t*>(a.sym_out + e + kQ) = w.y;
        } else {
#pragma unroll
            for (int j = 0; j < 8; ++j)
                if (kWhole || ((valid >> j) & 1u)) a.sym_out[e + (j & 3) + (j >> 2) * kQ] = (uint8_t)s[j];
        }
    }
    if (kHist) {
        uint32_t* h = s_hist + (threadIdx.x & (kHistCopies - 1)) * kHistStride;
#pragma unroll
        for (int j = 0; j < 8; ++j)
            if (kWhole || ((valid >> j) & 1u)) atomicAdd(&h[s[j]], 1u);
    }
}

// kMem: the new memory is stored (false: a dry pass that only counts symbols and leaves every input untouched).
// kDither: the instance behind the dithered entry points (stochastic choice between the two levels around a value).
// kT: threads of a block, 256 (eight elements of a chunk per thread) or 128 (sixteen, as in the packer: the dry pass,
// whose blocks would otherwise spend much of their time at the barrier of eight warps).
template <bool kSym, bool kHist, bool kMem, bool kDither, int kT>
__global__ void __launch_bounds__(kT, kT == 128 ? 5 : ((kMem || kDither) ? 3 : 4)) convert_kernel(ConvertArgs a) {
    wait_for_previous_kernel();
    static_assert(kT == 256 || kT == 128, "a thread owns eight or sixteen elements of a chunk");
    constexpr uint32_t kQ = kT == 256 ? kHalf : kQuarter;  // distance between the two groups of a pair
    extern __shared__ __align__(16) unsigned char smem_raw[];
    Feed& fd = *reinterpret_cast<Feed*>(smem_raw);
    uint32_t* s_hist = reinterpret_cast<uint32_t*>(smem_raw + sizeof(Feed));
    const Ctrl* ctrl = a.ws.ctrl;
    if (ctrl->abort) return;
    const uint32_t tid = threadIdx.x;
    const uint32_t n_chunks = ctrl->n_chunks;
    const FeedArgs fa{a.grad, a.mem, a.client_stride, a.n_clients};
    if ((uint64_t)blockIdx.x * a.group >= (uint64_t)n_chunks * a.n_clients) return;

    ChunkDesc next{};
    if (tid == 0) {
        mbar_init(&fd.bar[0], 1);
        mbar_init(&fd.bar[1], 1);
        fd.fail = 0u;
        fd.cur.init(n_chunks, a.group);
        next = a.ws.chunk_desc[fd.cur.chunk];
        feed_issue(fd, fa, a.ws, n_chunks, 0, next, true);
    }
    if (kHist)
        for (uint32_t i = tid; i < (uint32_t)(kHistStride * kHistCopies); i += kT) s_hist[i] = 0;
    __syncthreads();
    feed_fetch_fmt(fd, a.ws, 0);
    __syncthreads();

    uint32_t n_sat = 0, n_nf = 0, hist_seg = 0xffffffffu, cur_client = 0, parity = 0;
    bool hw_fail = false;
    const uint32_t q0 = tid * 4;
    for (uint64_t k = 0;; ++k) {
        if (tid == 0) feed_issue(fd, fa, a.ws, n_chunks, (uint32_t)(k + 1) & 1u, next, true);
        const FeedItem it = fd.item[k & 1u];
        if (!it.valid) break;
        if (it.client != cur_client) {  // counters are per client
            add_counts(&a.res[cur_client], n_sat, n_nf);
            n_sat = n_nf = 0;
            cur_client = it.client;
        }
        if (kHist && it.d.seg != hist_seg) {  // flush the private histograms when the segment changes
            __syncthreads();
            if (hist_seg != 0xffffffffu) {
                for (uint32_t b = tid; b < 256u; b += kT) {
                    uint32_t c = 0;
#pragma unroll
                    for (int i = 0; i < kHistCopies; ++i) { c += s_hist[b + i * kHistStride]; s_hist[b + i * kHistStride] = 0; }
                    if (c) atomicAdd(reinterpret_cast<unsigned long long*>(&a.hist_out[(size_t)hist_seg * 256 + b]), (unsigned long long)c);
                }
            }
            hist_seg = it.d.seg;
            __syncthreads();
        }
        const FmtDev f = fd.fmt[k & 1u];
        // a copy that never arrived (never expected): this thread writes nothing for the item, the block stops
        if (!feed_wait(fd, it, (uint32_t)k, parity)) {
            hw_fail = true;
        } else {
#pragma unroll
            for (uint32_t part = 0; part < 256u / kT; ++part) {  // one pair of groups, or two pairs half a chunk apart
                const uint32_t qp = q0 + part * kHalf;
                const uint32_t valid = it.tma ? 0xffu : quads_valid<kQ>(it.d.cnt, qp);
                float g[8], m[8];
                feed_get<kQ>(fd, fa, it, (uint32_t)k, qp, valid, g, m);
                if (it.tma) convert_item<kSym, kHist, kMem, kDither, true, kQ>(a, fd, it, k, f, qp, 0xffu, g, m, s_hist, n_sat, n_nf);
                else if (valid) convert_item<kSym, kHist, kMem, kDither, false, kQ>(a, fd, it, k, f, qp, valid, g, m, s_hist, n_sat, n_nf);
            }
        }
        feed_fetch_fmt(fd, a.ws, (uint32_t)(k + 1) & 1u);  // item k + 1 was published before the previous barrier
        __syncthreads();  // everyone has read ring slot k & 1 and item[k & 1] before thread 0 reuses them
        if (fd.fail) {    // the same for every thread: written before the barrier
            feed_drain(fd, (uint32_t)k, parity);
            break;
        }
    }
    add_counts(&a.res[cur_client], n_sat, n_nf);
    if (kHist) {
        __syncthreads();
        if (hist_seg != 0xffffffffu) {
            for (uint32_t b = tid; b < 256u; b += kT) {
                uint32_t c = 0;
#pragma unroll
                for (int i = 0; i < kHistCopies; ++i) c += s_hist[b + i * kHistStride];
                if (c) atomicAdd(reinterpret_cast<unsigned long long*>(&a.hist_out[(size_t)hist_seg * 256 + b]), (unsigned long long)c);
            }
        }
    }
    if (__syncthreads_or(hw_fail)) {  // the block stopped early, items of any client may be missing: the call fails
        for (uint32_t u = tid; u < a.n_clients; u += kT) set_status(&a.res[u], CO3_ERR_CUDA);
    }
}

// ------------------------------------------------------------------------------------------------
// pack: persistent blocks over (chunk, client) items.  Thread t owns symbols 4t .. 4t+3 and kC/2 + 4t .. kC/2 + 4t+3
// of the chunk.
// ------------------------------------------------------------------------------------------------
struct PackArgs {
    const float* grad;   // fused path
    float* mem;
    float decay;
    const uint8_t* sym;  // symbol path
    uint64_t client_stride;
    uint32_t n_clients;
    uint8_t* streams;
    size_t stream_capacity;
    co3_result* res;
    uint32_t group;      // consecutive items a block takes at a time
    uint32_t seed;       // key of the draw stream (dithered entry point)
    Ws ws;
};

// ORs an n-bit value (v, right-aligned, n <= 64, bits above n clear) into the chunk's bit buffer so that its
// last bit lands on stream bit end-1 (most significant bit first).  Words that receive only zeros are skipped.
__device__ __forceinline__ void or_if_nonzero(uint32_t word_addr, uint32_t v) {
    asm volatile("red.shared.or.b32 [%0], %1;" : : "r"(word_addr), "r"(v) : "memory");
}

// buf_addr: shared-window byte address of the chunk's bit buffer.
__device__ __forceinline__ void put_bits(uint32_t buf_addr, uint32_t end, uint64_t v) {
    const uint32_t lo = (uint32_t)v, hi = (uint32_t)(v >> 32);
    const uint32_t q = (0u - end) & 31u;  // free bits behind the value in its last word
    const uint32_t last = buf_addr + (((end + 31u) >> 5) << 2);  // one past the last word touched
    or_if_nonzero(last - 4u, lo << q);
    or_if_nonzero(last - 8u, __funnelshift_l(lo, hi, q));
    or_if_nonzero(last - 12u, __funnelshift_l(hi, 0u, q));
}


constexpr int kBitWords = kSlotWords;  // bit buffer of one chunk
constexpr int kPackThreads = 128;      // threads of a packing block: 16 symbols of a chunk each
constexpr int kPackWarps = kPackThreads / 32;
static_assert(kC == 16 * kPackThreads && kQuarter == 4 * kPackThreads, "four groups of four symbols per packing thread, a quarter chunk apart");
static_assert(kBitWords == 8 * kPackThreads, "two uint4 of the bit buffer per packing thread");

// Exclusive prefix sums of two words over the threads of a packing block with one barrier; tot[] receives the block
// sums.  scratch: 2 * kPackWarps words that no thread writes again before the block's next barrier after this call.
__device__ __forceinline__ void pack_scan2(const uint32_t (&x)[2], uint32_t* scratch, uint32_t (&ex)[2], uint32_t (&tot)[2]) {
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    uint32_t inc0 = x[0], inc1 = x[1];
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t y0 = __shfl_up_sync(0xffffffffu, inc0, d), y1 = __shfl_up_sync(0xffffffffu, inc1, d);
        if (lane >= (uint32_t)d) { inc0 += y0; inc1 += y1; }
    }
    if (lane == 31u) { scratch[warp] = inc0; scratch[kPackWarps + warp] = inc1; }
    __syncthreads();
    // the first lanes hold the warp sums; warp-wide reductions give the block totals and this warp's bases
    const uint32_t s0 = lane < (uint32_t)kPackWarps ? scratch[lane] : 0u;
    const uint32_t s1 = lane < (uint32_t)kPackWarps ? scratch[kPackWarps + lane] : 0u;
    tot[0] = __reduce_add_sync(0xffffffffu, s0);
    tot[1] = __reduce_add_sync(0xffffffffu, s1);
    ex[0] = __reduce_add_sync(0xffffffffu, lane < warp ? s0 : 0u) + inc0 - x[0];
    ex[1] = __reduce_add_sync(0xffffffffu, lane < warp ? s1 : 0u) + inc1 - x[1];
}

// Where the results of one work item go, worked out once per item by thread 0.
struct alignas(16) PackOut {
    uint16_t* sub;       // the chunk's 16 sub-chunk offsets in the client's container
    uint32_t* slot;      // the chunk's worst-case slot in the workspace
    uint32_t* chunk_bits;
    co3_result* res;     // the client's result
};

struct PackSmem {
    Feed feed;
    alignas(16) uint32_t bits[2][kBitWords];  // cleared and copied out 16 bytes at a time
    uint32_t enc[256];
    uint32_t scan[2][2 * kPackWarps];
    PackOut out[2];
    FeedCursor out_cur;  // the place in the item sequence of the thread that works out the output locations
};

// Eight of a packing thread's sixteen symbols (two groups of four, at q0 and q0 + kQuarter in the chunk): converted
// here unless kFromSym, then their codewords, each group's concatenated into at most 64 bits (wa, wb) of la and lb
// bits.  kWhole: the chunk is complete (and, on the fused path, was delivered through the ring).  `any` collects
// the table entries (for the no-codeword bit).  ok: what feed_wait returned.
template <bool kFromSym, bool kWhole, bool kDither>
__device__ __forceinline__ void pack_eight(const PackArgs& a, PackSmem& sm, const FeedArgs& fa, const FeedItem& it, uint32_t k,
                                           uint32_t q0, bool ok, uint32_t& n_sat, uint32_t& n_nf, uint32_t& la, uint32_t& lb,
                                           uint64_t& wa, uint64_t& wb, uint32_t& any) {
    const uint32_t valid = kWhole ? 0xffu : quads_valid<kQuarter>(it.d.cnt, q0);
    const uint64_t e = it.base + q0;
    uint32_t s[8];
    if (kFromSym) {
        if (kWhole && (reinterpret_cast<uintptr_t>(a.sym + e) & 3u) == 0) {
            const uint32_t wx = __ldg(reinterpret_cast<const uint32_t*>(a.sym + e));
            const uint32_t wy = __ldg(reinterpret_cast<const uint32_t*>(a.sym + e + kQuarter));
#pragma unroll
            for (int j = 0; j < 4; ++j) { s[j] = (wx >> (8 * j)) & 0xffu; s[4 + j] = (wy >> (8 * j)) & 0xffu; }
        } else {
#pragma unroll
            for (int j = 0; j < 8; ++j) s[j] = ((valid >> j) & 1u) ? a.sym[e + (j & 3) + (j >> 2) * kQuarter] : 0u;
        }
    } else {
        const FmtDev f = sm.feed.fmt[k & 1u];
        const Place at{a.seed, it.client, it.d.seg, (uint64_t)it.d.cis * kC + q0};
        float g[8], m[8], mo[8];
        if (ok) feed_get<kQuarter>(sm.feed, fa, it, k, q0, valid, g, m);
        if (!ok) {  // the copies never arrived (never expected): the memory is left alone, the block stops after this item
#pragma unroll
            for (int j = 0; j < 8; ++j) s[j] = 0u;
        } else if (kWhole) {
            convert8<true, kDither, kQuarter>(g, m, 0xffu, a.decay, f, at, mo, s, n_sat, n_nf, &sm.feed.g[k & 1u][q0], &sm.feed.m[k & 1u][q0]);
            store_quads_vec<kQuarter>(a.mem + e, mo);
        } else if (valid) {
            convert8<false, kDither, kQuarter>(g, m, valid, a.decay, f, at, mo, s, n_sat, n_nf);
            store_quads_any<kQuarter>(a.mem + e, valid, mo);
        }
    }
    uint32_t ent[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) ent[j] = (kWhole || ((valid >> j) & 1u)) ? sm.enc[s[j]] : 0u;
    any |= ent[0] | ent[1] | ent[2] | ent[3] | ent[4] | ent[5] | ent[6] | ent[7];
    // the low byte of an entry is its length, at most 16: sums of four stay inside the byte
    la = (ent[0] + ent[1] + ent[2] + ent[3]) & 0xffu;
    lb = (ent[4] + ent[5] + ent[6] + ent[7]) & 0xffu;
    const uint32_t c01 = ((ent[0] >> 8) << (ent[1] & 0xffu)) | (ent[1] >> 8);
    const uint32_t c23 = ((ent[2] >> 8) << (ent[3] & 0xffu)) | (ent[3] >> 8);
    const uint32_t c45 = ((ent[4] >> 8) << (ent[5] & 0xffu)) | (ent[5] >> 8);
    const uint32_t c67 = ((ent[6] >> 8) << (ent[7] & 0xffu)) | (ent[7] >> 8);
    wa = ((uint64_t)c01 << ((ent[2] + ent[3]) & 0xffu)) | c23;
    wb = ((uint64_t)c45 << ((ent[6] + ent[7]) & 0xffu)) | c67;
}

// One work item of the pack kernel for one thread: its 16 symbols (groups of four at 4t, 4t + kQuarter, ...), the
// block-wide scan of the groups' lengths, and the bits ORed into the chunk's buffer.
// Returns the chunk's total bit count; `missing` reports a symbol without codeword; off[c]: where the thread's group
// in quarter c starts in the chunk's bits.
template <bool kFromSym, bool kWhole, bool kDither>
__device__ __forceinline__ uint32_t pack_item(const PackArgs& a, PackSmem& sm, const FeedArgs& fa, const FeedItem& it,
                                              uint32_t k, bool ok, uint32_t& enc_seg, uint32_t& n_sat, uint32_t& n_nf,
                                              bool& missing, uint32_t (&off)[4]) {
    const uint32_t tid = threadIdx.x;
    uint32_t len[4], any = 0;
    uint64_t w[4];
    pack_eight<kFromSym, kWhole, kDither>(a, sm, fa, it, k, 4u * tid, ok, n_sat, n_nf, len[0], len[1], w[0], w[1], any);
    pack_eight<kFromSym, kWhole, kDither>(a, sm, fa, it, k, 4u * tid + kHalf, ok, n_sat, n_nf, len[2], len[3], w[2], w[3], any);
    missing = (any & kEncMissing) != 0;
    // One scan for the four groups, two to a word (low and high half): no sum can pass kC / 4 * 16 bits.  In the
    // chunk all groups of a quarter come before those of the next.
    const uint32_t x[2] = {len[0] | (len[1] << 16), len[2] | (len[3] << 16)};
    uint32_t ex[2], tot[2];
    pack_scan2(x, sm.scan[k & 1u], ex, tot);
    const uint32_t t0 = tot[0] & 0xffffu, t01 = t0 + (tot[0] >> 16), t012 = t01 + (tot[1] & 0xffffu);
    off[0] = ex[0] & 0xffffu;
    off[1] = t0 + (ex[0] >> 16);
    off[2] = t01 + (ex[1] & 0xffffu);
    off[3] = t012 + (ex[1] >> 16);
    // Behind the scan's barrier every thread has finished the previous item's copy-out and this item's table
    // look-ups: clear the other bit buffer and fetch the next item's tables.
    uint4* clr = reinterpret_cast<uint4*>(sm.bits[(k + 1) & 1u]);
    clr[tid] = make_uint4(0, 0, 0, 0);
    clr[tid + kPackThreads] = make_uint4(0, 0, 0, 0);
    const FeedItem& nx = sm.feed.item[(k + 1) & 1u];
    if (nx.valid && nx.d.seg != enc_seg) {
        enc_seg = nx.d.seg;
        sm.enc[tid] = a.ws.enc_lut[enc_seg * 256 + tid];
        sm.enc[tid + kPackThreads] = a.ws.enc_lut[enc_seg * 256 + tid + kPackThreads];
    }
    if (!kFromSym) feed_fetch_fmt(sm.feed, a.ws, (uint32_t)(k + 1) & 1u);
    if (!missing) {
        const uint32_t bits_addr = smem_addr(sm.bits[k & 1u]);
#pragma unroll
        for (int c = 0; c < 4; ++c) put_bits(bits_addr, off[c] + len[c], w[c]);
    }
    return t012 + (tot[1] >> 16);
}

// One thread of the block's second warp only (the first warp's thread 0 feeds the ring meanwhile): output locations of
// the next item of the sequence, for ring slot `slot`.  It walks the item sequence with a cursor of its own, in step
// with the feeding thread's; beyond the last item the locations are never used.
__device__ __forceinline__ void pack_out_set(const PackArgs& a, PackSmem& sm, uint32_t slot, uint64_t sub_off, uint32_t n_chunks) {
    FeedCursor cur = sm.out_cur;
    PackOut o;
    const size_t ci = (size_t)cur.client * a.ws.n_chunks_max + cur.chunk;
    o.sub = reinterpret_cast<uint16_t*>(a.streams + (size_t)cur.client * a.stream_capacity + sub_off) + (size_t)cur.chunk * kSubs;
    o.slot = a.ws.slots + ci * kSlotWords;
    o.chunk_bits = a.ws.chunk_bits + ci;
    o.res = a.res + cur.client;
    sm.out[slot] = o;
    cur.advance(n_chunks);
    sm.out_cur = cur;
}

// kDither: the instance behind the dithered entry point (see convert_kernel).
template <bool kFromSym, bool kDither>
__global__ void __launch_bounds__(kPackThreads, 5) pack_kernel(PackArgs a) {
    wait_for_previous_kernel();
    extern __shared__ __align__(16) unsigned char smem_raw[];
    PackSmem& sm = *reinterpret_cast<PackSmem*>(smem_raw);
    Ctrl* ctrl = a.ws.ctrl;
    if (ctrl->abort) return;
    const uint32_t tid = threadIdx.x;
    const uint32_t n_chunks = ctrl->n_chunks;
    const FeedArgs fa{a.grad, a.mem, a.client_stride, a.n_clients};
    if ((uint64_t)blockIdx.x * a.group >= (uint64_t)n_chunks * a.n_clients) return;
    const uint64_t sub_off = ctrl->sub_off;

    ChunkDesc next{};
    if (tid == 0) {
        mbar_init(&sm.feed.bar[0], 1);
        mbar_init(&sm.feed.bar[1], 1);
        sm.feed.fail = 0u;
        sm.feed.cur.init(n_chunks, a.group);
        next = a.ws.chunk_desc[sm.feed.cur.chunk];
        feed_issue(sm.feed, fa, a.ws, n_chunks, 0, next, !kFromSym);
    }
    if (tid == 32) {
        sm.out_cur.init(n_chunks, a.group);
        pack_out_set(a, sm, 0, sub_off, n_chunks);
    }
    reinterpret_cast<uint4*>(sm.bits[0])[tid] = make_uint4(0, 0, 0, 0);
    reinterpret_cast<uint4*>(sm.bits[0])[tid + kPackThreads] = make_uint4(0, 0, 0, 0);
    __syncthreads();
    uint32_t enc_seg = sm.feed.item[0].valid ? sm.feed.item[0].d.seg : 0u;
    sm.enc[tid] = a.ws.enc_lut[enc_seg * 256 + tid];
    sm.enc[tid + kPackThreads] = a.ws.enc_lut[enc_seg * 256 + tid + kPackThreads];
    feed_fetch_fmt(sm.feed, a.ws, 0);
    __syncthreads();

    uint32_t n_sat = 0, n_nf = 0, cur_client = 0, parity = 0;
    bool hw_fail = false;
    for (uint32_t k = 0;; ++k) {
        // item k + 1 goes into the ring slot and descriptor that item k - 1 used; every thread is past the
        // last barrier of item k - 1 and read them before it
        if (tid == 0) feed_issue(sm.feed, fa, a.ws, n_chunks, (k + 1) & 1u, next, !kFromSym);
        if (tid == 32) pack_out_set(a, sm, (k + 1) & 1u, sub_off, n_chunks);
        const FeedItem it = sm.feed.item[k & 1u];
        if (!it.valid) break;
        if (!kFromSym && it.client != cur_client) {
            add_counts(&a.res[cur_client], n_sat, n_nf);
            n_sat = n_nf = 0;
            cur_client = it.client;
        }
        const bool ok = kFromSym || feed_wait(sm.feed, it, k, parity);
        if (!ok) hw_fail = true;
        bool missing;
        uint32_t off[4], total;
        const bool whole = kFromSym ? it.d.cnt == (uint32_t)kC : it.tma != 0;
        if (whole) total = pack_item<kFromSym, true, kDither>(a, sm, fa, it, k, ok, enc_seg, n_sat, n_nf, missing, off);
        else total = pack_item<kFromSym, false, kDither>(a, sm, fa, it, k, ok, enc_seg, n_sat, n_nf, missing, off);
        const PackOut out = sm.out[k & 1u];
        // a sub-chunk of kS symbols is the groups of one warp in one quarter of the chunk
        static_assert(kS == 4 * 32 && kSubs == 4 * kPackWarps, "a warp's groups in a quarter make up one sub-chunk");
        if ((tid & 31u) == 0) {
#pragma unroll
            for (int c = 0; c < 4; ++c) out.sub[c * kPackWarps + (tid >> 5)] = (uint16_t)off[c];
        }
        if (__syncthreads_or(missing)) {  // bit buffer complete
            if (tid == 0) {
                set_status(out.res, CO3_ERR_NO_CODEWORD);
                atomicMin(&out.res->first_bad_chunk, it.chunk);
                a.ws.client_fail[it.client] = 1u;
            }
        }
        if (!kFromSym && sm.feed.fail) {  // the same for every thread: written before the barrier above
            feed_drain(sm.feed, k, parity);
            break;
        }
        if (tid == 0) *out.chunk_bits = total;
        // the chunk's words, 16 bytes at a time; what the last of these copies carries beyond the chunk's end is
        // zero and stays inside the slot
        const uint4* bits4 = reinterpret_cast<const uint4*>(sm.bits[k & 1u]);
        if (tid * 128u < total) reinterpret_cast<uint4*>(out.slot)[tid] = bits4[tid];
        if ((tid + kPackThreads) * 128u < total) reinterpret_cast<uint4*>(out.slot)[tid + kPackThreads] = bits4[tid + kPackThreads];
    }
    if (!kFromSym) add_counts(&a.res[cur_client], n_sat, n_nf);
    if (__syncthreads_or(hw_fail)) {  // the block stopped early, chunks of any client may be missing: the call fails
        for (uint32_t u = tid; u < a.n_clients; u += kPackThreads) set_status(&a.res[u], CO3_ERR_CUDA);
        if (tid == 0) a.ws.ctrl->abort = 1u;  // the kernels that would assemble the containers return at once
    }
}

// ------------------------------------------------------------------------------------------------
// scan: one block of 1024 threads per client.  Prefix sums of the chunk sizes give every chunk its
// place in the payload; the same block writes the header and the segment table.
// ------------------------------------------------------------------------------------------------
struct ScanArgs {
    const co3_seg* segs;
    uint32_t n_seg;
    uint64_t n_elem;
    uint8_t* streams;
    size_t stream_capacity;
    co3_result* res;
    uint32_t two_level;    // 1: chunk offsets come from the range kernels below, scan_kernel only finishes
    uint32_t n_ranges_max;
    Ws ws;
};

constexpr int kScanThreads = 1024;
static_assert(kRangeChunks == 4 * kScanThreads, "one range is one tile of four chunks per thread");

// Exclusive prefix of 32-bit per-thread sums over the 1024 threads of a block (two quantities at once);
// *tot_w / *tot_b receive the block totals, which must fit 32 bits (they do for up to 2^17 chunks).  Contains two
// __syncthreads().  s_w / s_b: 32 words each.
__device__ __forceinline__ void block_scan_1024x2(uint32_t w, uint32_t b, uint32_t* s_w, uint32_t* s_b, uint64_t& ex_w,
                                                  uint64_t& ex_b, uint64_t& tot_w, uint64_t& tot_b) {
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    uint32_t iw = w, ib = b;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t yw = __shfl_up_sync(0xffffffffu, iw, d), yb = __shfl_up_sync(0xffffffffu, ib, d);
        if (lane >= (uint32_t)d) { iw += yw; ib += yb; }
    }
    __syncthreads();  // earlier readers of s_w / s_b are done
    if (lane == 31u) { s_w[warp] = iw; s_b[warp] = ib; }
    __syncthreads();
    // every warp scans the 32 warp totals, one per lane
    uint32_t xw = s_w[lane], xb = s_b[lane];
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t yw = __shfl_up_sync(0xffffffffu, xw, d), yb = __shfl_up_sync(0xffffffffu, xb, d);
        if (lane >= (uint32_t)d) { xw += yw; xb += yb; }
    }
    tot_w = __shfl_sync(0xffffffffu, xw, 31);
    tot_b = __shfl_sync(0xffffffffu, xb, 31);
    const uint32_t bw = __shfl_sync(0xffffffffu, xw, (warp + 31u) & 31u), bb = __shfl_sync(0xffffffffu, xb, (warp + 31u) & 31u);
    ex_w = (uint64_t)((warp ? bw : 0u) + iw - w);
    ex_b = (uint64_t)((warp ? bb : 0u) + ib - b);
}

// Two-level scan for long inputs, step 1: words and bits of each range of kRangeChunks chunks.
__global__ void __launch_bounds__(kScanThreads) range_totals_kernel(ScanArgs a) {
    wait_for_previous_kernel();
    __shared__ uint32_t s_w[32], s_b[32];
    const Ctrl* ctrl = a.ws.ctrl;
    if (ctrl->abort) return;
    const uint32_t y = blockIdx.x, u = blockIdx.y, tid = threadIdx.x;
    const uint32_t n = ctrl->n_chunks;
    if ((uint64_t)y * kRangeChunks >= n) return;
    const uint32_t* bits = a.ws.chunk_bits + (size_t)u * a.ws.n_chunks_max;
    const uint32_t c0 = y * kRangeChunks + 4 * tid;
    uint32_t w = 0, b = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint32_t x = (c0 + i < n) ? bits[c0 + i] : 0u;
        b += x;
        w += (x + 31u) >> 5;
    }
    uint64_t ew, eb, tw, tb;
    block_scan_1024x2(w, b, s_w, s_b, ew, eb, tw, tb);
    if (tid == 0) {
        uint64_t* r = a.ws.range_tot + ((size_t)u * a.n_ranges_max + y) * 2;
        r[0] = tw;
        r[1] = tb;
    }
}

// Step 2: one block per client turns the range totals into exclusive prefixes and the client's totals.
__global__ void __launch_bounds__(kScanThreads) range_scan_kernel(ScanArgs a) {
    wait_for_previous_kernel();
    const Ctrl* ctrl = a.ws.ctrl;
    if (ctrl->abort) return;
    const uint32_t u = blockIdx.x, tid = threadIdx.x;
    const uint32_t n_ranges = (ctrl->n_chunks + kRangeChunks - 1) / kRangeChunks;
    uint64_t* r = a.ws.range_tot + (size_t)u * a.n_ranges_max * 2;
    // few ranges (one per 8 M elements): one thread walks them
    if (tid == 0) {
        uint64_t w = 0, b = 0;
        for (uint32_t y = 0; y < n_ranges; ++y) {
            const uint64_t tw = r[2 * y], tb = r[2 * y + 1];
            r[2 * y] = w;
            r[2 * y + 1] = b;
            w += tw;
            b += tb;
        }
        a.ws.totals[2 * u] = w;
        a.ws.totals[2 * u + 1] = b;
    }
}

// Step 3: every range scans its own chunks from its exclusive prefix and writes the chunk offsets.
__global__ void __launch_bounds__(kScanThreads) range_apply_kernel(ScanArgs a) {
    wait_for_previous_kernel();
    __shared__ uint32_t s_w[32], s_b[32];
    const Ctrl* ctrl = a.ws.ctrl;
    if (ctrl->abort) return;
    const uint32_t y = blockIdx.x, u = blockIdx.y, tid = threadIdx.x;
    const uint32_t n = ctrl->n_chunks;
    if ((uint64_t)y * kRangeChunks >= n) return;
    const uint32_t* bits = a.ws.chunk_bits + (size_t)u * a.ws.n_chunks_max;
    uint64_t* bit_prefix = a.ws.bit_prefix + (size_t)u * (a.ws.n_chunks_max + 1ull);
    uint8_t* stream = a.streams + (size_t)u * a.stream_capacity;
    uint64_t* word_off = reinterpret_cast<uint64_t*>(stream + ctrl->chunk_off);
    const uint64_t* r = a.ws.range_tot + ((size_t)u * a.n_ranges_max + y) * 2;
    const uint32_t c0 = y * kRangeChunks + 4 * tid;
    uint32_t bv[4], wv[4], w = 0, b = 0;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        bv[i] = (c0 + i < n) ? bits[c0 + i] : 0u;
        wv[i] = (bv[i] + 31u) >> 5;
        b += bv[i];
        w += wv[i];
    }
    uint64_t ew, eb, tw, tb;
    block_scan_1024x2(w, b, s_w, s_b, ew, eb, tw, tb);
    uint64_t pw = r[0] + ew, pb = r[1] + eb;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        if (c0 + i < n) {
            word_off[c0 + i] = pw;
            bit_prefix[c0 + i] = pb;
        }
        pw += wv[i];
        pb += bv[i];
    }
}

__global__ void __launch_bounds__(kScanThreads) scan_kernel(ScanArgs a) {
    wait_for_previous_kernel();
    __shared__ uint32_t s_w[32], s_b[32];
    const Ctrl* ctrl = a.ws.ctrl;
    if (ctrl->abort) return;
    const uint32_t u = blockIdx.x, tid = threadIdx.x;
    const uint32_t n = ctrl->n_chunks;
    const uint32_t* bits = a.ws.chunk_bits + (size_t)u * a.ws.n_chunks_max;
    uint64_t* bit_prefix = a.ws.bit_prefix + (size_t)u * (a.ws.n_chunks_max + 1ull);
    uint8_t* stream = a.streams + (size_t)u * a.stream_capacity;
    uint64_t* word_off = reinterpret_cast<uint64_t*>(stream + ctrl->chunk_off);

    // tiles of 8 * 1024 chunks: eight consecutive chunks per thread, warp scan, one exchange through shared memory
    uint64_t carry_w = 0, carry_b = 0;  // totals of the tiles already done (same in every thread)
    if (a.two_level) {  // the range kernels have written the chunk offsets already
        carry_w = a.ws.totals[2 * u];
        carry_b = a.ws.totals[2 * u + 1];
    } else {
        constexpr uint32_t kPer = 8;  // consecutive chunks per thread
        for (uint32_t base = 0; base < n; base += kPer * kScanThreads) {
            const uint32_t c0 = base + kPer * tid;
            uint32_t b[kPer], w[kPer], tw8 = 0, tb8 = 0;
#pragma unroll
            for (uint32_t i = 0; i < kPer; ++i) {
                b[i] = (c0 + i < n) ? bits[c0 + i] : 0u;
                w[i] = (b[i] + 31u) >> 5;
                tw8 += w[i];
                tb8 += b[i];
            }
            uint64_t ew, eb, tile_w, tile_b;
            block_scan_1024x2(tw8, tb8, s_w, s_b, ew, eb, tile_w, tile_b);
            uint64_t pw = carry_w + ew, pb = carry_b + eb;  // exclusive prefix of chunk c0
#pragma unroll
            for (uint32_t i = 0; i < kPer; ++i) {
                if (c0 + i < n) {
                    word_off[c0 + i] = pw;
                    bit_prefix[c0 + i] = pb;
                }
                pw += w[i];
                pb += b[i];
            }
            carry_w += tile_w;
            carry_b += tile_b;
        }
    }
    const uint64_t tw = carry_w, tb = carry_b;
    const uint64_t total_bytes = align16(ctrl->payload_off + 4ull * tw);
    const bool fits = total_bytes <= a.stream_capacity;
    const bool failed = a.ws.client_fail[u] != 0;
    if (tid == 0) {
        word_off[n] = tw;
        bit_prefix[n] = tb;
    }
    __syncthreads();
    for (uint32_t k = tid; k < a.n_seg; k += kScanThreads) {
        uint64_t* e = reinterpret_cast<uint64_t*>(stream + kHeaderBytes + 24ull * k);
        const uint32_t c0 = a.ws.first_chunk[k], c1 = a.ws.first_chunk[k + 1];
        e[0] = a.segs[k].n_elem;
        e[1] = c0;
        e[2] = bit_prefix[c1] - bit_prefix[c0];
    }
    if (tid == 0) {
        uint32_t* h32 = reinterpret_cast<uint32_t*>(stream);
        uint64_t* h64 = reinterpret_cast<uint64_t*>(stream);
        h32[0] = kMagic; h32[1] = 1u; h32[2] = a.n_seg; h32[3] = kC; h32[4] = kS; h32[5] = 0u;
        h64[3] = a.n_elem; h64[4] = n; h64[5] = tw; h64[6] = tb; h64[7] = total_bytes;
        // table padding up to the next section
        for (uint64_t o = kHeaderBytes + 24ull * a.n_seg; o < ctrl->chunk_off; o += 8) *reinterpret_cast<uint64_t*>(stream + o) = 0;
        for (uint64_t o = ctrl->chunk_off + 8ull * (n + 1ull); o < ctrl->sub_off; o += 8) *reinterpret_cast<uint64_t*>(stream + o) = 0;
        for (uint64_t o = ctrl->sub_off + 2ull * n * kSubs; o < ctrl->payload_off; o += 8) *reinterpret_cast<uint64_t*>(stream + o) = 0;
        co3_result* r = &a.res[u];
        r->payload_bits = tb;
        r->container_bytes = total_bytes;
        if (!fits) {
            set_status(r, CO3_ERR_CAPACITY);
            a.ws.client_fail[u] = 1u;
        } else if (!failed) {
            for (uint64_t o = ctrl->payload_off + 4ull * tw; o < total_bytes; o += 4) *reinterpret_cast<uint32_t*>(stream + o) = 0;
        }
    }
}

// compact: moves the chunks' words from their slots to their final positions; one warp per chunk, eight
// chunks of one client per block, loads batched eight deep.
__global__ void __launch_bounds__(kThreads) compact_kernel(ScanArgs a) {
    wait_for_previous_kernel();
    const Ctrl* ctrl = a.ws.ctrl;
    if (ctrl->abort) return;
    const uint32_t u = blockIdx.y, lane = threadIdx.x & 31u;
    const uint32_t chunk = blockIdx.x * (kThreads / 32) + (threadIdx.x >> 5);
    if (chunk >= ctrl->n_chunks || a.ws.client_fail[u]) return;
    uint8_t* stream = a.streams + (size_t)u * a.stream_capacity;
    const uint64_t w0 = reinterpret_cast<const uint64_t*>(stream + ctrl->chunk_off)[chunk];
    const size_t ci = (size_t)u * a.ws.n_chunks_max + chunk;
    const uint32_t words = (a.ws.chunk_bits[ci] + 31u) >> 5;
    const uint32_t* __restrict__ slot = a.ws.slots + ci * kSlotWords;
    uint32_t* __restrict__ dst = reinterpret_cast<uint32_t*>(stream + ctrl->payload_off) + w0;
    uint32_t i = lane;
    for (; i + 7 * 32 < words; i += 8 * 32) {
        uint32_t v[8];
#pragma unroll
        for (int r = 0; r < 8; ++r) v[r] = __ldg(slot + i + r * 32);
#pragma unroll
        for (int r = 0; r < 8; ++r) dst[i + r * 32] = v[r];
    }
    for (; i < words; i += 32) dst[i] = __ldg(slot + i);
}

// ------------------------------------------------------------------------------------------------
// decode
// ------------------------------------------------------------------------------------------------
struct DecArgs {
    const uint8_t* const* streams;  // device array of n_clients pointers, or null:
    const uint8_t* single;          // the one stream when `streams` is null
    size_t stream_bytes;
    uint32_t n_clients;
    const co3_seg* segs;
    uint32_t n_seg;
    uint64_t n_elem;
    float* out;        // average (or the single client's values); nullable when sym_out is given
    uint8_t* sym_out;  // nullable; only with n_clients == 1
    float* params;     // nullable: model parameters to update with the average (Algorithm 1, last step)
    float lr;          // learning rate of that update
    co3_result* res;
    uint32_t B;        // clients decoded side by side in one block
    uint32_t G;        // chunks per block (tile)
    Ws ws;
};

__device__ __forceinline__ const uint8_t* stream_of(const DecArgs& a, uint32_t u) {
    return a.streams ? a.streams[u] : a.single;
}

constexpr int kMaxPairs = 16;          // (chunk, client) pairs decoded side by side in one block
constexpr int kMultiPairs = 20;        // the same when the clients come in several batches (one chunk per block)
constexpr int kMultiThreads = 16 * kMultiPairs;
constexpr int kPaySlotWords = 456;     // staging per pair: 7 bits/symbol plus alignment; larger chunks are read in place
constexpr int kPaySlack = 72;          // words a reader may run past its chunk before the end check

// Fixed part of the shared memory of one decode block; behind it follow the symbol buffer
// sym[n_pairs][128] of one decode phase and the payload staging area pay[n_pairs * kPaySlotWords + kPaySlack].
struct DecSmem {
    uint16_t lut[kDecLut];
    float val[256];
    uint64_t bar;                          // completion barrier of the bulk copies of one batch
    uint32_t tile_elems;                   // elements of the tile: full chunks and the last one's count
    uint32_t pad;
    uint64_t chunk_elem0[kMultiPairs];       // first element of each chunk of the tile
    const uint32_t* pair_src[kMultiPairs];   // the pair's first payload word in global memory
    uint32_t pair_off[kMultiPairs];          // staged pairs: index of that word in pay[]
    uint32_t pair_words[kMultiPairs];
    uint32_t pair_staged[kMultiPairs];
    uint32_t pair_cnt[kMultiPairs];
    uint16_t sub[kMultiPairs][kSubs];        // sub-chunk bit offsets of each pair
};
static_assert(sizeof(DecSmem) % 16 == 0 && offsetof(DecSmem, sub) % 16 == 0, "dynamic arrays behind DecSmem must stay 16-byte aligned");

// A tile is decoded in kPhases rounds of kPhaseSyms symbols per sub-chunk: the symbol buffer between the
// decoding threads and the summing threads then holds a quarter of a chunk per pair.
constexpr int kPhases = 4;
constexpr int kPhaseSyms = kS / kPhases;            // 32 symbols of every sub-chunk per phase
constexpr int kPhaseWords = kPhaseSyms / 4;         // 8 symbol words per sub-chunk and phase
constexpr int kPairPhaseWords = kSubs * kPhaseWords;  // 128 symbol words per pair and phase

// Position of word j (0..7) of sub-chunk s in the phase's symbol buffer of pair p: rotated so that the 32
// threads of a warp (2 pairs x 16 sub-chunks, all at the same j) hit 32 different banks, and so do 32
// consecutive words read by the summing threads.
__device__ __forceinline__ uint32_t sym_slot(uint32_t p, uint32_t s, uint32_t j) {
    return s * kPhaseWords + ((j + (s >> 2) + 4u * (p & 1u)) & (kPhaseWords - 1));
}

// Second-level look-up for a codeword longer than the first table's index; rare, kept out of line so that
// the common path carries none of its instructions.  `win` holds the stream bits from the codeword's start.
__device__ __noinline__ uint32_t decode_long(const uint16_t* __restrict__ sub_tab, uint32_t ent, uint32_t win) {
    return __ldg(sub_tab + ((ent & 0xffu) << kSubBits) + ((win >> (32 - CO3_MAX_CODE_LEN)) & ((1u << kSubBits) - 1u)));
}

// A thread's view of its chunk's bits: two consecutive payload words held in registers and replaced one at a
// time as the position crosses a word boundary, so that a shared-memory load is issued only for the lanes that
// need a new word (about one per 32 bits consumed instead of two per window).
// kChecked: words beyond the chunk read as 0 (needed when the words are read in place from global memory);
// otherwise the words sit in shared memory with kPaySlack readable words behind them.
template <bool kChecked>
struct BitWindow {
    uint32_t hi, lo, wi;  // words wi and wi + 1 of the chunk
    __device__ __forceinline__ uint32_t word(const uint32_t* words, uint32_t nwords, uint32_t i) const {
        if (kChecked) return i < nwords ? __ldg(words + i) : 0u;
        return words[i];
    }
    __device__ __forceinline__ void start(const uint32_t* words, uint32_t nwords, uint32_t pos) {
        wi = pos >> 5;
        hi = word(words, nwords, wi);
        lo = word(words, nwords, wi + 1);
    }
    // The 32 stream bits that start at bit `pos`; pos lies in word wi or wi + 1 (it moved by at most 32 bits
    // since the last call).
    __device__ __forceinline__ uint32_t at(const uint32_t* words, uint32_t nwords, uint32_t pos) {
        if ((pos >> 5) != wi) {
            hi = lo;
            ++wi;
            lo = word(words, nwords, wi + 1);
        }
        return __funnelshift_l(lo, hi, pos);  // shift count taken modulo 32
    }
};

// Decodes two symbols from the position `pos` on (a codeword has at most 16 bits, so one 32-bit window holds
// both) and advances it.  Returns the two table entries: symbol in the low byte, 0xff = no codeword matched.
// Both look-ups are done assuming short codewords and tested together; if either hit a second-level marker
// the pair is redone step by step.
template <bool kChecked, bool kSecond>
__device__ __forceinline__ void decode_two(BitWindow<kChecked>& bw, const uint32_t* words, uint32_t nwords, uint32_t& pos,
                                           const uint16_t* __restrict__ s_lut, const uint16_t* __restrict__ sub_tab,
                                           uint32_t& e0, uint32_t& e1) {
    const uint32_t win = bw.at(words, nwords, pos);
    e0 = s_lut[win >> (32 - kDecBits)];
    if (!kSecond) {
        if (e0 >= kDecLong) e0 = decode_long(sub_tab, e0, win);
        e1 = 0;
        pos += e0 >> 8;
        return;
    }
    uint32_t l0 = e0 >> 8;
    uint32_t win1 = __funnelshift_l(0u, win, l0);  // win << (l0 mod 32): a marker's "length" is meaningless
    e1 = s_lut[win1 >> (32 - kDecBits)];
    uint32_t either = e0 | e1;
    asm("" : "+r"(either));  // one test, one branch for both entries
    if (either >= kDecLong) {
        if (e0 >= kDecLong) e0 = decode_long(sub_tab, e0, win);
        l0 = e0 >> 8;
        win1 = win << l0;
        e1 = s_lut[win1 >> (32 - kDecBits)];
        if (e1 >= kDecLong) e1 = decode_long(sub_tab, e1, win1);
    }
    pos += l0 + (e1 >> 8);
}

// One phase of one sub-chunk: decodes symbols [4 * j0, 4 * j0 + 32) of the sub-chunk (those below `my`) from bit
// position `pos` on into the pair's phase buffer, four per word, and advances `pos`.
template <bool kChecked, bool kWhole>
__device__ __forceinline__ void decode_part(const uint32_t* words, uint32_t nwords, uint32_t& pos, uint32_t j0, uint32_t my,
                                            const uint16_t* __restrict__ s_lut, const uint16_t* __restrict__ sub_tab,
                                            uint32_t* pair_buf, uint32_t p, uint32_t s, uint32_t& marks) {
    BitWindow<kChecked> bw;
    bw.start(words, nwords, pos);
#pragma unroll 2
    for (uint32_t jj = 0; jj < (uint32_t)kPhaseWords; ++jj) {
        const uint32_t j = j0 + jj;
        uint32_t w = 0;
        if (kWhole || j * 4 < my) {
            uint32_t e0, e1, e2 = 0, e3 = 0;
            if (kWhole || j * 4 + 1 < my) decode_two<kChecked, true>(bw, words, nwords, pos, s_lut, sub_tab, e0, e1);
            else decode_two<kChecked, false>(bw, words, nwords, pos, s_lut, sub_tab, e0, e1);
            if (kWhole || j * 4 + 3 < my) decode_two<kChecked, true>(bw, words, nwords, pos, s_lut, sub_tab, e2, e3);
            else if (j * 4 + 2 < my) decode_two<kChecked, false>(bw, words, nwords, pos, s_lut, sub_tab, e2, e3);
            w = __byte_perm(__byte_perm(e0, e1, 0x0040), __byte_perm(e2, e3, 0x0040), 0x5410);
            marks |= (~w - 0x01010101u) & w;  // bit 7 of a byte survives iff that byte of ~w is zero (symbol 0xff)
        }
        pair_buf[sym_slot(p, s, jj)] = w;
    }
}

// Adds, in client order, the values of the four symbols of word (s, j) of chunk cl of the tile's current phase
// for the nb clients of the batch.  Returns the last client's symbol word.
__device__ __forceinline__ uint32_t sum_word(const float* __restrict__ val, const uint32_t* __restrict__ sym, uint32_t cl,
                                             uint32_t s, uint32_t j, uint32_t B, uint32_t nb, float (&acc)[4]) {
    uint32_t symw = 0;
    uint32_t p = cl * B;
    const uint32_t* row = sym + p * kPairPhaseWords + s * kPhaseWords;
    const uint32_t rot = j + (s >> 2);
#pragma unroll 2
    for (uint32_t ul = 0; ul < nb; ++ul, ++p, row += kPairPhaseWords) {
        symw = row[(rot + 4u * (p & 1u)) & (kPhaseWords - 1)];
#pragma unroll
        for (int q = 0; q < 4; ++q) acc[q] = __fadd_rn(acc[q], val[(symw >> (8 * q)) & 0xffu]);
    }
    return symw;
}

// The same for one half of the word (symbols 2 * half and 2 * half + 1): the batched decoder of many clients splits
// every word between two threads so that the whole block takes part in the sum.
__device__ __forceinline__ void sum_half(const float* __restrict__ val, const uint32_t* __restrict__ sym, uint32_t s,
                                         uint32_t j, uint32_t half, uint32_t nb, float (&acc)[2]) {
    const uint32_t* row = sym + s * kPhaseWords;
    const uint32_t rot = j + (s >> 2), sh = 16u * half;
#pragma unroll 2
    for (uint32_t p = 0; p < nb; ++p, row += kPairPhaseWords) {
        const uint32_t symw = row[(rot + 4u * (p & 1u)) & (kPhaseWords - 1)] >> sh;
        acc[0] = __fadd_rn(acc[0], val[symw & 0xffu]);
        acc[1] = __fadd_rn(acc[1], val[(symw >> 8) & 0xffu]);
    }
}

// Where a tile's results go.  The chunks of a tile follow one another in one segment and all but the last
// are full, so element e of the tile (chunk index * kC + place in the chunk) is element e behind the tile's
// first one in the output as well.
struct TileOut {
    float* out;         // the tile's first element in the output vector (null: no values wanted)
    uint8_t* sym;       // the same in the symbol output (nullable)
    float* params;      // the same in the model parameters to update (nullable)
    float lr;
    uint32_t n_elem;    // elements of the tile
    bool out16, sym4, params16;  // out / params are 16-byte aligned, sym is 4-byte aligned
    float u, inv;       // the averages are acc / u, or acc * inv when u is a power of two (the product with
    bool pow2;          // the exact reciprocal rounds the same real number as the division)
};

// Averages the sums and stores the (up to four) elements that start at element e of the tile; e is a multiple
// of four below to.n_elem.  kPlain: acc holds values, not sums to be averaged.
template <bool kPlain>
__device__ __forceinline__ void write_word(const TileOut& to, uint32_t e, const float (&acc)[4], uint32_t symw) {
    const uint32_t nv = min(4u, to.n_elem - e);
    float r[4];
    if (kPlain) {  // one client: the average is the value itself
#pragma unroll
        for (int q = 0; q < 4; ++q) r[q] = acc[q];
    } else if (to.pow2) {
#pragma unroll
        for (int q = 0; q < 4; ++q) r[q] = __fmul_rn(acc[q], to.inv);
    } else {
#pragma unroll
        for (int q = 0; q < 4; ++q) r[q] = __fdiv_rn(acc[q], to.u);
    }
    if (to.out) {
        float* o = to.out + e;
        if (nv == 4 && to.out16) {
            *reinterpret_cast<float4*>(o) = make_float4(r[0], r[1], r[2], r[3]);
        } else {
            for (uint32_t q = 0; q < nv; ++q) o[q] = r[q];
        }
    }
    if (to.params) {  // w <- w - lr * avg: one multiplication and one subtraction, each rounded on its own
        float* w = to.params + e;
        if (nv == 4 && to.params16) {
            float4 x = *reinterpret_cast<const float4*>(w);
            x.x = __fsub_rn(x.x, __fmul_rn(to.lr, r[0]));
            x.y = __fsub_rn(x.y, __fmul_rn(to.lr, r[1]));
            x.z = __fsub_rn(x.z, __fmul_rn(to.lr, r[2]));
            x.w = __fsub_rn(x.w, __fmul_rn(to.lr, r[3]));
            *reinterpret_cast<float4*>(w) = x;
        } else {
            for (uint32_t q = 0; q < nv; ++q) w[q] = __fsub_rn(w[q], __fmul_rn(to.lr, r[q]));
        }
    }
    if (to.sym) {
        uint8_t* o = to.sym + e;
        if (nv == 4 && to.sym4) {
            *reinterpret_cast<uint32_t*>(o) = symw;
        } else {
            for (uint32_t q = 0; q < nv; ++q) o[q] = (uint8_t)(symw >> (8 * q));
        }
    }
}

// write_word for two elements (e even, below to.n_elem): averages and stores them, and applies the update.
__device__ __forceinline__ void write_half(const TileOut& to, uint32_t e, const float (&acc)[2]) {
    const uint32_t nv = min(2u, to.n_elem - e);
    float r[2];
    if (to.pow2) {
        r[0] = __fmul_rn(acc[0], to.inv);
        r[1] = __fmul_rn(acc[1], to.inv);
    } else {
        r[0] = __fdiv_rn(acc[0], to.u);
        r[1] = __fdiv_rn(acc[1], to.u);
    }
    if (to.out) {
        float* o = to.out + e;
        if (nv == 2 && to.out16) *reinterpret_cast<float2*>(o) = make_float2(r[0], r[1]);
        else for (uint32_t q = 0; q < nv; ++q) o[q] = r[q];
    }
    if (to.params) {  // w <- w - lr * avg: one multiplication and one subtraction, each rounded on its own
        float* w = to.params + e;
        if (nv == 2 && to.params16) {
            float2 x = *reinterpret_cast<const float2*>(w);
            x.x = __fsub_rn(x.x, __fmul_rn(to.lr, r[0]));
            x.y = __fsub_rn(x.y, __fmul_rn(to.lr, r[1]));
            *reinterpret_cast<float2*>(w) = x;
        } else {
            for (uint32_t q = 0; q < nv; ++q) w[q] = __fsub_rn(w[q], __fmul_rn(to.lr, r[q]));
        }
    }
}

// One block decodes a tile of G chunks for B clients at a time.  Warp 0 looks up where each (chunk, client)
// pair's payload lies and starts one bulk copy per pair into shared memory (plus the segment's tables);
// then 16 threads per pair (one per sub-chunk) decode into a symbol buffer, and finally every thread sums
// its share of the tile over the clients in client order.  kMulti: more clients than fit side by side: they
// come in equal batches of 16 to 20 (G = 1), the partial sums stay in registers between batches, and every symbol
// word is summed by two threads (two symbols each).  kSingle: one client, nothing to sum.
template <bool kMulti, bool kSingle>
__global__ void __launch_bounds__(kMulti ? kMultiThreads : kThreads, kMulti ? 3 : 4) decode_kernel(DecArgs a) {
    wait_for_previous_kernel();
    extern __shared__ __align__(16) unsigned char smem_raw[];
    DecSmem& sm = *reinterpret_cast<DecSmem*>(smem_raw);
    const uint32_t B = kSingle ? 1u : a.B, G = kMulti ? 1u : a.G;
    const uint32_t n_pairs = B * G, n_thr = 16u * n_pairs;
    uint32_t* const sm_sym = reinterpret_cast<uint32_t*>(smem_raw + sizeof(DecSmem));
    uint32_t* const sm_pay = sm_sym + n_pairs * kPairPhaseWords;
    const uint32_t pay_words = n_pairs * kPaySlotWords;

    const Ctrl* ctrl = a.ws.ctrl;
    if (ctrl->abort) return;
    const uint32_t tile = blockIdx.x, tid = threadIdx.x;
    if (tile >= ctrl->n_tiles) return;
    const TileDesc td = a.ws.tile_desc[tile];
    const uint64_t cap_words = (a.stream_bytes - ctrl->payload_off) / 4;
    const uint64_t readable16 = a.stream_bytes & ~(size_t)15u;  // bulk copies move whole 16-byte units
    const uint16_t* sub_tab = a.ws.dec_sub + (size_t)td.seg * kSubLut;

    if (tid == 0) mbar_init(&sm.bar, 1);
    float carry[kPhases][2];  // running sums across client batches (kMulti only)
    TileOut to;
    to.u = (float)a.n_clients;
    to.pow2 = (a.n_clients & (a.n_clients - 1u)) == 0;
    to.inv = __fdiv_rn(1.0f, to.u);
    bool err = false, hw_fail = false;
    uint32_t phase = 0;

    for (uint32_t u0 = 0; u0 < a.n_clients; u0 += B, phase ^= 1u) {
        const uint32_t nb = min(B, a.n_clients - u0);
        __syncthreads();  // barrier initialised; previous batch fully consumed
        // ---- pair descriptors (pair = one chunk of one client), staging plan, bulk copies
        if (tid < 32) {
            uint32_t nw = 0, cnt = 0, lead = 0, span = 0;  // span: words of the 16-byte aligned copy
            const uint32_t* src = nullptr;
            bool can_stage = false;
            const uint16_t* sub_src = nullptr;
            if (tid < n_pairs) {
                const uint32_t cl = tid / B, ul = tid % B;
                if (cl < td.n_chunks && ul < nb) {
                    const uint32_t chunk = td.chunk0 + cl;
                    const uint8_t* stream = stream_of(a, u0 + ul);
                    const uint64_t* word_off = reinterpret_cast<const uint64_t*>(stream + ctrl->chunk_off);
                    const uint64_t w0 = word_off[chunk], w1 = word_off[chunk + 1];
                    const ChunkDesc cd = a.ws.chunk_desc[chunk];
                    cnt = cd.cnt;
                    if (ul == 0) sm.chunk_elem0[cl] = cd.elem0;
                    if (ul == 0 && cl + 1 == td.n_chunks) sm.tile_elems = cl * kC + cd.cnt;
                    sub_src = reinterpret_cast<const uint16_t*>(stream + ctrl->sub_off) + (uint64_t)chunk * kSubs;
                    if (w0 > w1 || w1 > cap_words || w1 - w0 > (uint64_t)kSlotWords) {
                        err = true;
                        cnt = 0;
                    } else {
                        nw = (uint32_t)(w1 - w0);
                        const uint64_t byte0 = ctrl->payload_off + 4ull * w0;
                        src = reinterpret_cast<const uint32_t*>(stream + byte0);
                        lead = (uint32_t)(byte0 & 15u) / 4u;
                        span = (lead + nw + 3u) & ~3u;
                        can_stage = nw != 0 && (byte0 & ~15ull) + 4ull * span <= readable16;
                    }
                }
            }
            uint32_t inc = can_stage ? span : 0u;  // inclusive prefix of the staged spans over the pairs
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const uint32_t y = __shfl_up_sync(0xffffffffu, inc, d);
                if (tid >= (uint32_t)d) inc += y;
            }
            const bool staged = can_stage && inc <= pay_words;
            uint32_t bytes = (staged ? 4u * span : 0u) + (sub_src ? 2u * kSubs : 0u);
            if (tid == 0 && u0 == 0) bytes += 2u * kDecLut + 4u * 256u;  // the segment's tables, once
            const uint32_t total = __reduce_add_sync(0xffffffffu, bytes);
            if (tid == 0) {
                fence_async_smem();
                mbar_arrive_expect_tx(&sm.bar, total);
            }
            __syncwarp();
            if (tid == 0 && u0 == 0) {
                bulk_copy_g2s(sm.lut, a.ws.dec_lut + (size_t)td.seg * kDecLut, 2u * kDecLut, &sm.bar);
                bulk_copy_g2s(sm.val, a.ws.val_lut + (size_t)td.seg * 256, 4u * 256u, &sm.bar);
            }
            if (staged) bulk_copy_g2s(sm_pay + (inc - span), src - lead, 4u * span, &sm.bar);
            if (sub_src) bulk_copy_g2s(sm.sub[tid], sub_src, 2u * kSubs, &sm.bar);
            if (tid < n_pairs) {
                sm.pair_src[tid] = src;
                sm.pair_off[tid] = inc - span + lead;
                sm.pair_words[tid] = nw;
                sm.pair_staged[tid] = staged ? 1u : 0u;
                sm.pair_cnt[tid] = cnt;
            }
        }
        __syncthreads();
        if (!__syncthreads_and(mbar_wait(&sm.bar, phase))) {  // never expected: the copies are in bounds and aligned
            hw_fail = true;
            mbar_wait(&sm.bar, phase);
            break;
        }
        // ---- thread = (pair, sub-chunk): where its bits start and how many symbols it has
        const uint32_t p = tid >> 4, sc = tid & 15u;
        const uint32_t cnt = sm.pair_cnt[p];
        const uint32_t nw = sm.pair_words[p];
        uint32_t my = cnt > sc * kS ? min((uint32_t)kS, cnt - sc * kS) : 0u;
        const bool staged = sm.pair_staged[p] != 0;
        const uint32_t* const swords = sm_pay + sm.pair_off[p];  // staged copy in shared memory
        const uint32_t* const gwords = sm.pair_src[p];           // the words in place, in global memory
        uint32_t* pair_buf = sm_sym + p * kPairPhaseWords;
        uint32_t pos = my ? sm.sub[p][sc] : 0u, marks = 0;
        const bool last = cnt <= (sc + 1) * kS;
        const uint32_t expect = (my && !last) ? sm.sub[p][sc + 1] : 0u;
        if (my && pos > nw * 32u) {
            err = true;
            my = 0;
        }
        const bool had_symbols = my != 0;
        const bool first_batch = (u0 == 0), last_batch = (u0 + B >= a.n_clients);
        const uint32_t tile_words = min(G, td.n_chunks) * kPairPhaseWords;
        to.n_elem = sm.tile_elems;
        to.out = a.out ? a.out + sm.chunk_elem0[0] : nullptr;
        to.sym = a.sym_out ? a.sym_out + sm.chunk_elem0[0] : nullptr;
        to.params = a.params ? a.params + sm.chunk_elem0[0] : nullptr;
        to.lr = a.lr;
        to.params16 = (reinterpret_cast<uintptr_t>(to.params) & 15u) == 0;
        to.out16 = (reinterpret_cast<uintptr_t>(to.out) & 15u) == 0;
        to.sym4 = (reinterpret_cast<uintptr_t>(to.sym) & 3u) == 0;
#pragma unroll(kMulti ? kPhases : 1)
        for (int ph = 0; ph < kPhases; ++ph) {
            // ---- decode this phase's 32 symbols of the sub-chunk
            const uint32_t j0 = ph * kPhaseWords;
            if (my > j0 * 4) {
                if (!staged) decode_part<true, false>(gwords, nw, pos, j0, my, sm.lut, sub_tab, pair_buf, p, sc, marks);
                else if (my == (uint32_t)kS) decode_part<false, true>(swords, nw, pos, j0, my, sm.lut, sub_tab, pair_buf, p, sc, marks);
                else decode_part<false, false>(swords, nw, pos, j0, my, sm.lut, sub_tab, pair_buf, p, sc, marks);
            } else {
                for (uint32_t jj = 0; jj < (uint32_t)kPhaseWords; ++jj) pair_buf[sym_slot(p, sc, jj)] = 0;
            }
            __syncthreads();
            // ---- ordered sum over the clients of this batch; a thread owns whole symbol words: word w of the
            //      tile's phase is word (s, j) of chunk cl and starts at element e of the tile
            static_assert(kPairPhaseWords == 128 && kPhaseWords == 8 && kC == 2048 && kS == 128, "shifts below");
            if (kMulti) {
                if (tid < 2u * kPairPhaseWords) {  // B >= 16: the block has at least that many threads
                    const uint32_t half = tid >> 7, s = (tid >> 3) & 15u, j = tid & 7u;
                    const uint32_t e = (s << 7) + ph * kPhaseSyms + (j << 2) + 2u * half;
                    float acc[2];
                    acc[0] = first_batch ? 0.0f : carry[ph][0];
                    acc[1] = first_batch ? 0.0f : carry[ph][1];
                    sum_half(sm.val, sm_sym, s, j, half, nb, acc);
                    if (!last_batch) {
                        carry[ph][0] = acc[0];
                        carry[ph][1] = acc[1];
                    } else if (e < to.n_elem) {
                        write_half(to, e, acc);
                    }
                }
            } else {
                for (uint32_t w = tid; w < tile_words; w += n_thr) {
                    const uint32_t cl = w >> 7, s = (w >> 3) & 15u, j = w & 7u;
                    const uint32_t e = (cl << 11) + (s << 7) + ph * kPhaseSyms + (j << 2);
                    if (e >= to.n_elem) continue;
                    if (kSingle) {
                        const uint32_t symw = sm_sym[cl * kPairPhaseWords + sym_slot(cl, s, j)];
                        float v[4];
#pragma unroll
                        for (int q = 0; q < 4; ++q) v[q] = sm.val[(symw >> (8 * q)) & 0xffu];
                        write_word<true>(to, e, v, symw);
                    } else {
                        float acc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
                        const uint32_t symw = sum_word(sm.val, sm_sym, cl, s, j, B, nb, acc);
                        write_word<false>(to, e, acc, symw);
                    }
                }
            }
            __syncthreads();  // the phase buffer is free again
        }
        if (marks & 0x80808080u) err = true;
        if (had_symbols) {  // the sub-chunk must end where the next one starts, the last one inside the chunk's last word
            if (!last) {
                if (pos != expect) err = true;
            } else if (((pos + 31u) >> 5) != nw) {
                err = true;
            }
        }
    }
    const bool any_hw = __syncthreads_or(hw_fail);
    const bool any_err = __syncthreads_or(err);
    if (tid == 0) {
        if (any_hw) set_status(a.res, CO3_ERR_CUDA);
        if (any_err) set_status(a.res, CO3_ERR_CORRUPT);
        if (any_hw || any_err) atomicMin(&a.res->first_bad_chunk, td.chunk0);
    }
}

// ------------------------------------------------------------------------------------------------
// code build: Huffman code of one segment from its 256 weights (Sec. IV-A (ii)), one block per segment,
// thread = symbol.  Same construction and tie order as the host function co3_code_build: leaves ordered
// by (weight, symbol), merged nodes by age, a leaf before a merged node of equal weight; weights are halved
// and the construction repeated while the longest codeword exceeds CO3_MAX_CODE_LEN; canonical codewords.
// ------------------------------------------------------------------------------------------------
struct CodeBuildArgs {
    const uint64_t* weights;  // [n_seg][256]
    const co3_fmt* fmts;
    co3_code* out;
    co3_result* res;
};

// Same rule as the prepare kernel applies to symbols: the exponent code is not all ones, no "minus zero",
// and with flushed sub-normals exponent code 0 carries mantissa code 0.
__device__ __forceinline__ bool symbol_has_level(const co3_fmt& f, uint32_t sym) {
    const uint32_t nb = (uint32_t)f.exp_bits + f.mant_bits;
    if (sym >= (2u << nb)) return false;
    const uint32_t sign = sym >> nb, mag = sym & ((1u << nb) - 1u);
    const uint32_t efield = mag >> f.mant_bits, mfield = mag & ((1u << f.mant_bits) - 1u);
    if (efield == (1u << f.exp_bits) - 1u) return false;
    if (mag == 0) return sign == 0;
    if (efield == 0 && (f.flags & CO3_FMT_FLUSH_SUBNORMALS) && mfield != 0) return false;
    return true;
}

// Number of lanes, counted from lane 0, for which `ok` holds without a gap.
__device__ __forceinline__ uint32_t leading_lanes(bool ok) {
    const uint32_t bal = __ballot_sync(0xffffffffu, ok);
    return bal == 0xffffffffu ? 32u : (uint32_t)__ffs((int)~bal) - 1u;
}

// The two-queue merge of one tree, run by one warp.  node[0..n) holds the leaf weights in order; merged nodes
// are appended behind them; parent[] receives every node's parent.  Each step of the sequential method takes
// the two smallest of the queue heads, a leaf winning ties.  The warp takes whole runs of steps at once:
//   * while the second waiting leaf is not heavier than the merged queue's head, both picks are leaves, and
//     none of the nodes created meanwhile is consumed: up to 32 leaf pairs are merged side by side;
//   * while the second waiting merged node is lighter than the leaf head, both picks are merged nodes: up to 32
//     pairs of nodes that already exist are merged side by side;
//   * otherwise the step takes one of each.
// T is wide enough for the weight sum, and ~0 is larger than any sum.
template <typename T>
__device__ __forceinline__ void merge_queues(T* node, uint16_t* parent, uint32_t n) {
    const T kNone = ~(T)0;
    const uint32_t lane = threadIdx.x & 31u;
    uint32_t qa = 0, qb = n, t = n;  // leaves qa..n-1 and merged nodes qb..t-1 are waiting (same in every lane)
    while (t < 2 * n - 1) {
        // everything a step may need is requested at once: the two heads of both queues (the same addresses in every
        // lane) and this lane's pair in either queue
        const uint32_t ia = qa + 2 * lane, ib = qb + 2 * lane;
        const T a0 = qa < n ? node[qa] : kNone, a1 = qa + 1 < n ? node[qa + 1] : kNone;
        const T b0 = qb < t ? node[qb] : kNone, b1 = qb + 1 < t ? node[qb + 1] : kNone;
        const T la0 = ia < n ? node[ia] : kNone, la1 = ia + 1 < n ? node[ia + 1] : kNone;
        const T lb0 = ib < t ? node[ib] : kNone, lb1 = ib + 1 < t ? node[ib + 1] : kNone;
        uint32_t m;
        if (a1 != kNone && a1 <= b0) {
            // leaf pairs; with an empty merged queue the first pair's node becomes the head the others face
            const T head = b0 != kNone ? b0 : a0 + a1;
            m = leading_lanes(lane == 0 || (la1 != kNone && la1 <= head));
            if (lane < m) {
                node[t + lane] = la0 + la1;
                parent[ia] = parent[ia + 1] = (uint16_t)(t + lane);
            }
            qa += 2 * m;
        } else if (b1 != kNone && b1 < a0) {
            // pairs of merged nodes that exist already (the ones created here wait behind them)
            m = leading_lanes(lane == 0 || (lb1 != kNone && lb1 < a0));
            if (lane < m) {
                node[t + lane] = lb0 + lb1;
                parent[ib] = parent[ib + 1] = (uint16_t)(t + lane);
            }
            qb += 2 * m;
        } else {
            // one leaf and one merged node
            m = 1;
            if (lane == 0) {
                node[t] = a0 + b0;
                parent[qa] = parent[qb] = (uint16_t)t;
            }
            ++qa;
            ++qb;
        }
        t += m;
        __syncwarp();
    }
}

// One candidate tree, built by one warp: the weights after `h` halvings, max(1, w >> h) (halving h times
// with a floor of 1 gives exactly that).  The warp puts the leaves in order (a sort of (weight, symbol) keys for
// 32-bit weights, a count of the leaves before each symbol for wider ones), merges, and the lanes walk from their
// leaves to the root.  Returns the longest codeword; len_out[sym] receives the lengths.
template <typename T>
__device__ __forceinline__ uint32_t build_tree(const uint64_t* s_w, uint32_t h, uint32_t n, T* node, uint16_t* parent,
                                               uint8_t* len_out) {
    const uint32_t lane = threadIdx.x & 31u;
    T w[8];
    uint32_t rank[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const uint64_t x = s_w[lane + 32 * i];
        w[i] = x ? (T)max(x >> h, (uint64_t)1) : (T)0;
        rank[i] = 0;
    }
    if (sizeof(T) == 4) {
        // 32-bit weights: weight and symbol make one 64-bit key, and the warp sorts the 256 keys (eight per lane,
        // element e = 8 * lane + r) with a bitonic network: exchanges inside a lane between registers, across lanes by
        // shuffles.  A symbol that takes no part gets the largest key and ends up behind the n leaves.
        uint64_t key[8];
#pragma unroll
        for (int r = 0; r < 8; ++r) {
            const uint32_t sym = 8u * lane + (uint32_t)r;
            const uint64_t x = s_w[sym];
            key[r] = x ? ((max(x >> h, (uint64_t)1) << 8) | sym) : ~0ull;
        }
#pragma unroll
        for (int k = 2; k <= 256; k <<= 1) {
#pragma unroll
            for (int j = k >> 1; j > 0; j >>= 1) {
                if (j >= 8) {
                    const bool up = ((8u * lane) & (uint32_t)k) == 0;           // this element's run is ascending
                    const bool keep_min = (((lane & (uint32_t)(j >> 3)) == 0) == up);  // the pair's lower place takes the minimum
#pragma unroll
                    for (int r = 0; r < 8; ++r) {
                        const uint64_t other = __shfl_xor_sync(0xffffffffu, key[r], j >> 3);
                        key[r] = keep_min ? min(key[r], other) : max(key[r], other);
                    }
                } else {
#pragma unroll
                    for (int r = 0; r < 8; ++r) {
                        if ((r & j) == 0) {
                            const bool up = k < 8 ? ((r & k) == 0) : (((8u * lane) & (uint32_t)k) == 0);
                            const uint64_t lo = min(key[r], key[r ^ j]), hi = max(key[r], key[r ^ j]);
                            key[r] = up ? lo : hi;
                            key[r ^ j] = up ? hi : lo;
                        }
                    }
                }
            }
        }
        uint16_t* place = parent + 256;  // where each symbol's leaf went; free until the merge writes parents
#pragma unroll
        for (int r = 0; r < 8; ++r) {
            if (key[r] != ~0ull) {
                node[8u * lane + (uint32_t)r] = (T)(key[r] >> 8);
                place[key[r] & 0xffu] = (uint16_t)(8u * lane + (uint32_t)r);
            }
        }
        __syncwarp();
#pragma unroll
        for (int i = 0; i < 8; ++i) rank[i] = place[lane + 32 * i];
    } else {
        // wider weights: every lane counts, for each of its symbols, the leaves that come before it.  The candidate's
        // weights lie side by side for that (behind the leaves, where merged nodes go later); a symbol that takes no
        // part gets a weight above every other, so that it is never counted
        T* wp = node + 256;
#pragma unroll
        for (int i = 0; i < 8; ++i) wp[lane + 32 * i] = w[i] ? w[i] : ~(T)0;
        __syncwarp();
#pragma unroll 8
        for (uint32_t j = 0; j < 256; ++j) {
            const T wj = wp[j];
#pragma unroll
            for (int i = 0; i < 8; ++i) rank[i] += (wj < w[i] || (wj == w[i] && j < lane + 32 * i)) ? 1u : 0u;
        }
        __syncwarp();  // every lane is done with wp[] before the leaves and, later, the merged nodes are written
#pragma unroll
        for (int i = 0; i < 8; ++i)
            if (w[i]) node[rank[i]] = w[i];
    }
    __syncwarp();
    merge_queues<T>(node, parent, n);
    // from every leaf up to the root, the lane's eight walks side by side
    uint32_t v[8], len[8], longest = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        v[i] = w[i] ? rank[i] : 2 * n - 2;
        len[i] = 0;
    }
    for (;;) {
        bool moved = false;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            if (v[i] != 2 * n - 2) {
                v[i] = parent[v[i]];
                ++len[i];
                moved = true;
            }
        }
        if (!moved) break;
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        len_out[lane + 32 * i] = (uint8_t)len[i];
        longest = max(longest, len[i]);
    }
    return __reduce_max_sync(0xffffffffu, longest);
}

constexpr int kCandidates = kThreads / 32;  // trees built side by side, one per warp

__global__ void __launch_bounds__(kThreads) code_build_kernel(CodeBuildArgs a) {
    wait_for_previous_kernel();
    __shared__ uint64_t s_w[256];                    // weight of every symbol, 0 = takes no part
    __shared__ uint64_t s_node[kCandidates][512];    // per candidate: the n leaves in order, then the merged nodes by age
    __shared__ uint16_t s_parent[kCandidates][512];
    __shared__ uint8_t s_len[kCandidates][256];
    __shared__ uint32_t s_longest[kCandidates];
    __shared__ uint64_t s_red[8];
    const uint32_t k = blockIdx.x, sym = threadIdx.x, warp = sym >> 5;
    if (k == 0 && sym == 0) a.res->first_bad_chunk = 0xffffffffu;
    const co3_fmt f = a.fmts[k];
    bool fmt_ok = f.exp_bits >= 2 && 1u + f.exp_bits + f.mant_bits <= 8u && !(f.flags & ~CO3_FMT_FLUSH_SUBNORMALS);
    fmt_ok = fmt_ok && f.scale > 0.0f && f.inv_scale > 0.0f && !isinf(f.scale) && !isinf(f.inv_scale);
    const bool valid = fmt_ok && symbol_has_level(f, sym);
    uint64_t w = 0;
    if (valid) {
        w = a.weights[(size_t)k * 256 + sym];
        if (w == 0) w = 1;
    }
    // the weights must add up to less than 2^63: sum their halves separately, neither sum can wrap
    const uint64_t hi = block_sum_u64(w >> 32, s_red), lo = block_sum_u64(w & 0xffffffffull, s_red);
    const bool sum_ok = hi + (lo >> 32) < (1ull << 31);
    const uint32_t n = __syncthreads_count(valid);
    a.out[k].len[sym] = 0;
    a.out[k].bits[sym] = 0;
    if (!fmt_ok || !sum_ok || n < 2) {
        if (sym == 0) set_status(a.res, CO3_ERR_INVALID_ARG);
        return;
    }
    const bool narrow = hi == 0 && lo < 0xffffffffull;  // every weight sum fits 32 bits
    s_w[sym] = w;
    __syncthreads();
    // The code wanted is the one after the fewest halvings whose longest codeword fits.  Each warp tries one
    // number of halvings; eight at a time, until one fits (63 halvings leave all weights at 1).
    uint32_t len = 0;
    for (uint32_t h0 = 0;; h0 += kCandidates) {
        const uint32_t h = min(h0 + warp, 63u);
        uint32_t longest;
        if (narrow) longest = build_tree<uint32_t>(s_w, h, n, reinterpret_cast<uint32_t*>(s_node[warp]), s_parent[warp], s_len[warp]);
        else longest = build_tree<uint64_t>(s_w, h, n, s_node[warp], s_parent[warp], s_len[warp]);
        if ((sym & 31u) == 0) s_longest[warp] = longest;
        __syncthreads();
        uint32_t pick = kCandidates;
        for (int c = kCandidates - 1; c >= 0; --c)
            if (s_longest[c] <= (uint32_t)CO3_MAX_CODE_LEN) pick = (uint32_t)c;
        if (pick < (uint32_t)kCandidates) {
            len = s_len[pick][sym];
            break;
        }
        __syncthreads();  // everyone has read the candidates before they are rebuilt
    }
    // canonical codewords: in (length, symbol) order the codeword of a symbol is the sum of 2^(16 - length)
    // over the symbols before it, cut to its own length
    __syncthreads();
    s_len[0][sym] = (uint8_t)len;
    __syncthreads();
    if (valid) {
        uint32_t before = 0;
#pragma unroll 8
        for (uint32_t j = 0; j < 256; ++j) {
            const uint32_t lj = s_len[0][j];
            if (lj != 0 && (lj < len || (lj == len && j < sym))) before += 1u << (CO3_MAX_CODE_LEN - lj);
        }
        a.out[k].len[sym] = (uint8_t)len;
        a.out[k].bits[sym] = (uint16_t)(before >> (CO3_MAX_CODE_LEN - len));
    }
}

// ------------------------------------------------------------------------------------------------
// Fit of the converter's multiplier (Sec. III: a layer's gradients are zero-mean GenNorm(alpha, beta);
// Sec. IV-A (i): the multiplier minimises the expected squared conversion error under that model).
//   moments_kernel   per (chunk, client): sum v^2 and sum v^4 in fp64, v = g + gamma*m, fixed summation tree
//   fit_kernel       per layer: partial sums in fixed order -> sigma, kurtosis -> shape by bisection on
//                    Gamma(5/b)Gamma(1/b)/Gamma(3/b)^2 -> alpha -> tabulated best multiplier / alpha
// ------------------------------------------------------------------------------------------------
struct FitArgs {
    const float* grad;
    const float* mem;  // nullable: v = g
    float decay;
    uint64_t client_stride;
    uint32_t n_clients;
    co3_fmt* fmts;
    const co3_seg* segs;
    uint32_t n_seg;
    const float* log_tab;     // [n_tab][n_beta]
    const uint32_t* seg_tab;  // nullable: every layer uses table 0
    uint32_t n_tab, n_beta;
    float beta0, dbeta;
    double* stats;  // nullable, [n_seg][4]
    double2* part;  // [n_clients][n_chunks_max]
    double2* range_part;   // [n_seg][kFitRanges]
    uint32_t* range_done;  // [n_seg], zero at launch
    co3_result* res;
    Ws ws;
};

constexpr int kMomChunks = 4;  // chunks of one client per block

__device__ __forceinline__ void moments_add(float g, float m, float decay, bool has_m, double& s2, double& s4) {
    const float v = has_m ? __fmaf_rn(decay, m, g) : g;
    const double x2 = __dmul_rn((double)v, (double)v);
    s2 = __dadd_rn(s2, x2);
    s4 = __dadd_rn(s4, __dmul_rn(x2, x2));
}

// kNorms: the two sums are |g| and |m| (error magnitude, Sec. VI) instead of v^2 and v^4.
template <bool kNorms>
__global__ void __launch_bounds__(kThreads) moments_kernel(FitArgs a) {
    __shared__ double s_red[kMomChunks][2][kThreads / 32];
    const Ctrl* ctrl = a.ws.ctrl;
    if (ctrl->abort) return;
    const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
    const uint32_t n_chunks = ctrl->n_chunks, client = blockIdx.y;
    const bool has_m = a.mem != nullptr;
    const uint32_t i0 = tid * 8;
    const uint32_t c_first = blockIdx.x * kMomChunks;
    float g[kMomChunks][8], m[kMomChunks][8];
    uint32_t nv[kMomChunks];
    // all loads of the block's chunks first, then the arithmetic
#pragma unroll
    for (int j = 0; j < kMomChunks; ++j) {
        const uint32_t c = c_first + j;
        nv[j] = 0;
        if (c >= n_chunks) continue;
        const ChunkDesc d = a.ws.chunk_desc[c];
        const uint64_t base = (uint64_t)client * a.client_stride + d.elem0;
        const float* gp = a.grad + base;
        const float* mp = has_m ? a.mem + base : gp;
        nv[j] = d.cnt > i0 ? min(8u, d.cnt - i0) : 0u;
        const bool vec = d.cnt == (uint32_t)kC && ((reinterpret_cast<uintptr_t>(gp) | reinterpret_cast<uintptr_t>(mp)) & 15u) == 0;
        if (vec) {
            load8_vec(gp + i0, g[j]);
            if (has_m) load8_vec(mp + i0, m[j]);
        } else {
            load8_any(gp + i0, nv[j], g[j]);
            if (has_m) load8_any(mp + i0, nv[j], m[j]);
        }
    }
#pragma unroll
    for (int j = 0; j < kMomChunks; ++j) {
        double s2 = 0.0, s4 = 0.0;
#pragma unroll
        for (int e = 0; e < 8; ++e)
            if ((uint32_t)e < nv[j]) {
                if (kNorms) {
                    s2 = __dadd_rn(s2, fabs((double)g[j][e]));
                    s4 = __dadd_rn(s4, fabs((double)m[j][e]));
                } else {
                    moments_add(g[j][e], has_m ? m[j][e] : 0.0f, a.decay, has_m, s2, s4);
                }
            }
#pragma unroll
        for (int w = 16; w > 0; w >>= 1) {
            s2 = __dadd_rn(s2, __shfl_xor_sync(0xffffffffu, s2, w));
            s4 = __dadd_rn(s4, __shfl_xor_sync(0xffffffffu, s4, w));
        }
        if (lane == 0) { s_red[j][0][warp] = s2; s_red[j][1][warp] = s4; }
    }
    __syncthreads();
    if (tid < (uint32_t)kMomChunks && c_first + tid < n_chunks) {
        double t2 = 0.0, t4 = 0.0;
#pragma unroll
        for (int w = 0; w < kThreads / 32; ++w) { t2 = __dadd_rn(t2, s_red[tid][0][w]); t4 = __dadd_rn(t4, s_red[tid][1][w]); }
        a.part[(size_t)client * a.ws.n_chunks_max + c_first + tid] = make_double2(t2, t4);
    }
}

__device__ __forceinline__ double gennorm_kurtosis(double beta) {
    return exp(lgamma(5.0 / beta) + lgamma(1.0 / beta) - 2.0 * lgamma(3.0 / beta));
}

constexpr int kFitRanges = 64;  // a layer's partial sums are added up by this many blocks, each over a fixed share

__global__ void __launch_bounds__(kThreads) fit_kernel(FitArgs a) {
    __shared__ double s_red[2][kThreads / 32];
    __shared__ uint32_t s_last;
    const Ctrl* ctrl = a.ws.ctrl;
    if (ctrl->abort) return;
    const uint32_t k = blockIdx.x, r = blockIdx.y, tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
    const uint32_t c0 = a.ws.first_chunk[k], nck = a.ws.first_chunk[k + 1] - c0;
    const uint64_t items = (uint64_t)nck * a.n_clients;
    // block (k, r) adds the r-th share of the layer's (client, chunk) sums, every thread its own items in order;
    // the shares and the order in which they are combined do not depend on the GPU or on timing
    const uint64_t per = (items + kFitRanges - 1) / kFitRanges;
    const uint64_t i_lo = min(items, (uint64_t)r * per), i_hi = min(items, i_lo + per);
    double s2 = 0.0, s4 = 0.0;
    for (uint64_t i = i_lo + tid; i < i_hi; i += kThreads) {
        const uint32_t u = (uint32_t)(i / nck), c = (uint32_t)(i % nck);
        const double2 p = a.part[(size_t)u * a.ws.n_chunks_max + c0 + c];
        s2 = __dadd_rn(s2, p.x);
        s4 = __dadd_rn(s4, p.y);
    }
#pragma unroll
    for (int w = 16; w > 0; w >>= 1) {
        s2 = __dadd_rn(s2, __shfl_xor_sync(0xffffffffu, s2, w));
        s4 = __dadd_rn(s4, __shfl_xor_sync(0xffffffffu, s4, w));
    }
    if (lane == 0) { s_red[0][warp] = s2; s_red[1][warp] = s4; }
    __syncthreads();
    if (tid == 0) {
        s2 = s4 = 0.0;
#pragma unroll
        for (int w = 0; w < kThreads / 32; ++w) { s2 = __dadd_rn(s2, s_red[0][w]); s4 = __dadd_rn(s4, s_red[1][w]); }
        a.range_part[(size_t)k * kFitRanges + r] = make_double2(s2, s4);
        __threadfence();
        s_last = atomicAdd(&a.range_done[k], 1u) == (uint32_t)kFitRanges - 1u ? 1u : 0u;
    }
    __syncthreads();
    if (!s_last || warp != 0) return;  // the block that finishes a layer's sums last fits the layer
    __threadfence();
    s2 = s4 = 0.0;
    for (int q = 0; q < kFitRanges; ++q) {
        const double2 p = __ldcg(&a.range_part[(size_t)k * kFitRanges + q]);
        s2 = __dadd_rn(s2, p.x);
        s4 = __dadd_rn(s4, p.y);
    }

    // warp 0, every lane with the same values
    const double N = (double)a.segs[k].n_elem * (double)a.n_clients;
    bool ok = a.n_beta >= 2 && N > 0.0 && s2 > 0.0 && isfinite(s2) && isfinite(s4);
    const uint32_t tab = a.seg_tab ? a.seg_tab[k] : 0u;
    if (tab >= a.n_tab) ok = false;
    float sc = 0.0f;
    double sigma = 0.0, kurt = 0.0, beta = 0.0, alpha = 0.0;
    if (ok) {
        sigma = sqrt(s2 / N);
        kurt = N * s4 / (s2 * s2);
        const double blo = (double)a.beta0, bhi = (double)a.beta0 + (double)a.dbeta * (double)(a.n_beta - 1);
        // the kurtosis falls as the shape grows; outside the table's range the nearer end is taken.  Inside, the
        // interval is cut into 33 parts per round, one interior point per lane, until it is as narrow as fp64 allows
        double lo = blo, hi = bhi;
        const double k_end = gennorm_kurtosis(lane == 0 ? lo : hi);
        const bool below_lo = !(kurt < __shfl_sync(0xffffffffu, k_end, 0));
        const bool above_hi = !(kurt > __shfl_sync(0xffffffffu, k_end, 1));
        if (below_lo) beta = lo;
        else if (above_hi) beta = hi;
        else {
            for (int it = 0; it < 64 && hi - lo > 1e-15 * hi; ++it) {
                const double w = hi - lo;
                const double x = lo + w * ((double)(lane + 1) / 33.0);
                const uint32_t left = __popc(__ballot_sync(0xffffffffu, gennorm_kurtosis(x) > kurt));  // points left of the root
                const double nlo = left == 0 ? lo : lo + w * ((double)left / 33.0);
                const double nhi = left == 32 ? hi : lo + w * ((double)(left + 1) / 33.0);
                if (!(nhi - nlo < w)) break;  // no further progress in fp64
                lo = nlo;
                hi = nhi;
            }
            beta = 0.5 * (lo + hi);
        }
        alpha = sigma * sqrt(exp(lgamma(1.0 / beta) - lgamma(3.0 / beta)));
        double x = (beta - blo) / (double)a.dbeta;
        if (x < 0.0) x = 0.0;
        uint32_t i = (uint32_t)x;
        if (i > a.n_beta - 2) i = a.n_beta - 2;
        const double f = x - (double)i;
        const float* t = a.log_tab + (size_t)tab * a.n_beta;
        const double log_s = (double)t[i] + f * ((double)t[i + 1] - (double)t[i]);
        sc = (float)(exp(log_s) / alpha);
        if (!(sc > 0.0f) || isinf(sc)) ok = false;
    }
    if (lane != 0) return;
    if (!ok) {  // empty, all-zero or non-finite layer, or no usable table: the format is left as it was
        set_status(&a.res[0], CO3_ERR_INVALID_ARG);
        atomicMin(&a.res[0].first_bad_chunk, k);
        return;
    }
    a.fmts[k].scale = sc;
    a.fmts[k].inv_scale = __fdiv_rn(1.0f, sc);
    if (a.stats) {
        double* st = a.stats + 4 * (size_t)k;
        st[0] = sigma; st[1] = kurt; st[2] = beta; st[3] = alpha;
    }
}

// Error magnitude (Sec. VI): per client and layer the l1 norms of the gradient and of the memory, from the
// per-chunk sums of moments_kernel<true>.  Block (k, r, u) adds the r-th share of the chunk sums of layer k of
// client u; the block that finishes a (layer, client) last adds the shares in order and writes the result.
struct MagArgs {
    const double2* part;  // [n_clients][n_chunks_max]
    double2* range_part;  // [n_clients][n_seg][kFitRanges]
    uint32_t* range_done; // [n_clients][n_seg], zero at launch
    double* out;          // [n_clients][n_seg][2]
    uint32_t n_seg;
    Ws ws;
};

__global__ void __launch_bounds__(kThreads) magnitude_kernel(MagArgs a) {
    __shared__ double s_red[2][kThreads / 32];
    if (a.ws.ctrl->abort) return;
    const uint32_t k = blockIdx.x, r = blockIdx.y, u = blockIdx.z, tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
    const uint32_t c0 = a.ws.first_chunk[k], nck = a.ws.first_chunk[k + 1] - c0;
    const uint32_t per = (nck + kFitRanges - 1) / kFitRanges;
    const uint32_t i_lo = min(nck, r * per), i_hi = min(nck, i_lo + per);
    const double2* part = a.part + (size_t)u * a.ws.n_chunks_max + c0;
    double sg = 0.0, sm = 0.0;
    for (uint32_t i = i_lo + tid; i < i_hi; i += kThreads) {
        const double2 p = part[i];
        sg = __dadd_rn(sg, p.x);
        sm = __dadd_rn(sm, p.y);
    }
#pragma unroll
    for (int w = 16; w > 0; w >>= 1) {
        sg = __dadd_rn(sg, __shfl_xor_sync(0xffffffffu, sg, w));
        sm = __dadd_rn(sm, __shfl_xor_sync(0xffffffffu, sm, w));
    }
    if (lane == 0) { s_red[0][warp] = sg; s_red[1][warp] = sm; }
    __syncthreads();
    if (tid != 0) return;
    sg = sm = 0.0;
#pragma unroll
    for (int w = 0; w < kThreads / 32; ++w) { sg = __dadd_rn(sg, s_red[0][w]); sm = __dadd_rn(sm, s_red[1][w]); }
    const size_t cell = (size_t)u * a.n_seg + k;
    a.range_part[cell * kFitRanges + r] = make_double2(sg, sm);
    __threadfence();
    if (atomicAdd(&a.range_done[cell], 1u) != (uint32_t)kFitRanges - 1u) return;
    __threadfence();
    sg = sm = 0.0;
    for (int q = 0; q < kFitRanges; ++q) {
        const double2 p = __ldcg(&a.range_part[cell * kFitRanges + q]);
        sg = __dadd_rn(sg, p.x);
        sm = __dadd_rn(sm, p.y);
    }
    a.out[2 * cell] = sg;
    a.out[2 * cell + 1] = sm;
}

// ------------------------------------------------------------------------------------------------
// Huffman weights from the model (Sec. IV-A (ii): the code of a layer is designed for the GenNorm distribution
// fitted to it).  The probability of a symbol is the GenNorm mass of the interval of inputs the converter sends
// to its level: between the midpoints to the neighbouring levels, divided by the multiplier; the last level's
// interval has no upper end.  With F the distribution function of GenNorm(0, alpha, beta),
// F(x) - 1/2 = P(1/beta, (x/alpha)^beta) / 2 for x >= 0, P the regularised lower incomplete gamma function.
// ------------------------------------------------------------------------------------------------
struct WeightArgs {
    const co3_fmt* fmts;
    const double* stats;  // [n_seg][4]: beta at [2], alpha at [3]
    uint64_t* weights;    // [n_seg][256]
    co3_result* res;
};

// P(a, x) for a > 0, x >= 0: power series below x = a + 1, continued fraction of the complement above.
__device__ double gamma_p(double a, double x, double lgamma_a) {
    if (!(x > 0.0)) return 0.0;
    if (isinf(x)) return 1.0;
    const double front = exp(a * log(x) - x - lgamma_a);  // x^a e^-x / Gamma(a)
    if (x < a + 1.0) {
        double term = 1.0 / a, sum = term;
        for (int n = 1; n < 1000; ++n) {
            term *= x / (a + (double)n);
            sum += term;
            if (term < sum * 1e-17) break;
        }
        return fmin(1.0, front * sum);
    }
    const double tiny = 1e-300;
    double b = x + 1.0 - a, c = 1.0 / tiny, d = 1.0 / b, h = d;
    for (int i = 1; i < 1000; ++i) {
        const double an = -(double)i * ((double)i - a);
        b += 2.0;
        d = an * d + b;
        if (fabs(d) < tiny) d = tiny;
        c = b + an / c;
        if (fabs(c) < tiny) c = tiny;
        d = 1.0 / d;
        const double del = d * c;
        h *= del;
        if (fabs(del - 1.0) < 1e-16) break;
    }
    return fmax(0.0, 1.0 - front * h);
}

// Value of magnitude code c in the format (E, M), before the multiplier.
__device__ __forceinline__ double level_of(uint32_t c, uint32_t M, int emin) {
    const uint32_t efield = c >> M, mfield = c & ((1u << M) - 1u);
    if (efield == 0) return ldexp((double)mfield, emin - (int)M);
    return ldexp(1.0 + ldexp((double)mfield, -(int)M), (int)efield - 1 + emin);
}

__global__ void __launch_bounds__(kThreads) model_weights_kernel(WeightArgs a) {
    const uint32_t k = blockIdx.x, sym = threadIdx.x;
    const co3_fmt f = a.fmts[k];
    const double beta = a.stats[4 * (size_t)k + 2], alpha = a.stats[4 * (size_t)k + 3];
    const uint32_t E = f.exp_bits, M = f.mant_bits;
    const bool ok = E >= 2 && 1 + E + M <= 8 && (f.flags & ~CO3_FMT_FLUSH_SUBNORMALS) == 0 && f.scale > 0.0f &&
                    !isinf(f.scale) && beta > 0.0 && alpha > 0.0 && isfinite(beta) && isfinite(alpha);
    uint64_t w = 0;
    if (ok) {
        const bool flush = (f.flags & CO3_FMT_FLUSH_SUBNORMALS) != 0;
        const int emin = -((1 << (E - 1)) - 2);
        const uint32_t nb = E + M, max_code = (((1u << E) - 2u) << M) | ((1u << M) - 1u);
        const uint32_t sign = sym >> nb, c = sym & ((1u << nb) - 1u);
        const bool valid = sym < (2u << nb) && c <= max_code && !(sign && c == 0) && !(flush && c != 0 && (c >> M) == 0);
        if (valid) {
            const double inv_a = 1.0 / beta, lg = lgamma(inv_a);
            const double here = level_of(c, M, emin);
            double lo = 0.0, hi = INFINITY;  // ends of the interval, in units of the input
            if (c != 0) {
                const uint32_t prev = (flush && c == (1u << M)) ? 0u : c - 1u;
                lo = 0.5 * (level_of(prev, M, emin) + here) / (double)f.scale;
            }
            if (c != max_code) {
                const uint32_t next = (flush && c == 0) ? (1u << M) : c + 1u;
                hi = 0.5 * (here + level_of(next, M, emin)) / (double)f.scale;
            }
            const double p_lo = gamma_p(inv_a, pow(lo / alpha, beta), lg);
            const double p_hi = isinf(hi) ? 1.0 : gamma_p(inv_a, pow(hi / alpha, beta), lg);
            const double p = (c == 0 ? 1.0 : 0.5) * (p_hi - p_lo);  // zero collects both signs
            w = p > 0.0 ? (uint64_t)floor(p * 1073741824.0) : 0ull;
        }
    } else if (sym == 0) {
        set_status(&a.res[0], CO3_ERR_INVALID_ARG);
        atomicMin(&a.res[0].first_bad_chunk, k);
    }
    a.weights[(size_t)k * 256 + sym] = w;
}

}  // namespace co3

// ================================================================================================
// Host side: argument checks, workspace layout, launches.
// ================================================================================================
using namespace co3;

namespace {

struct WsLayout {
    size_t ctrl, first_chunk, chunk_desc, tile_desc, fmt, enc_lut, dec_lut, dec_sub, val_lut, client_fail, chunk_bits,
        bit_prefix, range_tot, totals, slots, total;
    uint32_t n_ranges_max;
    uint32_t n_chunks_max;
};

size_t up256(size_t x) { return (x + 255) & ~(size_t)255; }

bool ws_layout(uint64_t n_elem, uint32_t n_seg, uint32_t n_clients, WsLayout* L) {
    if (n_elem > (1ull << 40) || n_seg > (1u << 20)) return false;
    const uint64_t nc = n_elem / kC + n_seg;  // upper bound of the chunks of one client
    if (nc >= (1ull << 31)) return false;
    L->n_chunks_max = (uint32_t)nc;
    size_t o = 0;
    L->ctrl = o;        o += up256(sizeof(Ctrl));
    L->client_fail = o; o += up256(4 * (size_t)(n_clients ? n_clients : 1));  // directly behind ctrl: cleared with it
    L->first_chunk = o; o += up256(4 * ((size_t)n_seg + 1));
    L->chunk_desc = o;  o += up256(sizeof(ChunkDesc) * (size_t)nc);
    L->tile_desc = o;   o += up256(sizeof(TileDesc) * (size_t)nc);
    L->fmt = o;         o += up256(sizeof(FmtDev) * (size_t)n_seg);
    L->enc_lut = o;     o += up256(4 * 256 * (size_t)n_seg);
    L->dec_lut = o;     o += up256(2 * (size_t)kDecLut * n_seg);
    L->dec_sub = o;     o += up256(2 * (size_t)kSubLut * n_seg);
    L->val_lut = o;     o += up256(4 * 256 * (size_t)n_seg);
    L->chunk_bits = o;  o += up256(4 * (size_t)n_clients * nc);
    L->bit_prefix = o;  o += up256(8 * (size_t)n_clients * (nc + 1));
    L->n_ranges_max = (uint32_t)(nc / kRangeChunks + 1);
    L->range_tot = o;   o += up256(16 * (size_t)n_clients * L->n_ranges_max);
    L->totals = o;      o += up256(16 * (size_t)(n_clients ? n_clients : 1));
    L->slots = o;       o += up256(4 * (size_t)kSlotWords * n_clients * nc);
    L->total = o;
    return true;
}

Ws ws_pointers(void* base, const WsLayout& L) {
    char* b = static_cast<char*>(base);
    Ws w;
    w.ctrl = reinterpret_cast<Ctrl*>(b + L.ctrl);
    w.first_chunk = reinterpret_cast<uint32_t*>(b + L.first_chunk);
    w.chunk_desc = reinterpret_cast<ChunkDesc*>(b + L.chunk_desc);
    w.tile_desc = reinterpret_cast<TileDesc*>(b + L.tile_desc);
    w.fmt = reinterpret_cast<FmtDev*>(b + L.fmt);
    w.enc_lut = reinterpret_cast<uint32_t*>(b + L.enc_lut);
    w.dec_lut = reinterpret_cast<uint16_t*>(b + L.dec_lut);
    w.dec_sub = reinterpret_cast<uint16_t*>(b + L.dec_sub);
    w.val_lut = reinterpret_cast<float*>(b + L.val_lut);
    w.client_fail = reinterpret_cast<uint32_t*>(b + L.client_fail);
    w.chunk_bits = reinterpret_cast<uint32_t*>(b + L.chunk_bits);
    w.bit_prefix = reinterpret_cast<uint64_t*>(b + L.bit_prefix);
    w.range_tot = reinterpret_cast<uint64_t*>(b + L.range_tot);
    w.totals = reinterpret_cast<uint64_t*>(b + L.totals);
    w.slots = reinterpret_cast<uint32_t*>(b + L.slots);
    w.n_chunks_max = L.n_chunks_max;
    return w;
}

// Largest possible size of the container sections that precede the payload.
uint64_t fixed_part_bound(uint32_t n_seg, uint64_t n_chunks_max) {
    uint64_t o = align16(kHeaderBytes + 24ull * n_seg);
    o = align16(o + 8ull * (n_chunks_max + 1));
    o = align16(o + 2ull * n_chunks_max * kSubs);
    return o;
}

#define CO3_CUDA(call)                                  \
    do {                                                \
        if ((call) != cudaSuccess) return CO3_ERR_CUDA; \
    } while (0)

// Blocks of a persistent kernel: enough to fill every SM at the kernel's occupancy, never more than the work.
// grouped: items are handed out four consecutive ones at a time when that still leaves every block many groups
// (the kernels with private histograms, which flush them when the layer changes; the others balance better one by one).
constexpr uint32_t kItemGroup = 4;

template <typename Kernel>
int persistent_grid(Kernel kernel, int threads, size_t smem, uint64_t items, bool grouped, uint32_t* grid, uint32_t* group) {
    int dev = 0, sms = 0, per_sm = 0;
    CO3_CUDA(cudaGetDevice(&dev));
    CO3_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    CO3_CUDA(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    CO3_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, threads, smem));
    if (per_sm < 1) return CO3_ERR_CUDA;
    const uint64_t want = (uint64_t)sms * (uint64_t)per_sm;
    *group = (grouped && items >= 8ull * kItemGroup * want) ? kItemGroup : 1u;
    const uint64_t groups = (items + *group - 1) / *group;
    *grid = (uint32_t)(groups < want ? groups : want);
    return CO3_OK;
}

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

// Optional per-kernel timing (off by default): an event pair around every launch, read back by
// co3_profile_read.  Used by benchmarks to time the kernels inside the entry points.
struct Profiler {
    static constexpr int kMaxRecords = 16384;
    bool on = false;
    int n = 0;
    int ids[kMaxRecords];
    cudaEvent_t ev[kMaxRecords][2];
    int n_created = 0;
    void begin(int id, cudaStream_t st) {
        if (!on || n >= kMaxRecords) return;
        if (n >= n_created) {
            if (cudaEventCreate(&ev[n][0]) != cudaSuccess || cudaEventCreate(&ev[n][1]) != cudaSuccess) { on = false; return; }
            ++n_created;
        }
        ids[n] = id;
        cudaEventRecord(ev[n][0], st);
    }
    void end(cudaStream_t st) {
        if (!on || n >= kMaxRecords) return;
        cudaEventRecord(ev[n][1], st);
        ++n;
    }
};
Profiler g_prof;

// Launch of a kernel that follows another kernel of the same call: programmatic stream serialization lets its launch
// overlap the tail of that kernel; the kernel itself starts with wait_for_previous_kernel().
template <typename... Params, typename... Args>
cudaError_t launch_behind(void (*kernel)(Params...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

#define CO3_LAUNCH(id, st, ...)        \
    do {                               \
        g_prof.begin(id, st);          \
        __VA_ARGS__;                   \
        g_prof.end(st);                \
        CO3_CUDA(cudaGetLastError());  \
    } while (0)


int begin_call(const WsLayout& L, const Ws& ws, co3_result* res, uint32_t n_res, cudaStream_t st,
               const co3_fmt* fmts, const co3_code* codes, const co3_seg* segs, uint32_t n_seg, uint64_t n_elem,
               uint32_t tile_chunks, uint32_t n_fail, const uint8_t* const* streams = nullptr,
               const uint8_t* single = nullptr, size_t stream_bytes = 0, uint32_t n_streams = 0,
               void* also_clear = nullptr, size_t also_clear_bytes = 0) {
    // one launch clears the call-wide state with the per-client failure marks (side by side in the workspace), the
    // results, and what else the call wants zero (a multiple of four bytes)
    static_assert(sizeof(co3_result) % 4 == 0, "results are cleared word by word");
    ClearArgs cl{};
    cl.p[0] = reinterpret_cast<uint32_t*>(ws.ctrl);
    cl.words[0] = ((L.client_fail - L.ctrl) + 4 * (size_t)(n_fail ? n_fail : 1)) / 4;
    cl.p[1] = reinterpret_cast<uint32_t*>(res);
    cl.words[1] = sizeof(co3_result) * (size_t)n_res / 4;
    cl.p[2] = static_cast<uint32_t*>(also_clear);
    cl.words[2] = also_clear_bytes / 4;
    const uint64_t clear_words = cl.words[0] + cl.words[1] + cl.words[2];
    const uint32_t clear_blocks = (uint32_t)std::min<uint64_t>(1024, (clear_words + 4 * kThreads - 1) / (4 * kThreads));
    CO3_LAUNCH(CO3_KERNEL_CLEAR, st, CO3_CUDA(launch_behind(clear_kernel, clear_blocks ? clear_blocks : 1u, kThreads, 0, st, cl)));
    PrepArgs pa{fmts, codes, segs, n_seg, n_elem, tile_chunks, res, n_res, n_streams ? 1u : 0u, streams, single, stream_bytes, n_streams, ws};
    // extra blocks per segment when segments are long (their chunk descriptors are written in parallel)
    const uint64_t per_seg = L.n_chunks_max / (n_seg ? n_seg : 1);
    const uint32_t helpers = (uint32_t)std::min<uint64_t>(128, per_seg / (8 * kThreads) + 1);
    CO3_LAUNCH(CO3_KERNEL_PREPARE, st, CO3_CUDA(launch_behind(prepare_kernel, dim3(n_seg ? n_seg : 1, helpers), kThreads, 0, st, pa)));
    return CO3_OK;
}

int decode_common(const uint8_t* const* streams, const uint8_t* single, size_t stream_bytes, uint32_t n_clients,
                  const co3_fmt* fmts, const co3_code* codes, const co3_seg* segs, uint32_t n_seg, uint64_t n_elem,
                  uint32_t chunk_syms, float* out, uint8_t* sym_out, float* params, float lr, void* workspace,
                  size_t workspace_bytes, co3_result* res, cudaStream_t st) {
    if ((!streams && !single) || !fmts || !codes || !res || !workspace || n_clients == 0 || chunk_syms != (uint32_t)kC)
        return CO3_ERR_INVALID_ARG;
    if ((!segs && n_seg) || (!out && !sym_out && !params) || (sym_out && n_clients != 1)) return CO3_ERR_INVALID_ARG;
    if (params && !aligned(params, 16)) return CO3_ERR_INVALID_ARG;
    if (!aligned(workspace, 256) || (out && !aligned(out, 16)) || !aligned(res, 8)) return CO3_ERR_INVALID_ARG;
    WsLayout L;
    if (!ws_layout(n_elem, n_seg, 0, &L)) return CO3_ERR_INVALID_ARG;
    if (workspace_bytes < L.total) return CO3_ERR_CAPACITY;
    const Ws ws = ws_pointers(workspace, L);

    // B clients side by side and G chunks per block, 16 sub-chunk threads per (chunk, client) pair, at most
    // 16 pairs; small inputs take fewer chunks per block so that the grid still covers the GPU
    const bool multi = n_clients > (uint32_t)kMaxPairs;
    uint32_t B = n_clients;
    if (multi) {  // equal batches of at most kMultiPairs clients, never fewer than 16 side by side
        const uint32_t batches = (n_clients + kMultiPairs - 1) / kMultiPairs;
        B = std::max<uint32_t>(16u, (n_clients + batches - 1) / batches);
    }
    uint32_t G = multi ? 1u : (uint32_t)kMaxPairs / B;
    const uint32_t g_min = (B == 1) ? 2u : 1u;  // a block needs at least one full warp
    if (!multi && G > g_min) {
        int dev = 0, sms = 0;
        CO3_CUDA(cudaGetDevice(&dev));
        CO3_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
        const uint64_t want = L.n_chunks_max / (2 * (uint64_t)(sms > 0 ? sms : 1)) + 1;  // chunks per block that still give two waves
        if (want < G) G = (uint32_t)(want < g_min ? g_min : want);
    }
    const int rc = begin_call(L, ws, res, 1, st, fmts, codes, segs, n_seg, n_elem, G, 1, streams, single, stream_bytes, n_clients);
    if (rc != CO3_OK) return rc;
    DecArgs da{streams, single, stream_bytes, n_clients, segs, n_seg, n_elem, out, sym_out, params, lr, res, B, G, ws};
    const uint32_t tiles = (uint32_t)(L.n_chunks_max / G + n_seg);  // upper bound; surplus blocks return at once
    if (tiles == 0) return CO3_OK;
    const uint32_t n_pairs = B * G;
    const size_t smem = sizeof(DecSmem) + 4 * ((size_t)n_pairs * (kPairPhaseWords + kPaySlotWords) + kPaySlack);
    if (multi) {
        CO3_CUDA(cudaFuncSetAttribute(decode_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        CO3_LAUNCH(CO3_KERNEL_DECODE, st, CO3_CUDA(launch_behind(decode_kernel<true, false>, tiles, 16 * n_pairs, smem, st, da)));
    } else if (n_clients == 1) {
        CO3_CUDA(cudaFuncSetAttribute(decode_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        CO3_LAUNCH(CO3_KERNEL_DECODE, st, CO3_CUDA(launch_behind(decode_kernel<false, true>, tiles, 16 * n_pairs, smem, st, da)));
    } else {
        CO3_CUDA(cudaFuncSetAttribute(decode_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        CO3_LAUNCH(CO3_KERNEL_DECODE, st, CO3_CUDA(launch_behind(decode_kernel<false, false>, tiles, 16 * n_pairs, smem, st, da)));
    }
    return CO3_OK;
}

int encode_common(const float* grad, float* mem, float decay, const uint8_t* sym, const co3_fmt* fmts,
                  const co3_code* codes, const co3_seg* segs, uint32_t n_seg, uint64_t n_elem, uint32_t n_clients,
                  uint64_t client_stride, uint8_t* streams_out, size_t stream_capacity, uint32_t chunk_syms,
                  void* workspace, size_t workspace_bytes, co3_result* res, cudaStream_t st, bool dither = false,
                  uint32_t seed = 0) {
    if (!codes || !res || !workspace || !streams_out || n_clients == 0 || n_clients > 65535u ||
        chunk_syms != (uint32_t)kC)
        return CO3_ERR_INVALID_ARG;
    if (!segs && n_seg) return CO3_ERR_INVALID_ARG;
    if (sym == nullptr && (!grad || !mem || !fmts || !aligned(grad, 16) || !aligned(mem, 16))) return CO3_ERR_INVALID_ARG;
    if (!aligned(workspace, 256) || !aligned(streams_out, 16) || (stream_capacity & 15u) || !aligned(res, 8))
        return CO3_ERR_INVALID_ARG;
    if (n_clients > 1 && client_stride < n_elem) return CO3_ERR_INVALID_ARG;
    WsLayout L;
    if (!ws_layout(n_elem, n_seg, n_clients, &L)) return CO3_ERR_INVALID_ARG;
    if (workspace_bytes < L.total) return CO3_ERR_CAPACITY;
    if (stream_capacity < fixed_part_bound(n_seg, L.n_chunks_max)) return CO3_ERR_CAPACITY;
    const Ws ws = ws_pointers(workspace, L);
    const int rc = begin_call(L, ws, res, n_clients, st, sym ? nullptr : fmts, codes, segs, n_seg, n_elem, 1, n_clients);
    if (rc != CO3_OK) return rc;
    if (L.n_chunks_max) {
        PackArgs pa{grad, mem, decay, sym, client_stride, n_clients, streams_out, stream_capacity, res, 1u, seed, ws};
        const uint64_t items = (uint64_t)L.n_chunks_max * n_clients;
        uint32_t grid = 0;
#define CO3_PACK_CASE(S, D)                                                                                          \
    {                                                                                                                \
        const int g = persistent_grid(pack_kernel<S, D>, kPackThreads, sizeof(PackSmem), items, false, &grid, &pa.group); \
        if (g != CO3_OK) return g;                                                                                   \
        CO3_LAUNCH(CO3_KERNEL_PACK, st, CO3_CUDA(launch_behind(pack_kernel<S, D>, grid, kPackThreads, sizeof(PackSmem), st, pa))); \
    }
        if (sym) CO3_PACK_CASE(true, false)
        else if (dither) CO3_PACK_CASE(false, true)
        else CO3_PACK_CASE(false, false)
#undef CO3_PACK_CASE
    }
    // inputs beyond a few tiles of chunks per client: offsets by a two-level scan over many blocks
    const uint32_t two_level = L.n_chunks_max > 4u * kRangeChunks ? 1u : 0u;
    ScanArgs sa{segs, n_seg, n_elem, streams_out, stream_capacity, res, two_level, L.n_ranges_max, ws};
    if (two_level) {
        const dim3 rgrid(L.n_ranges_max, n_clients);
        CO3_LAUNCH(CO3_KERNEL_SCAN, st, CO3_CUDA(launch_behind(range_totals_kernel, rgrid, kScanThreads, 0, st, sa)));
        CO3_LAUNCH(CO3_KERNEL_SCAN, st, CO3_CUDA(launch_behind(range_scan_kernel, n_clients, kScanThreads, 0, st, sa)));
        CO3_LAUNCH(CO3_KERNEL_SCAN, st, CO3_CUDA(launch_behind(range_apply_kernel, rgrid, kScanThreads, 0, st, sa)));
    }
    CO3_LAUNCH(CO3_KERNEL_SCAN, st, CO3_CUDA(launch_behind(scan_kernel, n_clients, kScanThreads, 0, st, sa)));
    if (L.n_chunks_max) {
        CO3_LAUNCH(CO3_KERNEL_COMPACT, st, CO3_CUDA(launch_behind(compact_kernel, dim3((L.n_chunks_max + kThreads / 32 - 1) / (kThreads / 32), n_clients), kThreads, 0, st, sa)));
    }
    return CO3_OK;
}

}  // namespace

extern "C" {

const char* co3_status_string(int status) {
    switch (status) {
        case CO3_OK: return "ok";
        case CO3_ERR_INVALID_ARG: return "invalid argument or descriptor";
        case CO3_ERR_CAPACITY: return "stream or workspace too small";
        case CO3_ERR_NO_CODEWORD: return "symbol without codeword";
        case CO3_ERR_NONFINITE: return "non-finite input (stream still valid)";
        case CO3_ERR_CORRUPT: return "corrupt stream";
        case CO3_ERR_CUDA: return "CUDA runtime error";
        default: return "unknown status";
    }
}

int co3_profile_enable(int on) {
    g_prof.n = 0;
    g_prof.on = on != 0;
    return CO3_OK;
}

int co3_profile_read(double* total_ms, uint32_t* launches) {
    if (!total_ms || !launches) return CO3_ERR_INVALID_ARG;
    for (int i = 0; i < CO3_KERNEL_COUNT; ++i) { total_ms[i] = 0.0; launches[i] = 0; }
    for (int r = 0; r < g_prof.n; ++r) {
        float ms = 0.0f;
        CO3_CUDA(cudaEventSynchronize(g_prof.ev[r][1]));
        CO3_CUDA(cudaEventElapsedTime(&ms, g_prof.ev[r][0], g_prof.ev[r][1]));
        total_ms[g_prof.ids[r]] += ms;
        launches[g_prof.ids[r]] += 1;
    }
    g_prof.n = 0;
    return CO3_OK;
}

int co3_workspace_bytes(uint64_t n_elem, uint32_t n_seg, uint32_t n_clients, uint32_t chunk_syms, size_t* out) {
    if (!out || chunk_syms != (uint32_t)kC) return CO3_ERR_INVALID_ARG;
    WsLayout L;
    if (!ws_layout(n_elem, n_seg, n_clients, &L)) return CO3_ERR_INVALID_ARG;
    *out = L.total;
    return CO3_OK;
}

int co3_stream_capacity_bytes(uint64_t n_elem, uint32_t n_seg, uint32_t chunk_syms, size_t* out) {
    if (!out || chunk_syms != (uint32_t)kC) return CO3_ERR_INVALID_ARG;
    WsLayout L;
    if (!ws_layout(n_elem, n_seg, 0, &L)) return CO3_ERR_INVALID_ARG;
    // every chunk rounds its bits up to a word: at most n_elem/2 words plus one per chunk
    const uint64_t words = (n_elem * CO3_MAX_CODE_LEN + 31) / 32 + L.n_chunks_max;
    *out = (size_t)align16(fixed_part_bound(n_seg, L.n_chunks_max) + 4ull * words);
    return CO3_OK;
}

static int convert_common(const float* grad, float* mem, bool store_mem, float decay, const co3_fmt* fmts,
                          const co3_seg* segs, uint32_t n_seg, uint64_t n_elem, uint32_t n_clients,
                          uint64_t client_stride_elems, uint8_t* sym_out, uint64_t* hist_out, co3_result* res,
                          void* workspace, size_t workspace_bytes, cudaStream_t st, bool dither = false,
                          uint32_t seed = 0) {
    if (!grad || !mem || !fmts || !res || !workspace || n_clients == 0 || n_clients > 65535u) return CO3_ERR_INVALID_ARG;
    if (!segs && n_seg) return CO3_ERR_INVALID_ARG;
    if (!aligned(grad, 16) || !aligned(mem, 16) || !aligned(workspace, 256) || !aligned(res, 8) ||
        (hist_out && !aligned(hist_out, 8)))
        return CO3_ERR_INVALID_ARG;
    if (n_clients > 1 && client_stride_elems < n_elem) return CO3_ERR_INVALID_ARG;
    WsLayout L;
    if (!ws_layout(n_elem, n_seg, 0, &L)) return CO3_ERR_INVALID_ARG;
    if (workspace_bytes < L.total) return CO3_ERR_CAPACITY;
    const Ws ws = ws_pointers(workspace, L);
    const int rc = begin_call(L, ws, res, n_clients, st, fmts, nullptr, segs, n_seg, n_elem, 1, 1, nullptr, nullptr, 0, 0,
                              hist_out, hist_out ? 8 * 256 * (size_t)n_seg : 0);
    if (rc != CO3_OK) return rc;
    if (L.n_chunks_max == 0) return CO3_OK;
    ConvertArgs ca{grad, mem, decay, client_stride_elems, n_clients, sym_out, hist_out, res, 1u, seed, ws};
    const uint64_t items = (uint64_t)L.n_chunks_max * n_clients;
    const size_t smem = sizeof(Feed) + (hist_out ? 4 * (size_t)kHistStride * kHistCopies : 0);
    uint32_t grid = 0;
#define CO3_CONVERT_CASE2(S, H, M, D)                                                                                \
    {                                                                                                                \
        constexpr int T = (!(M) && !(D)) ? 128 : kThreads; /* the dry pass runs 128-thread blocks */                 \
        const int g = persistent_grid(convert_kernel<S, H, M, D, T>, T, smem, items, H, &grid, &ca.group);           \
        if (g != CO3_OK) return g;                                                                                   \
        CO3_LAUNCH(CO3_KERNEL_CONVERT, st, CO3_CUDA(launch_behind(convert_kernel<S, H, M, D, T>, grid, T, smem, st, ca))); \
    }
#define CO3_CONVERT_CASE(S, H, M)                  \
    {                                              \
        if (dither) CO3_CONVERT_CASE2(S, H, M, true) \
        else CO3_CONVERT_CASE2(S, H, M, false)     \
    }
    if (!store_mem) CO3_CONVERT_CASE(false, true, false)
    else if (sym_out && hist_out) CO3_CONVERT_CASE(true, true, true)
    else if (sym_out) CO3_CONVERT_CASE(true, false, true)
    else if (hist_out) CO3_CONVERT_CASE(false, true, true)
    else CO3_CONVERT_CASE(false, false, true)
#undef CO3_CONVERT_CASE2
#undef CO3_CONVERT_CASE
    return CO3_OK;
}

int co3_convert(const float* grad, float* mem, float decay, const co3_fmt* fmts, const co3_seg* segs, uint32_t n_seg,
                uint64_t n_elem, uint32_t n_clients, uint64_t client_stride_elems, uint8_t* sym_out,
                uint64_t* hist_out, co3_result* res, void* workspace, size_t workspace_bytes, void* stream) {
    return convert_common(grad, mem, true, decay, fmts, segs, n_seg, n_elem, n_clients, client_stride_elems, sym_out,
                          hist_out, res, workspace, workspace_bytes, static_cast<cudaStream_t>(stream));
}

int co3_histogram(const float* grad, const float* mem, float decay, const co3_fmt* fmts, const co3_seg* segs,
                  uint32_t n_seg, uint64_t n_elem, uint32_t n_clients, uint64_t client_stride_elems,
                  uint64_t* hist_out, co3_result* res, void* workspace, size_t workspace_bytes, void* stream) {
    if (!hist_out) return CO3_ERR_INVALID_ARG;
    // the kernel instance without the memory store never writes through this pointer
    return convert_common(grad, const_cast<float*>(mem), false, decay, fmts, segs, n_seg, n_elem, n_clients,
                          client_stride_elems, nullptr, hist_out, res, workspace, workspace_bytes,
                          static_cast<cudaStream_t>(stream));
}

int co3_convert_dither(const float* grad, float* mem, float decay, const co3_fmt* fmts, const co3_seg* segs,
                       uint32_t n_seg, uint64_t n_elem, uint32_t n_clients, uint64_t client_stride_elems,
                       uint32_t seed, uint8_t* sym_out, uint64_t* hist_out, co3_result* res, void* workspace,
                       size_t workspace_bytes, void* stream) {
    return convert_common(grad, mem, true, decay, fmts, segs, n_seg, n_elem, n_clients, client_stride_elems, sym_out,
                          hist_out, res, workspace, workspace_bytes, static_cast<cudaStream_t>(stream), true, seed);
}

int co3_histogram_dither(const float* grad, const float* mem, float decay, const co3_fmt* fmts, const co3_seg* segs,
                         uint32_t n_seg, uint64_t n_elem, uint32_t n_clients, uint64_t client_stride_elems,
                         uint32_t seed, uint64_t* hist_out, co3_result* res, void* workspace, size_t workspace_bytes,
                         void* stream) {
    if (!hist_out) return CO3_ERR_INVALID_ARG;
    return convert_common(grad, const_cast<float*>(mem), false, decay, fmts, segs, n_seg, n_elem, n_clients,
                          client_stride_elems, nullptr, hist_out, res, workspace, workspace_bytes,
                          static_cast<cudaStream_t>(stream), true, seed);
}

// ------------------------------------------------------------------------------------------------
// co3_convert_static: the convert entry point for callers that must not allocate device memory.
// Its scratch space is the file-scope array below, part of the library image: every device that loads
// the library holds one copy until the process exits.
// ------------------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_static_scratch[CO3_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
// Device address of g_static_scratch on each device, null until that device's first call.  In host code the
// array's name is only a handle for cudaGetSymbolAddress, never an address a kernel may use.
void* g_static_scratch_addr[kMaxDevices];

int static_scratch_address(void** out) {
    int dev = -1;
    CO3_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return CO3_ERR_INVALID_ARG;
    if (g_static_scratch_addr[dev] == nullptr) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) return CO3_ERR_CUDA;
        g_static_scratch_addr[dev] = p;
    }
    *out = g_static_scratch_addr[dev];
    return CO3_OK;
}
}  // namespace

int co3_code_build_device(const uint64_t* weights, const co3_fmt* fmts, uint32_t n_seg, co3_code* codes_out,
                          co3_result* res, void* stream) {
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (!weights || !fmts || !codes_out || !res || n_seg == 0 || n_seg > (1u << 20)) return CO3_ERR_INVALID_ARG;
    if (!aligned(weights, 8) || !aligned(fmts, 4) || !aligned(codes_out, 2) || !aligned(res, 8)) return CO3_ERR_INVALID_ARG;
    ClearArgs cl{};
    cl.p[0] = reinterpret_cast<uint32_t*>(res);
    cl.words[0] = sizeof(co3_result) / 4;
    CO3_LAUNCH(CO3_KERNEL_CLEAR, st, CO3_CUDA(launch_behind(clear_kernel, 1u, kThreads, 0, st, cl)));
    CodeBuildArgs ca{weights, fmts, codes_out, res};
    CO3_LAUNCH(CO3_KERNEL_CODE_BUILD, st, CO3_CUDA(launch_behind(code_build_kernel, n_seg, kThreads, 0, st, ca)));
    return CO3_OK;
}

int co3_convert_static(const float* grad, float* mem, float decay, const co3_fmt* fmts, const co3_seg* segs,
                       uint32_t n_seg, uint64_t n_elem, uint32_t n_clients, uint64_t client_stride_elems,
                       uint8_t* sym_out, uint64_t* hist_out, co3_result* res, void* stream) {
    size_t need = 0;
    const int rc = co3_workspace_bytes(n_elem, n_seg, 0, CO3_CHUNK_SYMS, &need);
    if (rc != CO3_OK) return rc;
    if (need > (size_t)CO3_STATIC_SCRATCH_BYTES) return CO3_ERR_CAPACITY;  // layout too large for the built-in scratch
    void* scratch = nullptr;
    const int ra = static_scratch_address(&scratch);
    if (ra != CO3_OK) return ra;
    return co3_convert(grad, mem, decay, fmts, segs, n_seg, n_elem, n_clients, client_stride_elems, sym_out, hist_out,
                       res, scratch, (size_t)CO3_STATIC_SCRATCH_BYTES, stream);
}

int co3_fit_scale(const float* grad, const float* mem, float decay, co3_fmt* fmts, const co3_seg* segs, uint32_t n_seg,
                  uint64_t n_elem, uint32_t n_clients, uint64_t client_stride_elems, const float* log_tab,
                  const uint32_t* seg_tab, uint32_t n_tab, uint32_t n_beta, float beta0, float dbeta, double* stats_out,
                  co3_result* res, void* workspace, size_t workspace_bytes, void* stream) {
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (!grad || !fmts || !segs || !log_tab || !res || !workspace || n_seg == 0 || n_clients == 0 || n_clients > 65535u)
        return CO3_ERR_INVALID_ARG;
    if (n_tab == 0 || n_beta < 2 || !(dbeta > 0.0f) || !(beta0 > 0.0f)) return CO3_ERR_INVALID_ARG;
    if (!aligned(grad, 16) || (mem && !aligned(mem, 16)) || !aligned(workspace, 256) || !aligned(res, 8) ||
        !aligned(fmts, 4) || !aligned(log_tab, 4) || (stats_out && !aligned(stats_out, 8)))
        return CO3_ERR_INVALID_ARG;
    if (n_clients > 1 && client_stride_elems < n_elem) return CO3_ERR_INVALID_ARG;
    WsLayout L;
    if (!ws_layout(n_elem, n_seg, n_clients, &L)) return CO3_ERR_INVALID_ARG;
    if (workspace_bytes < L.total) return CO3_ERR_CAPACITY;
    const Ws ws = ws_pointers(workspace, L);
    // layout only: the formats' multipliers are what this call produces, so they are not validated here
    const int rc = begin_call(L, ws, res, 1, st, nullptr, nullptr, segs, n_seg, n_elem, 1, 1);
    if (rc != CO3_OK) return rc;
    // the per-(chunk, client) partial sums take the place of the encoder's chunk slots (16 of 4096 bytes each)
    // and behind them the per-layer range sums and completion counters of the fit
    double2* part = reinterpret_cast<double2*>(ws.slots);
    static_assert(16 * (kFitRanges + 1) + 4 <= 4 * kSlotWords, "the fit's scratch fits in the slots of n_seg chunks");
    double2* range_part = part + (size_t)n_clients * L.n_chunks_max;
    uint32_t* range_done = reinterpret_cast<uint32_t*>(range_part + (size_t)n_seg * kFitRanges);
    CO3_CUDA(cudaMemsetAsync(range_done, 0, 4 * (size_t)n_seg, st));
    FitArgs fa{grad, mem, decay, client_stride_elems, n_clients, fmts, segs, n_seg, log_tab, seg_tab, n_tab, n_beta,
               beta0, dbeta, stats_out, part, range_part, range_done, res, ws};
    if (L.n_chunks_max) {
        const dim3 grid((L.n_chunks_max + kMomChunks - 1) / kMomChunks, n_clients);
        CO3_LAUNCH(CO3_KERNEL_FIT, st, moments_kernel<false><<<grid, kThreads, 0, st>>>(fa));
    }
    CO3_LAUNCH(CO3_KERNEL_FIT, st, fit_kernel<<<dim3(n_seg, kFitRanges), kThreads, 0, st>>>(fa));
    return CO3_OK;
}

int co3_error_magnitude(const float* grad, const float* mem, const co3_seg* segs, uint32_t n_seg, uint64_t n_elem,
                        uint32_t n_clients, uint64_t client_stride_elems, double* norms_out, co3_result* res,
                        void* workspace, size_t workspace_bytes, void* stream) {
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (!grad || !mem || !segs || !norms_out || !res || !workspace || n_seg == 0 || n_clients == 0 || n_clients > 65535u)
        return CO3_ERR_INVALID_ARG;
    if (!aligned(grad, 16) || !aligned(mem, 16) || !aligned(workspace, 256) || !aligned(res, 8) || !aligned(norms_out, 8))
        return CO3_ERR_INVALID_ARG;
    if (n_clients > 1 && client_stride_elems < n_elem) return CO3_ERR_INVALID_ARG;
    WsLayout L;
    if (!ws_layout(n_elem, n_seg, n_clients, &L)) return CO3_ERR_INVALID_ARG;
    if (workspace_bytes < L.total) return CO3_ERR_CAPACITY;
    const Ws ws = ws_pointers(workspace, L);
    const int rc = begin_call(L, ws, res, 1, st, nullptr, nullptr, segs, n_seg, n_elem, 1, 1);
    if (rc != CO3_OK) return rc;
    // scratch inside the encoder's chunk slots: 16 bytes per (chunk, client), then 16 * kFitRanges + 4 per (layer, client)
    double2* part = reinterpret_cast<double2*>(ws.slots);
    double2* range_part = part + (size_t)n_clients * L.n_chunks_max;
    uint32_t* range_done = reinterpret_cast<uint32_t*>(range_part + (size_t)n_seg * n_clients * kFitRanges);
    CO3_CUDA(cudaMemsetAsync(range_done, 0, 4 * (size_t)n_seg * n_clients, st));
    FitArgs fa{};
    fa.grad = grad;
    fa.mem = mem;
    fa.client_stride = client_stride_elems;
    fa.n_clients = n_clients;
    fa.part = part;
    fa.ws = ws;
    if (L.n_chunks_max) {
        const dim3 grid((L.n_chunks_max + kMomChunks - 1) / kMomChunks, n_clients);
        CO3_LAUNCH(CO3_KERNEL_FIT, st, moments_kernel<true><<<grid, kThreads, 0, st>>>(fa));
    }
    MagArgs ma{part, range_part, range_done, norms_out, n_seg, ws};
    CO3_LAUNCH(CO3_KERNEL_FIT, st, magnitude_kernel<<<dim3(n_seg, kFitRanges, n_clients), kThreads, 0, st>>>(ma));
    return CO3_OK;
}

int co3_model_weights(const co3_fmt* fmts, const double* stats, uint32_t n_seg, uint64_t* weights_out, co3_result* res,
                      void* stream) {
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (!fmts || !stats || !weights_out || !res || n_seg == 0 || n_seg > (1u << 20)) return CO3_ERR_INVALID_ARG;
    if (!aligned(fmts, 4) || !aligned(stats, 8) || !aligned(weights_out, 8) || !aligned(res, 8)) return CO3_ERR_INVALID_ARG;
    CO3_CUDA(cudaMemsetAsync(res, 0, sizeof(co3_result), st));
    CO3_CUDA(cudaMemsetAsync(&res->first_bad_chunk, 0xff, 4, st));
    WeightArgs wa{fmts, stats, weights_out, res};
    CO3_LAUNCH(CO3_KERNEL_FIT, st, model_weights_kernel<<<n_seg, kThreads, 0, st>>>(wa));
    return CO3_OK;
}

int co3_encode(const float* grad, float* mem, float decay, const co3_fmt* fmts, const co3_code* codes,
               const co3_seg* segs, uint32_t n_seg, uint64_t n_elem, uint32_t n_clients, uint64_t client_stride_elems,
               uint8_t* streams_out, size_t stream_capacity, uint32_t chunk_syms, void* workspace,
               size_t workspace_bytes, co3_result* res, void* stream) {
    if (!grad || !mem || !fmts) return CO3_ERR_INVALID_ARG;
    return encode_common(grad, mem, decay, nullptr, fmts, codes, segs, n_seg, n_elem, n_clients, client_stride_elems,
                         streams_out, stream_capacity, chunk_syms, workspace, workspace_bytes, res,
                         static_cast<cudaStream_t>(stream));
}

int co3_encode_dither(const float* grad, float* mem, float decay, const co3_fmt* fmts, const co3_code* codes,
                      const co3_seg* segs, uint32_t n_seg, uint64_t n_elem, uint32_t n_clients,
                      uint64_t client_stride_elems, uint32_t seed, uint8_t* streams_out, size_t stream_capacity,
                      uint32_t chunk_syms, void* workspace, size_t workspace_bytes, co3_result* res, void* stream) {
    if (!grad || !mem || !fmts) return CO3_ERR_INVALID_ARG;
    return encode_common(grad, mem, decay, nullptr, fmts, codes, segs, n_seg, n_elem, n_clients, client_stride_elems,
                         streams_out, stream_capacity, chunk_syms, workspace, workspace_bytes, res,
                         static_cast<cudaStream_t>(stream), true, seed);
}

int co3_encode_symbols(const uint8_t* sym, const co3_code* codes, const co3_seg* segs, uint32_t n_seg, uint64_t n_elem,
                       uint32_t n_clients, uint64_t client_stride_elems, uint8_t* streams_out, size_t stream_capacity,
                       uint32_t chunk_syms, void* workspace, size_t workspace_bytes, co3_result* res, void* stream) {
    if (!sym) return CO3_ERR_INVALID_ARG;
    return encode_common(nullptr, nullptr, 0.0f, sym, nullptr, codes, segs, n_seg, n_elem, n_clients,
                         client_stride_elems, streams_out, stream_capacity, chunk_syms, workspace, workspace_bytes, res,
                         static_cast<cudaStream_t>(stream));
}

int co3_decode_aggregate(const uint8_t* const* streams, size_t stream_bytes, uint32_t n_clients, const co3_fmt* fmts,
                         const co3_code* codes, const co3_seg* segs, uint32_t n_seg, uint64_t n_elem,
                         uint32_t chunk_syms, float* avg_out, void* workspace, size_t workspace_bytes, co3_result* res,
                         void* stream) {
    if (!avg_out) return CO3_ERR_INVALID_ARG;
    if (!streams) return CO3_ERR_INVALID_ARG;
    return decode_common(streams, nullptr, stream_bytes, n_clients, fmts, codes, segs, n_seg, n_elem, chunk_syms, avg_out,
                         nullptr, nullptr, 0.0f, workspace, workspace_bytes, res, static_cast<cudaStream_t>(stream));
}

int co3_decode_aggregate_update(const uint8_t* const* streams, size_t stream_bytes, uint32_t n_clients, const co3_fmt* fmts,
                                const co3_code* codes, const co3_seg* segs, uint32_t n_seg, uint64_t n_elem,
                                uint32_t chunk_syms, float lr, float* params, float* avg_out, void* workspace,
                                size_t workspace_bytes, co3_result* res, void* stream) {
    if (!params || !streams) return CO3_ERR_INVALID_ARG;
    return decode_common(streams, nullptr, stream_bytes, n_clients, fmts, codes, segs, n_seg, n_elem, chunk_syms, avg_out,
                         nullptr, params, lr, workspace, workspace_bytes, res, static_cast<cudaStream_t>(stream));
}

int co3_decode(const uint8_t* stream_in, size_t stream_bytes, const co3_fmt* fmts, const co3_code* codes,
               const co3_seg* segs, uint32_t n_seg, uint64_t n_elem, uint32_t chunk_syms, float* ghat_out,
               uint8_t* sym_out, void* workspace, size_t workspace_bytes, co3_result* res, void* stream) {
    if (!stream_in || !aligned(stream_in, 16)) return CO3_ERR_INVALID_ARG;
    if (!ghat_out && !sym_out) return CO3_ERR_INVALID_ARG;
    return decode_common(nullptr, stream_in, stream_bytes, 1, fmts, codes, segs, n_seg, n_elem, chunk_syms, ghat_out,
                         sym_out, nullptr, 0.0f, workspace, workspace_bytes, res, static_cast<cudaStream_t>(stream));
}

}  // extern "C"
