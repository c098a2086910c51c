// Kernels and C-ABI host layer of the FFD sparse decode-attention library (sm_100a).
#include <cuda_runtime.h>
#include <math.h>
#include <string.h>

#include <mutex>

#include "../../include/ffd.h"
#include "ffd_kernels.cuh"
#include "ffd_fused.cuh"

namespace ffd {

// ---- quantize (App. A.1) ----------------------------------------------------------------------------------
// One CTA of 128 threads per (logical block, KV head, sequence).  The K tile goes through shared memory
// once: thread c owns channel c for the absmax / scale, then thread (mt, lane) assembles its 16 bytes of the
// packed layout.
struct QuantParams {
    const __nv_bfloat16* k_cache;
    uint8_t* k_quant;
    __half* k_scales;
    const int32_t* block_table;
    const int32_t* seq_lens;
    const int32_t* first_token;
    int Hkv, max_blocks, num_pages;
};

__device__ __forceinline__ uint32_t quant_code(float x, float s) {
    const bool neg = x < 0.f;
    const bool big = fabsf(x) >= s;
    return neg ? (big ? 0u : 1u) : (big ? 3u : 2u);
}

// One (page, KV head) tile, staged in shared memory as sk[64][128], by 128 threads: per-channel scale over the first
// `rows` rows (App. A.1), then the packed 2-bit codes.  Contains a __syncthreads().
// GROUP: the 128 calling threads are part of a larger CTA and meet at named barrier 1 instead of the CTA's.
template <bool GROUP = false>
__device__ __forceinline__ void quantize_tile(const __nv_bfloat16* sk, float* ss, int rows, __half* scales_out,
                                              uint8_t* codes_out, int tid) {
    {
        float a = 0.f;
#pragma unroll 16
        for (int r = 0; r < kBlk; ++r)   // (independent reads; rows past the sequence's end do not count)
            if (r < rows) a = fmaxf(a, fabsf(__bfloat162float(sk[r * kD + tid])));
        float s32 = __fdiv_rn(a, 1.5f);
        s32 = fminf(s32, 65504.f);
        const __half s = __float2half_rn(s32);
        scales_out[tid] = s;
        ss[tid] = __half2float(s);
    }
    if (GROUP) asm volatile("bar.sync 1, 128;\n" ::: "memory");
    else __syncthreads();
    const int mt = tid >> 5, lane = tid & 31, r = lane >> 2, j = lane & 3;
    uint32_t w[4] = {0u, 0u, 0u, 0u};
#pragma unroll
    for (int i = 0; i < 8; ++i) {
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int c = 32 * j + 4 * i + u;
            const float s = ss[c];
            const uint32_t lo_row = quant_code(__bfloat162float(sk[(16 * mt + r) * kD + c]), s);
            const uint32_t hi_row = quant_code(__bfloat162float(sk[(16 * mt + r + 8) * kD + c]), s);
            const int shift = 2 * i + 16 * (u & 1);
            w[(u >> 1) * 2 + 0] |= lo_row << shift;   // W0 / W2: token r
            w[(u >> 1) * 2 + 1] |= hi_row << shift;   // W1 / W3: token r + 8
        }
    }
    reinterpret_cast<uint4*>(codes_out)[mt * 32 + lane] = make_uint4(w[0], w[1], w[2], w[3]);
}

__device__ __forceinline__ void residual_rows(const __nv_bfloat16* sk, const float* ss, const float* sinv, int rows,
                                              int8_t* res_out, int tid);

// k_res != nullptr: also writes the tile's 8-bit residuals (see residual_kernel)
__global__ void __launch_bounds__(128) quantize_kernel(QuantParams p, int8_t* k_res) {
    const int g = blockIdx.y, b = blockIdx.z;
    pdl_launch_dependents();
    pdl_wait();
    int n = p.seq_lens[b];
    const int cap = p.max_blocks * kBlk;
    n = n < 0 ? 0 : (n > cap ? cap : n);
    const int nb = (n + kBlk - 1) / kBlk;
    const int first = p.first_token ? max(p.first_token[b], 0) / kBlk : 0;
    __shared__ __align__(16) __nv_bfloat16 sk[kBlk * kD];
    __shared__ float ss[kD], sinv[kD];
    const int tid = threadIdx.x;
    // the grid's x extent is bounded; every CTA walks its share of the blocks that need (re)quantizing
    for (int blk = first + blockIdx.x; blk < nb; blk += gridDim.x) {
        const int page = p.block_table ? p.block_table[(size_t)b * p.max_blocks + blk] : b * p.max_blocks + blk;
        if (page < 0 || page >= p.num_pages) continue;
        const int rows = min(kBlk, n - blk * kBlk);
        const size_t tile = (size_t)page * p.Hkv + g;
        const uint4* src = reinterpret_cast<const uint4*>(p.k_cache + tile * kBlk * kD);
        uint4* dst = reinterpret_cast<uint4*>(sk);
        __syncthreads();   // the previous block's tile is no longer needed
#pragma unroll
        for (int x = 0; x < 8; ++x) dst[tid + 128 * x] = ldg_stream(src + tid + 128 * x);
        __syncthreads();
        quantize_tile(sk, ss, rows, p.k_scales + tile * kD, p.k_quant + tile * kCodeBytes, tid);
        if (k_res) {   // (uniform over the CTA)
            sinv[tid] = __fdiv_rn(254.f, ss[tid]);
            __syncthreads();
            residual_rows(sk, ss, sinv, rows, k_res + tile * kBlk * kD, tid);
        }
    }
}

// ---- 8-bit residual (Sec. 3.1: k -> {k_quant, k_res}) ------------------------------------------------------
// For every valid element: the part of the key its 2-bit level misses, on the grid s / 254 of the channel's own
// scale (a mid-rise level leaves a remainder in [-s/2, s/2]): code8 = clamp(rint((x - level * s) * (254 / s))),
// each operation one IEEE binary32 operation; s = 0 (all-zero channel) and padding rows give 0.  The level is
// recomputed from x and the stored scale with the quantizer's own comparison, so the codes need not be unpacked.
// Runs after the quantizer (it reads the scales); row-major int8 [page][KV head][64][128].
struct ResidualParams {
    const __nv_bfloat16* k_cache;
    const __half* k_scales;
    int8_t* k_res;
    const int32_t* block_table;
    const int32_t* seq_lens;
    const int32_t* first_token;
    int Hkv, max_blocks, num_pages;
};

__device__ __forceinline__ int residual_code(float x, float s, float inv) {
    const float level_s = __fmul_rn((float)quant_code(x, s) - 1.5f, s);   // exact
    float t = rintf(__fmul_rn(__fsub_rn(x, level_s), inv));
    t = fminf(fmaxf(t, -127.f), 127.f);
    return s == 0.f ? 0 : (int)t;
}

__global__ void __launch_bounds__(128) residual_kernel(ResidualParams p) {
    const int g = blockIdx.y, b = blockIdx.z;
    pdl_launch_dependents();
    pdl_wait();
    int n = p.seq_lens[b];
    const int cap = p.max_blocks * kBlk;
    n = n < 0 ? 0 : (n > cap ? cap : n);
    const int nb = (n + kBlk - 1) / kBlk;
    const int first = p.first_token ? max(p.first_token[b], 0) / kBlk : 0;
    __shared__ __align__(16) __nv_bfloat16 sk[kBlk * kD];
    __shared__ float ss[kD], sinv[kD];
    const int tid = threadIdx.x;
    for (int blk = first + blockIdx.x; blk < nb; blk += gridDim.x) {
        const int page = p.block_table ? p.block_table[(size_t)b * p.max_blocks + blk] : b * p.max_blocks + blk;
        if (page < 0 || page >= p.num_pages) continue;
        const int rows = min(kBlk, n - blk * kBlk);
        const size_t tile = (size_t)page * p.Hkv + g;
        const uint4* src = reinterpret_cast<const uint4*>(p.k_cache + tile * kBlk * kD);
        uint4* dst = reinterpret_cast<uint4*>(sk);
        __syncthreads();   // the previous block's tile is no longer needed
#pragma unroll
        for (int x = 0; x < 8; ++x) dst[tid + 128 * x] = ldg_stream(src + tid + 128 * x);
        ss[tid] = __half2float(p.k_scales[tile * kD + tid]);
        sinv[tid] = __fdiv_rn(254.f, ss[tid]);
        __syncthreads();
        residual_rows(sk, ss, sinv, rows, p.k_res + tile * kBlk * kD, tid);
    }
}

// the residual codes of a staged tile (sk) given its scales (ss) and 254 / scale (sinv), by 128 threads: 16 consecutive
// channels of one token per thread and pass; rows past the sequence end get 0
__device__ __forceinline__ void residual_rows(const __nv_bfloat16* sk, const float* ss, const float* sinv, int rows,
                                              int8_t* res_out, int tid) {
    uint4* out = reinterpret_cast<uint4*>(res_out);
#pragma unroll
    for (int x = 0; x < 4; ++x) {
        const int chunk = tid + 128 * x, row = chunk >> 3, c0 = (chunk & 7) * 16;
        uint32_t w[4] = {0u, 0u, 0u, 0u};
        if (row < rows) {
#pragma unroll
            for (int u = 0; u < 16; ++u) {
                const int c = c0 + u;
                const int code = residual_code(__bfloat162float(sk[row * kD + c]), ss[c], sinv[c]);
                w[u >> 2] |= (uint32_t)(code & 0xff) << (8 * (u & 3));
            }
        }
        out[chunk] = make_uint4(w[0], w[1], w[2], w[3]);
    }
}

// ---- deeper thumbnails: 4 and 8 bits (App. "Bandwidth Proportionality of Quantization Depth") ----------------
// s = fp16(fp32(absmax) / (2^(b-1) - 1/2)); the cell of |x| is found by exact comparisons with k * s (exact in
// binary32: at most 7 x 11 significant bits), ties outward, +-0 on the positive side; an all-zero channel (s = 0)
// takes the outermost positive level like the 2-bit quantizer.  Packed order: see WideScan.
template <int BITS>
__device__ __forceinline__ uint32_t wide_code(float x, float s) {
    constexpr int kHalf = 1 << (BITS - 1);
    const float ax = fabsf(x);
    int m = kHalf - 1;
    if (s > 0.f) {
        m = (int)fminf(__fdiv_rn(ax, s), (float)(kHalf - 1));   // within one of the cell; settled by the exact comparisons below
        while (m + 1 <= kHalf - 1 && ax >= __fmul_rn((float)(m + 1), s)) ++m;
        while (m > 0 && ax < __fmul_rn((float)m, s)) --m;
    }
    return x < 0.f ? (uint32_t)(kHalf - 1 - m) : (uint32_t)(kHalf + m);
}

template <int BITS>
__global__ void __launch_bounds__(128) quantize_wide_kernel(QuantParams p) {
    const int g = blockIdx.y, b = blockIdx.z;
    pdl_launch_dependents();
    pdl_wait();
    int n = p.seq_lens[b];
    const int cap = p.max_blocks * kBlk;
    n = n < 0 ? 0 : (n > cap ? cap : n);
    const int nb = (n + kBlk - 1) / kBlk;
    const int first = p.first_token ? max(p.first_token[b], 0) / kBlk : 0;
    __shared__ __align__(16) __nv_bfloat16 sk[kBlk * kD];
    __shared__ float ss[kD];
    const int tid = threadIdx.x;
    constexpr float kTop = (float)(1 << (BITS - 1)) - 0.5f;
    for (int blk = first + blockIdx.x; blk < nb; blk += gridDim.x) {
        const int page = p.block_table ? p.block_table[(size_t)b * p.max_blocks + blk] : b * p.max_blocks + blk;
        if (page < 0 || page >= p.num_pages) continue;
        const int rows = min(kBlk, n - blk * kBlk);
        const size_t tile = (size_t)page * p.Hkv + g;
        const uint4* src = reinterpret_cast<const uint4*>(p.k_cache + tile * kBlk * kD);
        uint4* dst = reinterpret_cast<uint4*>(sk);
        __syncthreads();   // the previous block's tile is no longer needed
#pragma unroll
        for (int x = 0; x < 8; ++x) dst[tid + 128 * x] = ldg_stream(src + tid + 128 * x);
        __syncthreads();
        {
            float a = 0.f;
            for (int r = 0; r < kBlk; ++r)
                if (r < rows) a = fmaxf(a, fabsf(__bfloat162float(sk[r * kD + tid])));
            const __half s = __float2half_rn(fminf(__fdiv_rn(a, kTop), 65504.f));
            p.k_scales[tile * kD + tid] = s;
            ss[tid] = __half2float(s);
        }
        __syncthreads();
        const int mt = tid >> 5, lane = tid & 31, r = lane >> 2, j = lane & 3;
        uint32_t* out = reinterpret_cast<uint32_t*>(p.k_quant + tile * WideScan<BITS>::kTileBytes);
        for (int i = 0; i < 8; ++i) {
            uint32_t c[4][2];   // A register x, low / high element
#pragma unroll
            for (int x = 0; x < 4; ++x)
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int tok = 16 * mt + r + 8 * (x & 1), ch = 32 * j + 4 * i + 2 * (x >> 1) + e;
                    c[x][e] = wide_code<BITS>(__bfloat162float(sk[tok * kD + ch]), ss[ch]);
                }
            if (BITS == 4) {
                uint32_t w = 0;
#pragma unroll
                for (int x = 0; x < 4; ++x) w |= (c[x][0] << (4 * x)) | (c[x][1] << (16 + 4 * x));
                out[WideScan<BITS>::word(mt, lane, i)] = w;
            } else {
                out[WideScan<BITS>::word(mt, lane, 2 * i)] = c[0][0] | (c[1][0] << 8) | (c[0][1] << 16) | (c[1][1] << 24);
                out[WideScan<BITS>::word(mt, lane, 2 * i + 1)] = c[2][0] | (c[3][0] << 8) | (c[2][1] << 16) | (c[3][1] << 24);
            }
        }
    }
}

// canonical codes [pages, Hkv, 64, 128] (0 .. 2^b - 1) from the packed layout of the deeper thumbnails
template <int BITS>
__global__ void __launch_bounds__(128) unpack_wide_kernel(const uint8_t* k_quant, uint8_t* codes, size_t tiles) {
    const size_t tile = blockIdx.x;
    if (tile >= tiles) return;
    const int tid = threadIdx.x;
    const int mt = tid >> 5, lane = tid & 31, r = lane >> 2, j = lane & 3;
    const uint32_t* w = reinterpret_cast<const uint32_t*>(k_quant + tile * WideScan<BITS>::kTileBytes);
    uint8_t* dst = codes + tile * kBlk * kD;
    for (int i = 0; i < 8; ++i)
        for (int x = 0; x < 4; ++x)
            for (int e = 0; e < 2; ++e) {
                const int tok = 16 * mt + r + 8 * (x & 1), ch = 32 * j + 4 * i + 2 * (x >> 1) + e;
                uint32_t c;
                if (BITS == 4) c = (w[WideScan<BITS>::word(mt, lane, i)] >> (4 * x + 16 * e)) & 0xFu;
                else c = (w[WideScan<BITS>::word(mt, lane, 2 * i + (x >> 1))] >> (8 * (x & 1) + 16 * e)) & 0xFFu;
                dst[tok * kD + ch] = (uint8_t)c;
            }
}

// ---- whole-cache quantizer ---------------------------------------------------------------------------------
// The same arithmetic as quantize_tile, organised for bandwidth: per element the plain routine spends ~9
// instructions (16-bit shared-memory reads, conversions, two compares, selects, shifts) and is instruction-bound at
// 3 TB/s.  Here a tile is staged with cp.async, all shared-memory reads are 16 bytes, and the code of a pair of
// channels comes from three packed bf16 compares:
//   code = [x > -s] + [x >= 0] + [x >= s]   (0..3; -0 counts as >= 0)
// x is a bf16, s an fp16 with more mantissa bits, so "x >= s" is tested against t = the smallest bf16 >= s (the same
// truth value for every bf16 x), "x > -s" against -t; a channel whose scale is 0 holds only zeros and takes code 3,
// as the comparison form of App. A.1 gives it (its lower threshold becomes -inf).  Adding 128 to the sum leaves the
// code in the two low mantissa bits of each half.  Inputs must be finite.
// One tile in flight per CTA and twelve small CTAs per SM measured faster than fewer CTAs with a ring of tiles each
// (6.0 vs 5.2 TB/s with three stages): the phases of a tile are separated by block-wide barriers, and more
// independent CTAs hide them better than a deeper ring does.
constexpr int kQbThreads = 128;
constexpr int kQbStages = 1;
constexpr int kQbSmem = kQbStages * kTileBytes + 8 * 16 * 16 + 2 * kD * 2;

__device__ __forceinline__ uint32_t qb_chunk(int row, int chunk) {   // byte offset of a 16-byte chunk in a staged tile
    return (uint32_t)(row * 256 + ((chunk ^ ((row & 1) << 1)) << 4));   // (with the read order below: conflict-free)
}

__global__ void __launch_bounds__(kQbThreads) quantize_bulk_kernel(QuantParams p) {
    extern __shared__ __align__(1024) unsigned char qsm[];
    const int b = blockIdx.y, tid = threadIdx.x;
    pdl_launch_dependents();
    pdl_wait();
    int n = p.seq_lens[b];
    const int cap = p.max_blocks * kBlk;
    n = n < 0 ? 0 : (n > cap ? cap : n);
    const int nb = (n + kBlk - 1) / kBlk;
    const int first = p.first_token ? max(p.first_token[b], 0) / kBlk : 0;
    const int count = max(nb - first, 0) * p.Hkv;              // (block, head) tiles of this sequence
    const uint32_t ring = smem_u32(qsm);
    uint4* red = reinterpret_cast<uint4*>(qsm + kQbStages * kTileBytes);          // [8 row groups][16 chunks]
    unsigned short* tq = reinterpret_cast<unsigned short*>(qsm + kQbStages * kTileBytes + 2048);   // upper thresholds
    unsigned short* lq = tq + kD;                                                                  // lower thresholds

    // tile number x of this CTA -> global tile index, or -1 (bad page-table entry: skipped)
    auto tile_of = [&](int x, int& rows) -> long long {
        const int idx = blockIdx.x + x * gridDim.x;
        const int blk = first + idx / p.Hkv, g = idx % p.Hkv;
        rows = min(kBlk, n - blk * kBlk);
        const int page = p.block_table ? p.block_table[(size_t)b * p.max_blocks + blk] : b * p.max_blocks + blk;
        if (page < 0 || page >= p.num_pages) return -1;
        return (long long)page * p.Hkv + g;
    };
    auto issue = [&](int x) {   // start the copy of this CTA's tile x (one commit group, maybe empty)
        if (blockIdx.x + x * gridDim.x < count) {
            int rows;
            const long long tile = tile_of(x, rows);
            if (tile >= 0) {
                const uint4* src = reinterpret_cast<const uint4*>(p.k_cache + tile * kBlk * kD);
                const uint32_t stage = ring + (x % kQbStages) * kTileBytes;
#pragma unroll
                for (int y = 0; y < 8; ++y) {
                    const int q = tid + kQbThreads * y;
                    cp_async16(stage + qb_chunk(q >> 4, q & 15), src + q);
                }
            }
        }
        asm volatile("cp.async.commit_group;\n" ::: "memory");
    };

    for (int x = 0; blockIdx.x + x * gridDim.x < count; ++x) {
        __syncthreads();              // every thread is done with the previous tile
        issue(x);
        asm volatile("cp.async.wait_group 0;\n" ::: "memory");
        __syncthreads();
        int rows;
        const long long tile = tile_of(x, rows);
        if (tile < 0) continue;   // (uniform over the CTA)
        const uint32_t stage = ring + (x % kQbStages) * kTileBytes;
        {   // per-channel maximum of |K| over the valid rows: thread (row group, chunk) takes every 8th row
            const int grp = tid >> 4, cg = tid & 15;
            __nv_bfloat162 acc[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) acc[k] = __floats2bfloat162_rn(0.f, 0.f);
#pragma unroll
            for (int pass = 0; pass < 8; ++pass) {
                const int row = pass * 8 + grp;
                if (row < rows) {
                    const uint4 v = lds128(stage + qb_chunk(row, cg));
                    const uint32_t wds[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        acc[k] = __hmax2(acc[k], __habs2(*reinterpret_cast<const __nv_bfloat162*>(&wds[k])));
                }
            }
            red[grp * 16 + cg] = make_uint4(*reinterpret_cast<uint32_t*>(&acc[0]), *reinterpret_cast<uint32_t*>(&acc[1]),
                                            *reinterpret_cast<uint32_t*>(&acc[2]), *reinterpret_cast<uint32_t*>(&acc[3]));
        }
        __syncthreads();
        {   // thread = channel: the scale (App. A.1) and the two bf16 thresholds that stand for it
            const unsigned short* r16 = reinterpret_cast<const unsigned short*>(red);
            unsigned short m = 0;
#pragma unroll
            for (int grp = 0; grp < 8; ++grp) m = max(m, r16[grp * 128 + tid]);   // non-negative bf16: bit order = value order
            const float a = __uint_as_float((uint32_t)m << 16);
            float s32 = __fdiv_rn(a, 1.5f);
            s32 = fminf(s32, 65504.f);
            const __half s = __float2half_rn(s32);
            p.k_scales[tile * kD + tid] = s;
            const uint32_t sb = __float_as_uint(__half2float(s));
            const unsigned short t = (unsigned short)((sb + 0xFFFFu) >> 16);     // smallest bf16 >= s
            tq[tid] = t;
            lq[tid] = t == 0 ? (unsigned short)0xFF80u : (unsigned short)(t | 0x8000u);   // -t, or -inf for an all-zero channel
        }
        __syncthreads();
        {   // codes: thread (M-tile, r, j) packs tokens 16 mt + r and + 8, channels 32 j .. 32 j + 31
            const int mt = tid >> 5, lane = tid & 31, r = lane >> 2, j = lane & 3;
            const int r0 = 16 * mt + r, r1 = r0 + 8;
            const __nv_bfloat162 zero = __floats2bfloat162_rn(0.f, 0.f);
            const __nv_bfloat162 bias = __floats2bfloat162_rn(128.f, 128.f);
            uint32_t w[4] = {0u, 0u, 0u, 0u};
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {
                // lanes j = 2, 3 take their four chunks one step ahead of lanes j = 0, 1: the chunks 4j + k and
                // 4(j + 2) + k lie 128 bytes apart, i.e. in the same banks
                const int k = (kk + (j >> 1)) & 3;
                const uint4 v0 = lds128(stage + qb_chunk(r0, 4 * j + k));
                const uint4 v1 = lds128(stage + qb_chunk(r1, 4 * j + k));
                const uint4 tv = *reinterpret_cast<const uint4*>(tq + 32 * j + 8 * k);
                const uint4 lv = *reinterpret_cast<const uint4*>(lq + 32 * j + 8 * k);
                const uint32_t x0[4] = {v0.x, v0.y, v0.z, v0.w}, x1[4] = {v1.x, v1.y, v1.z, v1.w};
                const uint32_t th[4] = {tv.x, tv.y, tv.z, tv.w}, tl[4] = {lv.x, lv.y, lv.z, lv.w};
#pragma unroll
                for (int pr = 0; pr < 4; ++pr) {   // channels 8k + 2pr, + 1: i = 2k + pr / 2, u = 2 (pr % 2), + 1
                    const __nv_bfloat162 hi = *reinterpret_cast<const __nv_bfloat162*>(&th[pr]);
                    const __nv_bfloat162 lo = *reinterpret_cast<const __nv_bfloat162*>(&tl[pr]);
                    const int shift = 2 * (2 * k + (pr >> 1));
#pragma unroll
                    for (int rs = 0; rs < 2; ++rs) {
                        const __nv_bfloat162 x = *reinterpret_cast<const __nv_bfloat162*>(rs ? &x1[pr] : &x0[pr]);
                        const __nv_bfloat162 c =
                            __hadd2(__hadd2(__hge2(x, hi), __hge2(x, zero)), __hadd2(__hgt2(x, lo), bias));
                        w[(pr & 1) * 2 + rs] |= (*reinterpret_cast<const uint32_t*>(&c) & 0x00030003u) << shift;
                    }
                }
            }
            reinterpret_cast<uint4*>(p.k_quant + tile * kCodeBytes)[mt * 32 + lane] = make_uint4(w[0], w[1], w[2], w[3]);
        }
    }
    cp_async_drain();
}

// ---- cache append (Sec. 3.3: every step-varying index lives on the device) ---------------------------------
struct AppendParams {
    const __nv_bfloat16* k_new;   // [B, Hkv, 128]
    const __nv_bfloat16* v_new;
    __nv_bfloat16* k_cache;
    __nv_bfloat16* v_cache;
    uint8_t* k_quant;
    __half* k_scales;
    const int32_t* block_table;
    int32_t* seq_lens;
    uint32_t* status;
    int Hkv, max_blocks, num_pages;
    int8_t* k_res;                // nullable: 2 + 8 bit key format, the block's residuals are redone too
};

// One CTA of 128 threads (one per channel) per (KV head, sequence): the new token's K and V rows go to position
// seq_lens[b] of the cache, and the block they fall into is re-quantized over its rows up to and including the new one.
__global__ void __launch_bounds__(128) append_kernel(AppendParams p) {
    const int g = blockIdx.x, b = blockIdx.y, tid = threadIdx.x;
    pdl_launch_dependents();
    pdl_wait();
    const int pos = p.seq_lens[b];
    if (pos < 0 || pos >= p.max_blocks * kBlk) {   // no room (or a corrupt length): reported, nothing written
        if (tid == 0) atomicOr(p.status, kDevBadSeqLen);
        return;
    }
    const int blk = pos / kBlk, row = pos % kBlk;
    const int page = p.block_table ? p.block_table[(size_t)b * p.max_blocks + blk] : b * p.max_blocks + blk;
    if (page < 0 || page >= p.num_pages) {
        if (tid == 0) atomicOr(p.status, kDevBadPage);
        return;
    }
    __shared__ __align__(16) __nv_bfloat16 sk[kBlk * kD];
    __shared__ float ss[kD];
    const size_t tile = (size_t)page * p.Hkv + g;
    const size_t unit = (size_t)b * p.Hkv + g;
    const __nv_bfloat16 kn = p.k_new[unit * kD + tid];
    p.v_cache[(tile * kBlk + row) * kD + tid] = p.v_new[unit * kD + tid];
    p.k_cache[(tile * kBlk + row) * kD + tid] = kn;
    // the rows before the new one (16-byte vectors: 16 per row)
    const uint4* src = reinterpret_cast<const uint4*>(p.k_cache + tile * kBlk * kD);
    uint4* dst = reinterpret_cast<uint4*>(sk);
    for (int x = tid; x < row * (kD / 8); x += 128) dst[x] = src[x];
    sk[row * kD + tid] = kn;
    __syncthreads();
    quantize_tile(sk, ss, row + 1, p.k_scales + tile * kD, p.k_quant + tile * kCodeBytes, tid);
    if (p.k_res) {   // (uniform over the CTA)
        __shared__ float sinv[kD];
        sinv[tid] = __fdiv_rn(254.f, ss[tid]);
        __syncthreads();
        residual_rows(sk, ss, sinv, row + 1, p.k_res + tile * kBlk * kD, tid);
    }
}

// after every CTA of append_kernel has read the lengths: one more token per sequence that had room
__global__ void __launch_bounds__(256) bump_lengths_kernel(int32_t* seq_lens, int batch, int cap) {
    pdl_launch_dependents();
    pdl_wait();
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b < batch) {
        const int n = seq_lens[b];
        if (n >= 0 && n < cap) seq_lens[b] = n + 1;
    }
}

// canonical codes [pages, Hkv, 64, 128] from the packed layout
__global__ void __launch_bounds__(128) unpack_kernel(const uint8_t* k_quant, uint8_t* codes, size_t tiles) {
    const size_t tile = blockIdx.x;
    if (tile >= tiles) return;
    const int tid = threadIdx.x;
    const int mt = tid >> 5, lane = tid & 31, r = lane >> 2, j = lane & 3;
    const uint4 v = reinterpret_cast<const uint4*>(k_quant + tile * kCodeBytes)[mt * 32 + lane];
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    uint8_t* dst = codes + tile * kBlk * kD;
    for (int i = 0; i < 8; ++i)
        for (int u = 0; u < 4; ++u) {
            const int c = 32 * j + 4 * i + u;
            const int shift = 2 * i + 16 * (u & 1);
            dst[(16 * mt + r) * kD + c] = (w[(u >> 1) * 2 + 0] >> shift) & 3u;
            dst[(16 * mt + r + 8) * kD + c] = (w[(u >> 1) * 2 + 1] >> shift) & 3u;
        }
}

constexpr int kPmHintBlocks = 64;
constexpr int kPmWarps = 24;   // one warp per sink / local block in the default configuration (1 + 16), the rest sample
constexpr int kPmSamples = 7;  // blocks sampled between the sink and the local window for the scheduling hint

// ---- pseudo-max (Sec. 3.2; Alg. 1 "Pseudo-max estimation") ------------------------------------------------
// One CTA per (KV head, sequence): its warps scan the sink and local blocks and reduce the block maxima.
// APPEND (ffd_append_decode): the CTA first appends the new token of its (sequence, KV head) as append_kernel does
// — rows written, tail block re-quantized — and works with the new length; new_lens[b] receives that length for
// the kernels that follow (the caller's seq_lens is only read here; the combine kernel updates it at the end).
template <bool APPEND>
__global__ void __launch_bounds__(kPmWarps * 32) pseudomax_kernel(DecodeParams p, AppendParams ap, int32_t* new_lens) {
    const int g = blockIdx.x, b = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // Wait first, then let the fused kernel start: whatever the fused kernel does ahead of its own dependency wait
    // (it draws its first work tickets there) then runs after everything that precedes this kernel has finished,
    // the previous call's reset of the work counters included.
    pdl_wait();
    pdl_launch_dependents();
    int n = clamped_seq_len(p, b);
    int tail_blk = -1;   // APPEND: the block whose thumbnails warps 0..3 of this CTA rewrite (warp 0 scans it)
    if (APPEND) {
        __shared__ __align__(16) __nv_bfloat16 sk[kBlk * kD];
        __shared__ float ss[kD];
        const int tid = threadIdx.x;
        const int pos = n;
        const bool room = pos < p.max_blocks * kBlk;
        if (!room && tid == 0) atomicOr(p.status, kDevBadSeqLen);   // reported, nothing appended
        int page = -1;
        if (room) {
            n = pos + 1;
            page = page_of(p, b, pos / kBlk);   // (reports a bad entry; the rows are then not written)
        }
        if (g == 0 && tid == 0) new_lens[b] = n;
        if (page >= 0) {   // (uniform over the CTA)
            tail_blk = pos / kBlk;
            if (tid < kD) {   // warps 0..3 append and re-quantize while the other warps already scan
                const int row = pos % kBlk;
                const size_t tile = tile_index(p, page, g);
                const size_t unit = (size_t)b * p.Hkv + g;
                const __nv_bfloat16 kn = ap.k_new[unit * kD + tid];
                ap.v_cache[(tile * kBlk + row) * kD + tid] = ap.v_new[unit * kD + tid];
                ap.k_cache[(tile * kBlk + row) * kD + tid] = kn;
                sk[row * kD + tid] = kn;
                const uint4* src = reinterpret_cast<const uint4*>(ap.k_cache + tile * kBlk * kD);
                uint4* dst = reinterpret_cast<uint4*>(sk);
                for (int x = tid; x < row * (kD / 8); x += kD) dst[x] = src[x];
                asm volatile("bar.sync 1, 128;\n" ::: "memory");
                quantize_tile<true>(sk, ss, row + 1, ap.k_scales + tile * kD, ap.k_quant + tile * kCodeBytes, tid);
                __threadfence_block();
                asm volatile("bar.sync 1, 128;\n" ::: "memory");   // warp 0 may now read the new thumbnails
            }
        }
    }
    const int nb = (n + kBlk - 1) / kBlk;
    const int ns = min(p.n_sink, nb);
    const int local_begin = max(nb - p.n_local, ns);
    const int count = ns + (nb - local_begin);
    __shared__ float smax[kPmWarps][kMaxG];
    __shared__ float sbm[kPmHintBlocks][kMaxG];   // block maxima of the first sink / local blocks, for the hint below
    __shared__ float sthr[kMaxG];
    for (int x = threadIdx.x; x < kPmHintBlocks * kMaxG; x += kPmWarps * 32) (&sbm[0][0])[x] = -INFINITY;
    __syncthreads();
    ScanQuery sq;
    const __nv_bfloat16* q_group = p.q + ((size_t)b * p.Hq + (size_t)g * p.G) * kD;
    scan_setup(sq, q_group, p.G, lane, p.sm_scale);
    unsigned char* rec = p.qrec + (size_t)(b * p.Hkv + g) * kQrecBytes;
    if (warp == 0) {   // query record of this (sequence, KV head): the fused kernel stages it per work item
        uint4* dst = reinterpret_cast<uint4*>(rec);
#pragma unroll
        for (int x = 0; x < 4; ++x)
            dst[x * 32 + lane] = make_uint4(sq.qh[4 * x], sq.qh[4 * x + 1], sq.qh[4 * x + 2], sq.qh[4 * x + 3]);
        // |q| in the same fragment layout, with the pre-scaling of the k-steps undone (exact: powers of four)
        uint4* dst_abs = reinterpret_cast<uint4*>(rec + kQrecAbs);
#pragma unroll
        for (int x = 0; x < 4; ++x) {
            uint32_t a[4];
#pragma unroll
            for (int y = 0; y < 4; ++y) {
                const float undo = 1.0f / scan_pos_scale(2 * x + (y >> 1));
                const __half2 v = __hmul2(__habs2(*reinterpret_cast<const __half2*>(&sq.qh[4 * x + y])),
                                          __floats2half2_rn(undo, undo));
                a[y] = *reinterpret_cast<const uint32_t*>(&v);
            }
            dst_abs[x * 32 + lane] = make_uint4(a[0], a[1], a[2], a[3]);
        }
    }
    // Besides the sink and local blocks, a few blocks spread evenly over the middle of the sequence are scanned.
    // They never enter m_tilde: they only tell the scheduler below how dense this unit's selection will be.
    const int middle = local_begin - ns;
    const int nsamp = min(kPmSamples, middle);
    float best = -INFINITY;
    // blocks s = 0 .. count + nsamp - 1 are dealt to the warps round-robin; with a tail block being rewritten
    // (APPEND) warp 0 takes that one (it is s = count - 1, the last local block) after its part in rewriting it,
    // warps 1..3 join once they are done with theirs, and the other warps never touch it
    const bool special = APPEND && tail_blk >= 0;
    const int first_s = special ? (warp == 0 ? count - 1 : warp - 1) : warp;
    const int step_s = special ? kPmWarps - 1 : kPmWarps;
    for (int s0 = first_s; s0 < count + nsamp; s0 += step_s) {
        int s = s0;
        if (special && warp != 0) {          // skip over the tail block's slot
            if (s >= count - 1) ++s;
            if (s >= count + nsamp) break;
        } else if (special && s0 != count - 1) break;   // warp 0: the tail block only
        const bool sample = s >= count;
        const int blk = sample ? ns + (int)(((long long)(2 * (s - count) + 1) * middle) / (2 * nsamp))
                               : (s < ns ? s : local_begin + (s - ns));
        const int page = page_of(p, b, blk);
        if (page < 0) continue;
        const size_t tile = tile_index(p, page, g);
        const int rows = min(kBlk, n - blk * kBlk);
        float band;
        ScanRegs sr;
        if (APPEND && blk == tail_blk)
            scan_load_plain(sr, reinterpret_cast<const uint4*>(p.k_quant + tile * kCodeBytes),
                            reinterpret_cast<const uint4*>(p.k_scales + tile * kD), lane);
        else
            scan_load(sr, reinterpret_cast<const uint4*>(p.k_quant + tile * kCodeBytes),
                      reinterpret_cast<const uint4*>(p.k_scales + tile * kD), lane);
        float bm = scan_compute<true>(sr, sq, lane, rows, band);
        if (bm != bm) {   // (uniform) a scale too large for the fp16 operand: binary32 on the ordinary lanes
            bm = scan_block_wide(reinterpret_cast<const uint4*>(p.k_quant + tile * kCodeBytes), p.k_scales + tile * kD,
                                 q_group, p.G, lane, rows, p.sm_scale, nullptr, 0);
            if (!(fabsf(bm) < INFINITY) && lane < p.G) atomicOr(p.status, kDevRange);
        }
        if (lane < kMaxG && s < kPmHintBlocks) sbm[s][lane] = bm;
        if (!sample) best = fmaxf(best, bm);
    }
    if (lane < kMaxG) smax[warp][lane] = best;
    __syncthreads();
    if (threadIdx.x < 8) {
        // thresholds m_tilde - delta for the scan (delta = +inf gives -inf: every block passes); unused heads: +inf
        float thr = INFINITY;
        if (threadIdx.x < p.G) {
            float m = -INFINITY;
            for (int w = 0; w < kPmWarps; ++w) m = fmaxf(m, smax[w][threadIdx.x]);
            p.mtilde[(size_t)b * p.Hq + g * p.G + threadIdx.x] = m;
            thr = m - p.delta;
        }
        if (threadIdx.x < kMaxG) {   // (lane h of warp 0 holds the unit of head h)
            float* consts = reinterpret_cast<float*>(rec + kQrecThr);
            const float bmul = 1.5f * 1.02f * sq.unit * (1.0f / 1048576.0f);
            consts[threadIdx.x] = thr;
            consts[4 + threadIdx.x] = sq.unit;
            consts[8 + threadIdx.x] = bmul;
            consts[12 + threadIdx.x] = 1e-3f + bmul * (1.0f / 131072.0f);
            sthr[threadIdx.x] = thr;
        }
    }
    __syncthreads();
    // Scheduling hint for the fused kernel: a (sequence, KV head) that keeps at least half of the sampled middle
    // blocks (of its sink / local blocks, when the sequence has no middle) is a "dense" unit: its work items are
    // expensive for the attend warps and are handed out first.  The hint only orders the work; it never changes a
    // result.
    int h_begin = 0, hinted = min(count, kPmHintBlocks);
    if (nsamp > 0 && count + nsamp <= kPmHintBlocks) { h_begin = count; hinted = nsamp; }
    bool kept_any = false;
    if ((int)threadIdx.x < hinted)
        for (int h = 0; h < p.G; ++h) kept_any |= sbm[h_begin + threadIdx.x][h] >= sthr[h];
    const int kept = __syncthreads_count(kept_any);
    if (threadIdx.x == 0) {
        const int bg = b * p.Hkv + g;
        // the longest and the shortest sequence of the batch, for the fused kernel's draw plan
        atomicMax(&p.len_stats[0], (unsigned)nb);
        atomicMax(&p.len_stats[1], (unsigned)(p.max_blocks - nb));
        atomicAdd(&p.len_stats[2], (unsigned)item_count(p, nb));   // work items that exist
        // The list is filled from both ends with counters that every completed call leaves at zero.  A header that was
        // never initialised, or counters left behind by an interrupted call, must not become store indices.
        if (p.status[kHeaderCookieWord] != kHeaderCookie) {
            atomicOr(p.status, kDevBadWorkspace);
        } else {
            const bool heavy = hinted > 0 && 2 * kept >= hinted;
            const unsigned idx = atomicAdd(&p.class_counts[heavy ? 0 : 1], 1u);
            if (idx < (unsigned)p.units) p.unit_list[heavy ? (int)idx : p.units - 1 - (int)idx] = make_int2(bg, n);
            else atomicOr(p.status, kDevBadWorkspace);
        }
    }
}

// ---- dense decode attention over one split of one (sequence, KV head) (Sec. 4.2 baseline) ------------------
struct BlockRef {
    int blk;        // logical block, -1 = none
    int rows;       // valid tokens
    size_t tile;    // (page, KV head) tile index
};

__global__ void __launch_bounds__(kWarps * 32, 1) dense_kernel(DecodeParams p) {
    extern __shared__ __align__(1024) unsigned char smem[];
    const int split = blockIdx.x, g = blockIdx.y, b = blockIdx.z;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int r = lane >> 2, j = lane & 3;
    pdl_launch_dependents();
    pdl_wait();
    const int n = clamped_seq_len(p, b);
    const int nb = (n + kBlk - 1) / kBlk;
    const int blk_begin = split * p.blocks_per_split;
    const int blk_end = min(nb, blk_begin + p.blocks_per_split);

    __shared__ int next_blk;
    __shared__ float sm_m[kWarps][kMaxG], sm_l[kWarps][kMaxG];
    const uint32_t kslot = smem_u32(smem) + warp * 2 * kSlotBytes;
    const uint32_t vslot = kslot + kSlotBytes;
    const uint32_t kbar = smem_u32(smem) + kWarps * 2 * kSlotBytes + warp * 16;
    const uint32_t vbar = kbar + 8;
    if (threadIdx.x == 0) next_blk = blk_begin;
    if (lane == 0) {
        mbar_init(kbar, 32);
        mbar_init(vbar, 32);
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    __syncthreads();

    const __nv_bfloat16* q_group = p.q + ((size_t)b * p.Hq + (size_t)g * p.G) * kD;
    const size_t head0 = (size_t)b * p.Hq + (size_t)g * p.G;
    AttendState st;
    attend_setup(st, q_group, p.G, lane);
    const unsigned group_mask = (1u << p.G) - 1u;
    const float logit_scale_log2 = p.sm_scale * kLog2e;
    const uint4* kbase = reinterpret_cast<const uint4*>(p.k_cache);
    const uint4* vbase = reinterpret_cast<const uint4*>(p.v_cache);
    constexpr size_t kTileVec = kTileBytes / 16;

    // next block of this split for this warp (skipping blocks whose page index is bad)
    auto fetch = [&]() {
        BlockRef ref{-1, 0, 0};
        for (;;) {
            int blk = 0;
            if (lane == 0) blk = atomicAdd(&next_blk, 1);
            blk = __shfl_sync(kFull, blk, 0);
            if (blk >= blk_end) return ref;
            const int page = page_of(p, b, blk);
            if (page < 0) continue;
            ref.blk = blk;
            ref.rows = min(kBlk, n - blk * kBlk);
            ref.tile = tile_index(p, page, g);
            return ref;
        }
    };

    BlockRef cur = fetch();
    BlockRef pending{-1, 0, 0};     // block whose K/V copies are in flight
    uint32_t phase = 0;
    bool ok = true;
    while (cur.blk >= 0 && ok) {
        const BlockRef nxt = fetch();
        const uint4* ksrc = kbase + cur.tile * kTileVec;
        const uint4* vsrc = vbase + cur.tile * kTileVec;
        if (pending.blk >= 0) {
            ok = attend_block(st, kslot, vslot, kbar, vbar, phase, ksrc, vsrc, lane, pending.rows, group_mask,
                              logit_scale_log2);
        } else {
            tile_copy_async(kslot, ksrc, lane, kbar);
            tile_copy_async(vslot, vsrc, lane, vbar);
        }
        pending = cur;
        cur = nxt;
    }
    if (ok && pending.blk >= 0)
        ok = attend_block(st, kslot, vslot, kbar, vbar, phase, nullptr, nullptr, lane, pending.rows, group_mask,
                          logit_scale_log2);
    cp_async_drain();
    if (!ok && lane == 0) atomicOr(p.status, kDevTimeout);

    // fold the warp's state: row sums over the 4 lanes of a row, bf16 remainder rows onto the main rows
    float l = st.l;
    l += __shfl_xor_sync(kFull, l, 1);
    l += __shfl_xor_sync(kFull, l, 2);
#pragma unroll
    for (int nt = 0; nt < 16; ++nt) {
        st.acc[nt][0] += __shfl_xor_sync(kFull, st.acc[nt][0], 16);
        st.acc[nt][1] += __shfl_xor_sync(kFull, st.acc[nt][1], 16);
    }
    // the warp's own K slot is free now: it holds the warp's [4][128] accumulators for the merge
    float* my_acc = reinterpret_cast<float*>(smem + (size_t)warp * 2 * kSlotBytes);
    if (r < kMaxG) {
        if (j == 0) { sm_m[warp][r] = st.m; sm_l[warp][r] = l; }
#pragma unroll
        for (int nt = 0; nt < 16; ++nt) {
            my_acc[r * kD + attend_channel(nt, 2 * j)] = st.acc[nt][0];
            my_acc[r * kD + attend_channel(nt, 2 * j + 1)] = st.acc[nt][1];
        }
    }
    __syncthreads();
    // merge the warps; each work item is one head and a pair of channels
    for (int item = threadIdx.x; item < p.G * (kD / 2); item += kWarps * 32) {
        const int h = item / (kD / 2), c = (item % (kD / 2)) * 2;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) M = fmaxf(M, sm_m[w][h]);
        float L = 0.f, a0 = 0.f, a1 = 0.f;
        if (M != -INFINITY) {
#pragma unroll
            for (int w = 0; w < kWarps; ++w) {
                const float f = exp2f(sm_m[w][h] - M);
                const float* wacc = reinterpret_cast<const float*>(smem + (size_t)w * 2 * kSlotBytes) + h * kD + c;
                L += f * sm_l[w][h];
                a0 += f * wacc[0];
                a1 += f * wacc[1];
            }
        }
        const size_t slot = (head0 + h) * p.splits + split;
        if (c == 0) { p.part_ml[2 * slot] = M; p.part_ml[2 * slot + 1] = L; }
        *reinterpret_cast<float2*>(p.part_acc + slot * kD + c) = make_float2(a0, a1);
    }
}

// precise scan of one block straight from global memory, out of line (the rare re-check of a block whose fast result
// is too close to the threshold): its registers must not weigh on the caller's hot loop
__device__ __noinline__ float scan_precise_from_global(const uint4* codes_tile, const uint4* scales_tile,
                                                       const __nv_bfloat16* q_group, int G, int lane, int rows,
                                                       float sm_scale) {
    ScanQuery sq;
    scan_setup(sq, q_group, G, lane, sm_scale);
    ScanRegs sr;
    scan_load(sr, codes_tile, scales_tile, lane);
    float band;
    float bm = scan_compute<true>(sr, sq, lane, rows, band);
    if (bm != bm)   // (a scale too large for the fp16 operand)
        bm = scan_block_wide(codes_tile, reinterpret_cast<const __half*>(scales_tile), q_group, G, lane, rows, sm_scale, nullptr, 0);
    return bm;
}

// ---- scan, select and decode as three kernels -----------------------------------------------------------------
// The path of the 4- and 8-bit thumbnails on large geometries and of the comparison selection rules (ffd_decode_select):
//   scan_blocks_kernel   block maxima of the approximate logits of every block (Alg. 1 "Top-delta selection", the scores)
//   select_kernel        the rule: which blocks each head keeps
//   small_sparse_kernel<0>  exact attention over the kept blocks and the merge of the splits
// Scan: one warp per block, many warps per SM; the codes of a long cache stream through, which the decode kernel's seven
// fat warps per SM cannot do for codes this wide.  Writes p.bmax[b][head][block] (precise accumulation, the arithmetic
// of m_tilde); NaN for a block whose page index is bad (never kept, ignored by every maximum).
constexpr int kScanCtaBlocks = 64;   // blocks of one (sequence, KV head) per CTA: 8 per warp
template <int BITS>
__global__ void __launch_bounds__(256, 2) scan_blocks_kernel(DecodeParams p) {
    const int g = blockIdx.y, b = blockIdx.z;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int r = lane >> 2, j = lane & 3;
    pdl_launch_dependents();
    pdl_wait();
    const int n = clamped_seq_len(p, b);
    const int nb = (n + kBlk - 1) / kBlk;
    const int first = blockIdx.x * kScanCtaBlocks;
    if (first >= nb) return;
    const int last = min(nb, first + kScanCtaBlocks);
    const __nv_bfloat16* q_group = p.q + ((size_t)b * p.Hq + (size_t)g * p.G) * kD;
    float* out = p.bmax + ((size_t)b * p.Hq + (size_t)g * p.G) * p.max_blocks;
    auto raw_page = [&](int blk) {
        return p.block_table ? p.block_table[(size_t)b * p.max_blocks + blk] : b * p.max_blocks + blk;
    };
    auto prefetch = [&](int page) {
        if (page >= 0 && page < p.num_pages) {
            const size_t tile = tile_index(p, page, g);
            wide_prefetch_l2<BITS>(p.k_quant + tile * WideScan<BITS>::kTileBytes, p.k_scales + tile * kD, lane);
        }
    };
    if constexpr (BITS == 2) {
        // 2-bit thumbnails: the next block's codes and scales wait in registers while the current block is scored
        ScanQuery sq;
        scan_setup(sq, q_group, p.G, lane, p.sm_scale);
        auto tile_of = [&](int blk) -> long long {
            if (blk >= last) return -1;
            const int page = page_of(p, b, blk);
            return page < 0 ? -1 : (long long)tile_index(p, page, g);
        };
        auto load = [&](ScanRegs& sr, long long tile) {
            if (tile >= 0)
                scan_load(sr, reinterpret_cast<const uint4*>(p.k_quant + (size_t)tile * kCodeBytes),
                          reinterpret_cast<const uint4*>(p.k_scales + (size_t)tile * kD), lane);
        };
        int blk = first + warp;
        long long tile = tile_of(blk);
        ScanRegs cur;
        load(cur, tile);
        for (; blk < last; blk += 8) {
            const long long next_tile = tile_of(blk + 8);
            ScanRegs nxt;
            load(nxt, next_tile);
            float bm = __int_as_float(0x7fc00000);
            if (tile >= 0) {
                const int rows = min(kBlk, n - blk * kBlk);
                float band;
                bm = scan_compute<true>(cur, sq, lane, rows, band);
                if (bm != bm) {   // the fp16 operand overflowed: binary32 on the ordinary lanes
                    bm = scan_block_wide(reinterpret_cast<const uint4*>(p.k_quant + (size_t)tile * kCodeBytes),
                                         p.k_scales + (size_t)tile * kD, q_group, p.G, lane, rows, p.sm_scale, nullptr, 0);
                    if (!(fabsf(bm) < INFINITY)) {
                        if (j < p.G) atomicOr(p.status, kDevRange);
                        bm = INFINITY;
                    }
                }
            }
            if (r == 0 && j < p.G) out[(size_t)j * p.max_blocks + blk] = bm;
            tile = next_tile;
            cur = nxt;
        }
        return;
    }
    // the warp's first two tiles are on their way while it prepares its query fragments
    int blk = first + warp;
    int page = blk < last ? raw_page(blk) : -1;
    int next_page = blk + 8 < last ? raw_page(blk + 8) : -1;
    prefetch(page);
    prefetch(next_page);
    ScanQuery sq;
    scan_setup_wide(sq, q_group, p.G, lane, p.sm_scale);
    for (; blk < last; blk += 8) {
        const int after = blk + 16 < last ? raw_page(blk + 16) : -1;   // (read now, used for the hint one turn later)
        float bm = __int_as_float(0x7fc00000);
        if (page >= 0 && page < p.num_pages) {
            const size_t tile = tile_index(p, page, g);
            float band;
            bm = scan_wide<BITS, true>(p.k_quant + tile * WideScan<BITS>::kTileBytes, p.k_scales + tile * kD, sq, lane,
                                       min(kBlk, n - blk * kBlk), band);
            if (bm != bm) {   // scales beyond the fp16 operand's range: reported, the block kept
                if (j < p.G) atomicOr(p.status, kDevRange);
                bm = INFINITY;
            }
        } else if (lane == 0) {
            atomicOr(p.status, kDevBadPage);
        }
        if (r == 0 && j < p.G) out[(size_t)j * p.max_blocks + blk] = bm;
        page = next_page;
        next_page = after;
        prefetch(after);
    }
}

// ---- select: the rule that turns block maxima into decisions ----------------------------------------------------
// One CTA per (sequence, query head).  Rules (ffd.h FFD_RULE_*):
//   0 pseudo-max     keep = bm >= m_tilde - delta, m_tilde over the sink and local blocks (Alg. 1, Eq. 1)
//   1 global max     keep = bm >= max over all blocks - delta (the comparison rule of Sec. 5.2: a reduction of its own)
//   2 running max    keep = bm >= max(m_tilde, bm of blocks 0 .. blk) - delta: what a streaming scan in logical block
//                    order knows when it meets the block
//   3 top-k          keep = bm >= the k-th largest block maximum (Fig. 1a's fixed budget; ties kept): a radix select,
//                    four passes over the head's maxima
// Writes keep_bits (one byte per (block, head of the group), the bytes of a block side by side), m_tilde, and the
// kept_mask / block_max outputs.
constexpr int kSelectThreads = 256;
enum : int { kRulePseudoMax = 0, kRuleGlobalMax = 1, kRuleRunningMax = 2, kRuleTopK = 3 };

__device__ __forceinline__ uint32_t select_key(float x) {   // order-preserving: larger float <-> larger key
    const uint32_t u = __float_as_uint(x);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float select_unkey(uint32_t k) {
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

__global__ void __launch_bounds__(kSelectThreads) select_kernel(DecodeParams p, int rule, int top_k) {
    const int head = blockIdx.x, b = blockIdx.y;
    const int g = head / p.G, h = head % p.G;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    pdl_launch_dependents();
    pdl_wait();
    const int n = clamped_seq_len(p, b);
    const int nb = (n + kBlk - 1) / kBlk;
    const size_t head0 = (size_t)b * p.Hq + (size_t)g * p.G;
    uint8_t* bits = p.keep_bits + ((size_t)b * p.Hkv + g) * p.max_blocks * kMaxG + h;
    __shared__ float red_a[kSelectThreads / 32], red_b[kSelectThreads / 32];
    __shared__ unsigned hist[256];
    __shared__ unsigned sel_prefix, sel_remaining, sel_valid;
    const int ns = min(p.n_sink, nb);
    const int local_begin = max(nb - p.n_local, ns);
    {
        const float* v = p.bmax + (head0 + h) * p.max_blocks;
        // m_tilde and the global maximum (NaN = bad page: fmaxf passes it over)
        float mt = -INFINITY, gm = -INFINITY;
        unsigned valid = 0;
#pragma unroll 4
        for (int blk = tid; blk < nb; blk += kSelectThreads) {
            const float x = v[blk];
            gm = fmaxf(gm, x);
            if (blk < ns || blk >= local_begin) mt = fmaxf(mt, x);
            valid += x == x;
        }
#pragma unroll
        for (int o = 16; o; o >>= 1) {
            mt = fmaxf(mt, __shfl_xor_sync(kFull, mt, o));
            gm = fmaxf(gm, __shfl_xor_sync(kFull, gm, o));
            valid += __shfl_xor_sync(kFull, valid, o);
        }
        if (lane == 0) { red_a[warp] = mt; red_b[warp] = gm; }
        if (tid == 0) sel_valid = 0;
        __syncthreads();
        if (lane == 0) atomicAdd(&sel_valid, valid);
#pragma unroll
        for (int w = 0; w < kSelectThreads / 32; ++w) { mt = fmaxf(mt, red_a[w]); gm = fmaxf(gm, red_b[w]); }
        if (tid == 0) p.mtilde[head0 + h] = mt;
        float thr = (rule == kRuleGlobalMax ? gm : mt) - p.delta;   // delta = +inf: -inf, everything finite passes
        if (rule == kRuleTopK) {
            __syncthreads();
            thr = -INFINITY;
            if ((unsigned)top_k < sel_valid) {   // radix select of the k-th largest key, eight bits at a time
                if (tid == 0) { sel_prefix = 0; sel_remaining = (unsigned)top_k; }
                for (int shift = 24; shift >= 0; shift -= 8) {
                    hist[tid] = 0;   // (kSelectThreads == 256 bins)
                    __syncthreads();
                    const unsigned prefix = sel_prefix;
                    const unsigned high = shift == 24 ? 0u : 0xffffffffu << (shift + 8);
                    for (int blk = tid; blk < nb; blk += kSelectThreads) {
                        const float x = v[blk];
                        if (x == x) {
                            const uint32_t key = select_key(x);
                            if ((key & high) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1u);
                        }
                    }
                    __syncthreads();
                    if (warp == 0) {   // lane L owns bins 8 L .. 8 L + 7; the k-th largest is counted from the top bin down
                        unsigned c[8], mine = 0;
#pragma unroll
                        for (int i = 0; i < 8; ++i) { c[i] = hist[8 * lane + i]; mine += c[i]; }
                        unsigned incl = mine;   // keys in this lane's bins and in all higher ones
#pragma unroll
                        for (int o = 1; o < 32; o <<= 1) {
                            const unsigned y = __shfl_down_sync(kFull, incl, o);
                            if (lane + o < 32) incl += y;
                        }
                        const unsigned above = incl - mine, left = sel_remaining;
                        __syncwarp();
                        if (above < left && left <= incl) {   // exactly one lane
                            unsigned l = left - above;
                            int i = 7;
                            for (; i > 0 && c[i] < l; --i) l -= c[i];
                            sel_prefix = prefix | ((unsigned)(8 * lane + i) << shift);
                            sel_remaining = l;
                        }
                    }
                    __syncthreads();
                }
                thr = select_unkey(sel_prefix);
            }
        }
        float carry = mt;   // rule 2: the reference before the current chunk
        for (int base = 0; base < nb; base += kSelectThreads) {
            const int blk = base + tid;
            const float x = blk < nb ? v[blk] : __int_as_float(0x7fc00000);
            float t = thr;
            if (rule == kRuleRunningMax) {
                float run = x == x ? x : -INFINITY;   // inclusive prefix maximum over the chunk
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const float y = __shfl_up_sync(kFull, run, o);
                    if (lane >= o) run = fmaxf(run, y);
                }
                __syncthreads();
                if (lane == 31) red_a[warp] = run;
                __syncthreads();
                float before = carry, total = carry;
#pragma unroll
                for (int w = 0; w < kSelectThreads / 32; ++w) {
                    if (w < warp) before = fmaxf(before, red_a[w]);
                    total = fmaxf(total, red_a[w]);
                }
                t = fmaxf(before, run) - p.delta;
                carry = total;
            }
            if (blk < nb) {
                const bool keep = x >= t;   // (NaN never passes)
                bits[(size_t)blk * kMaxG] = keep ? 1 : 0;
                const size_t o = (head0 + h) * p.max_blocks + blk;
                if (p.kept_mask) p.kept_mask[o] = keep ? 1 : 0;
                if (p.block_max) p.block_max[o] = x;
            }
        }
    }
}

// the deeper scans' precise pass, out of line: it runs for the sink and local blocks and for the rare block within
// the fast pass's error band of the threshold, and inlining it twice costs the decode loop its registers
template <int BITS>
__device__ __noinline__ float scan_wide_precise(const unsigned char* codes_tile, const __half* scales_tile, const ScanQuery& sq,
                                                int lane, int rows) {
    float band;
    return scan_wide<BITS, true>(codes_tile, scales_tile, sq, lane, rows, band);
}

// ---- the whole sparse step in one launch, for launches with little work -----------------------------------------
// With fewer than two 32-block work items per SM the persistent kernel and its two companions (pseudo-max before,
// combine after) are three dependent launches of a few microseconds each around almost no work.  This kernel does the
// step in one: a CTA per (split of the sequence, KV head, sequence), the grid of the dense kernel.  Every CTA first
// scans the unit's sink and local blocks itself (precise arithmetic, the blocks come from the L2 after the first CTA)
// and so has m_tilde without waiting for anybody (Sec. 3.2, Alg. 1 "Pseudo-max estimation"); then its warps take the
// blocks of its split one by one: scan, top-delta test (Eq. 1), exact attention over the kept ones through the same
// staged pipeline as the dense kernel (Alg. 1 "Fine-grained refinement").  The CTA's partial goes to the workspace; the
// CTA that finds itself the last of its unit to arrive (a counter in the workspace, left at zero again) merges the
// unit's partials (log-sum-exp) and writes the output.  No CTA waits for another.
template <int BITS>
__global__ void __launch_bounds__(kWarps * 32, 1) small_sparse_kernel(DecodeParams p, uint32_t* arrive) {
    extern __shared__ __align__(1024) unsigned char smem[];
    const int split = blockIdx.x, g = blockIdx.y, b = blockIdx.z;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int r = lane >> 2, j = lane & 3;
    pdl_launch_dependents();
    pdl_wait();
    // the query fragments first: their loads fly while the sequence length (which everything else hangs on) arrives
    const __nv_bfloat16* q_group = p.q + ((size_t)b * p.Hq + (size_t)g * p.G) * kD;
    ScanQuery sq;
    if constexpr (BITS == 2) scan_setup(sq, q_group, p.G, lane, p.sm_scale);
    else if constexpr (BITS != 0) scan_setup_wide(sq, q_group, p.G, lane, p.sm_scale);
    const int n = clamped_seq_len(p, b);
    const int nb = (n + kBlk - 1) / kBlk;
    const int blk_begin = split * p.blocks_per_split;
    const int blk_end = min(nb, blk_begin + p.blocks_per_split);

    __shared__ int is_last;
    __shared__ float sm_m[kWarps][kMaxG], sm_l[kWarps][kMaxG];
    __shared__ float smax[kWarps][kMaxG];
    const uint32_t kslot = smem_u32(smem) + warp * 2 * kSlotBytes;
    const uint32_t vslot = kslot + kSlotBytes;
    const uint32_t kbar = smem_u32(smem) + kWarps * 2 * kSlotBytes + warp * 16;
    const uint32_t vbar = kbar + 8;
    if (lane == 0) {
        mbar_init(kbar, 32);
        mbar_init(vbar, 32);
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    const size_t head0 = (size_t)b * p.Hq + (size_t)g * p.G;
    AttendState st;
    bool ok = true;
    if (blk_begin >= nb) attend_reset(st);
    if (blk_begin < nb) {   // (uniform over the CTA; a split past the sequence's end only reports an empty partial)
        constexpr size_t kCodeTile = BITS == 2 ? (size_t)kCodeBytes : (size_t)WideScan<BITS>::kTileBytes;
        // BITS == 0: the decisions come from the select kernel that ran before this one (p.keep_bits)
        // scan of one block, precise or fast.  2 bits: from the codes in registers, with the binary32 fallback when the
        // fp16 operand overflowed; deeper thumbnails: straight from global memory (an overflow there -- scales beyond
        // 30000 -- is reported and the block kept)
        auto judge = [&](bool precise, const ScanRegs& sr, size_t tile, int rows, float& band) {
            float bm = 0.f;
            if constexpr (BITS == 0) {
                band = 0.f;
                return bm;
            } else if constexpr (BITS == 2) {
                bm = precise ? scan_compute<true>(sr, sq, lane, rows, band) : scan_compute<false>(sr, sq, lane, rows, band);
            } else {
                band = 0.f;
                bm = precise ? scan_wide_precise<BITS>(p.k_quant + tile * kCodeTile, p.k_scales + tile * kD, sq, lane, rows)
                             : scan_wide<BITS, false>(p.k_quant + tile * kCodeTile, p.k_scales + tile * kD, sq, lane, rows, band);
                if (bm != bm) {
                    band = 0.f;
                    if (j < p.G) atomicOr(p.status, kDevRange);
                    bm = INFINITY;
                }
                return bm;
            }
            if (bm != bm) {
                bm = scan_block_wide(reinterpret_cast<const uint4*>(p.k_quant + tile * kCodeBytes), p.k_scales + tile * kD,
                                     q_group, p.G, lane, rows, p.sm_scale, nullptr, 0);
                band = 0.f;
                if (!(fabsf(bm) < INFINITY) && j < p.G) { atomicOr(p.status, kDevRange); bm = INFINITY; }   // reported, kept
            }
            return bm;
        };
        // deeper thumbnails: no codes wait in registers; instead every warp asks L2 for the tiles of its blocks two
        // turns ahead (a hint: a bad page index is simply not prefetched; the scan itself reports it)
        auto raw_page = [&](int blk) {
            return p.block_table ? p.block_table[(size_t)b * p.max_blocks + blk] : b * p.max_blocks + blk;
        };
        auto prefetch_page = [&](int page) {
            if (page >= 0 && page < p.num_pages) {
                const size_t tile = tile_index(p, page, g);
                wide_prefetch_l2<BITS>(p.k_quant + tile * kCodeTile, p.k_scales + tile * kD, lane);
            }
        };
        auto prefetch_block = [&](int blk) {
            if (blk < blk_end) prefetch_page(raw_page(blk));
        };
        {   // m_tilde over the sink and local blocks: warp w takes every kWarps-th of them, the next one's codes on their
            // way into registers while the current one is scanned
            const int ns = min(p.n_sink, nb);
            const int local_begin = max(nb - p.n_local, ns);
            const int count = ns + (nb - local_begin);
            auto ref_of = [&](int s) {
                BlockRef ref{-1, 0, 0};
                if (s < count) {
                    const int blk = s < ns ? s : local_begin + (s - ns);
                    const int page = page_of(p, b, blk);
                    if (page >= 0) { ref.blk = blk; ref.rows = min(kBlk, n - blk * kBlk); ref.tile = tile_index(p, page, g); }
                }
                return ref;
            };
            float best = -INFINITY;
            BlockRef cur = ref_of(BITS == 0 ? count : warp);
            if constexpr (BITS != 2 && BITS != 0) {   // this warp's sink / local blocks on their way into L2 before the first is scanned
                for (int s = warp; s < count; s += kWarps) {
                    const BlockRef ref = ref_of(s);
                    if (ref.blk >= 0) wide_prefetch_l2<BITS>(p.k_quant + ref.tile * kCodeTile, p.k_scales + ref.tile * kD, lane);
                }
                prefetch_block(blk_begin + warp);
                prefetch_block(blk_begin + warp + kWarps);
            }
            ScanRegs cur_regs;
            if (BITS == 2 && cur.blk >= 0)
                scan_load(cur_regs, reinterpret_cast<const uint4*>(p.k_quant + cur.tile * kCodeBytes),
                          reinterpret_cast<const uint4*>(p.k_scales + cur.tile * kD), lane);
            for (int s = BITS == 0 ? count : warp; s < count; s += kWarps) {
                const BlockRef nxt = ref_of(s + kWarps);
                ScanRegs nxt_regs;
                if (BITS == 2 && nxt.blk >= 0)
                    scan_load(nxt_regs, reinterpret_cast<const uint4*>(p.k_quant + nxt.tile * kCodeBytes),
                              reinterpret_cast<const uint4*>(p.k_scales + nxt.tile * kD), lane);
                float band;
                if (cur.blk >= 0) best = fmaxf(best, judge(true, cur_regs, cur.tile, cur.rows, band));
                cur = nxt;
                cur_regs = nxt_regs;
            }
            if (lane < kMaxG) smax[warp][lane] = best;
        }
        __syncthreads();
        float thr = INFINITY;   // of head lane % 4
        if (j < p.G) {
            float m = -INFINITY;
#pragma unroll
            for (int w = 0; w < kWarps; ++w) m = fmaxf(m, smax[w][j]);
            thr = m - p.delta;   // delta = +inf -> -inf: everything passes
            if (BITS != 0 && split == 0 && warp == 0 && r == 0) p.mtilde[head0 + j] = m;
        }
        attend_reset(st);
        attend_load_q(st.qa, q_group, p.G, lane);
        const float logit_scale_log2 = p.sm_scale * kLog2e;
        const uint4* kbase = reinterpret_cast<const uint4*>(p.k_cache);
        const uint4* vbase = reinterpret_cast<const uint4*>(p.v_cache);
        constexpr size_t kTileVec = kTileBytes / 16;
        // next block of this split for this warp: blocks blk_begin + warp, + kWarps, ... (a fixed assignment, so that
        // the order of the sums does not change from run to run), skipping blocks whose page index is bad
        int my_next = blk_begin + warp;
        auto fetch = [&]() {
            BlockRef ref{-1, 0, 0};
            for (;;) {
                const int blk = my_next;
                my_next += kWarps;
                if (blk >= blk_end) return ref;
                const int page = page_of(p, b, blk);
                if (page < 0) continue;
                ref.blk = blk;
                ref.rows = min(kBlk, n - blk * kBlk);
                ref.tile = tile_index(p, page, g);
                return ref;
            }
        };
        auto load_codes = [&](ScanRegs& sr, const BlockRef& ref) {
            if constexpr (BITS == 2)
                scan_load(sr, reinterpret_cast<const uint4*>(p.k_quant + ref.tile * kCodeBytes),
                          reinterpret_cast<const uint4*>(p.k_scales + ref.tile * kD), lane);
        };
        BlockRef pending{-1, 0, 0};     // kept block whose K/V copies are in flight
        unsigned pending_keep = 0;
        uint32_t phase = 0;
        // a kept block: its K/V copies start now; the block kept before it is attended while they fly
        auto consume = [&](const BlockRef& blk_ref, unsigned keep4) {
            const uint4* ksrc = kbase + blk_ref.tile * kTileVec;
            const uint4* vsrc = vbase + blk_ref.tile * kTileVec;
            if (pending.blk >= 0) {
                ok = attend_block(st, kslot, vslot, kbar, vbar, phase, ksrc, vsrc, lane, pending.rows, pending_keep,
                                  logit_scale_log2);
            } else {
                tile_copy_async(kslot, ksrc, lane, kbar);
                tile_copy_async(vslot, vsrc, lane, vbar);
            }
            pending = blk_ref;
            pending_keep = keep4;
        };
        if constexpr (BITS == 0) {
            // The select kernel's decisions, 32 of the warp's blocks at a time (lane L looks at the L-th of them); only the
            // kept ones cost a page lookup and a turn of the pipeline.
            static_assert(kMaxG == 4, "one 32-bit word of decision bytes per block");
            const uint32_t* bits = reinterpret_cast<const uint32_t*>(p.keep_bits) + ((size_t)b * p.Hkv + g) * p.max_blocks;
            const uint32_t group_mask = p.G >= 4 ? 0x01010101u : (1u << (8 * p.G)) - 1u & 0x01010101u;   // (bytes of absent heads are never written)
            for (int base = blk_begin + warp; base < blk_end && ok; base += 32 * kWarps) {
                const int mine = base + lane * kWarps;
                const uint32_t word = mine < blk_end ? bits[mine] & group_mask : 0u;
                const unsigned k4 = (word & 1u) | ((word >> 7) & 2u) | ((word >> 14) & 4u) | ((word >> 21) & 8u);
                unsigned any = __ballot_sync(kFull, k4 != 0);
                while (any && ok) {
                    const int src = __ffs(any) - 1;
                    any &= any - 1;
                    const unsigned keep4 = __shfl_sync(kFull, k4, src);
                    const int blk = base + src * kWarps;
                    const int page = page_of(p, b, blk);
                    if (page < 0) continue;
                    consume(BlockRef{blk, min(kBlk, n - blk * kBlk), tile_index(p, page, g)}, keep4);
                }
            }
        }
        BlockRef cur = fetch();
        if (BITS == 0) cur.blk = -1;
        ScanRegs cur_regs;
        if (cur.blk >= 0) load_codes(cur_regs, cur);
        int pf_blk = blk_begin + warp + 2 * kWarps, pf_page = -1;   // (the page index is read one turn before its use)
        if (BITS != 2 && BITS != 0 && pf_blk < blk_end) pf_page = raw_page(pf_blk);
        while (cur.blk >= 0 && ok) {
            if constexpr (BITS != 2) {
                prefetch_page(pf_page);
                pf_blk += kWarps;
                pf_page = pf_blk < blk_end ? raw_page(pf_blk) : -1;
            }
            // the next block's codes on their way into registers before this one is judged
            const BlockRef nxt = fetch();
            ScanRegs nxt_regs;
            if (nxt.blk >= 0) load_codes(nxt_regs, nxt);
            float band;
            float bm = judge(false, cur_regs, cur.tile, cur.rows, band);
            // too close to call with the fast accumulation: redo the block with the arithmetic m_tilde used
            if (__any_sync(kFull, (j < p.G) && fabsf(bm - thr) <= band)) {
                if constexpr (BITS == 2)
                    bm = scan_precise_from_global(reinterpret_cast<const uint4*>(p.k_quant + cur.tile * kCodeBytes),
                                                  reinterpret_cast<const uint4*>(p.k_scales + cur.tile * kD), q_group, p.G, lane,
                                                  cur.rows, p.sm_scale);
                else
                    bm = judge(true, cur_regs, cur.tile, cur.rows, band);
            }
            const bool keep = (j < p.G) && (bm >= thr);
            const unsigned keep4 = __ballot_sync(kFull, keep) & 0xFu;
            if (r == 0 && j < p.G) {
                const size_t o = (head0 + j) * p.max_blocks + cur.blk;
                if (p.kept_mask) p.kept_mask[o] = keep ? 1 : 0;
                if (p.block_max) p.block_max[o] = bm;
            }
            if (keep4) consume(cur, keep4);
            cur = nxt;
            cur_regs = nxt_regs;
        }
        if (ok && pending.blk >= 0)
            ok = attend_block(st, kslot, vslot, kbar, vbar, phase, nullptr, nullptr, lane, pending.rows, pending_keep,
                              logit_scale_log2);
        cp_async_drain();
        if (!ok && lane == 0) atomicOr(p.status, kDevTimeout);
    } else {
        __syncthreads();   // (the barrier the other branch passes)
    }

    // fold the warp's state: row sums over the 4 lanes of a row, bf16 remainder rows onto the main rows
    float l = st.l;
    l += __shfl_xor_sync(kFull, l, 1);
    l += __shfl_xor_sync(kFull, l, 2);
#pragma unroll
    for (int nt = 0; nt < 16; ++nt) {
        st.acc[nt][0] += __shfl_xor_sync(kFull, st.acc[nt][0], 16);
        st.acc[nt][1] += __shfl_xor_sync(kFull, st.acc[nt][1], 16);
    }
    // the warp's own K slot is free now: it holds the warp's [4][128] accumulators for the merge
    float* my_acc = reinterpret_cast<float*>(smem + (size_t)warp * 2 * kSlotBytes);
    if (r < kMaxG) {
        if (j == 0) { sm_m[warp][r] = st.m; sm_l[warp][r] = l; }
#pragma unroll
        for (int nt = 0; nt < 16; ++nt) {
            my_acc[r * kD + attend_channel(nt, 2 * j)] = st.acc[nt][0];
            my_acc[r * kD + attend_channel(nt, 2 * j + 1)] = st.acc[nt][1];
        }
    }
    __syncthreads();
    // merge the warps; each work item is one head and a pair of channels
    for (int item = threadIdx.x; item < p.G * (kD / 2); item += kWarps * 32) {
        const int h = item / (kD / 2), c = (item % (kD / 2)) * 2;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) M = fmaxf(M, sm_m[w][h]);
        float L = 0.f, a0 = 0.f, a1 = 0.f;
        if (M != -INFINITY) {
#pragma unroll
            for (int w = 0; w < kWarps; ++w) {
                const float f = exp2f(sm_m[w][h] - M);
                const float* wacc = reinterpret_cast<const float*>(smem + (size_t)w * 2 * kSlotBytes) + h * kD + c;
                L += f * sm_l[w][h];
                a0 += f * wacc[0];
                a1 += f * wacc[1];
            }
        }
        const size_t slot = (head0 + h) * p.splits + split;
        if (c == 0) { p.part_ml[2 * slot] = M; p.part_ml[2 * slot + 1] = L; }
        *reinterpret_cast<float2*>(p.part_acc + slot * kD + c) = make_float2(a0, a1);
    }
    // the last CTA of the unit to get here merges the unit's splits
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        is_last = 0;
        if (p.status[kHeaderCookieWord] != kHeaderCookie) {   // counters that were never zeroed decide nothing
            atomicOr(p.status, kDevBadWorkspace);
        } else {
            const unsigned old = atomicAdd(&arrive[b * p.Hkv + g], 1u);
            is_last = old + 1u == gridDim.x;
            if (is_last) arrive[b * p.Hkv + g] = 0u;   // for the next call
        }
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    // The (m, l) pairs of all splits first, side by side, into shared memory (the K/V slots are free now); then every
    // thread sums its pair of channels over the splits with several loads in flight.
    float2* s_ml = reinterpret_cast<float2*>(smem);   // [G][splits]
    const int nsp = (int)gridDim.x;
    for (int x = threadIdx.x; x < p.G * nsp; x += kWarps * 32) {
        const int h = x / nsp, sp = x % nsp;
        const float2 ml = __ldcg(reinterpret_cast<const float2*>(p.part_ml + 2 * ((head0 + h) * p.splits + sp)));
        s_ml[x] = ml.y > 0.f ? ml : make_float2(-INFINITY, 0.f);
    }
    __syncthreads();
    // one work item = one head and four channels: G * 32 <= 128 items, a single pass of the CTA's 224 threads
    for (int item = threadIdx.x; item < p.G * (kD / 4); item += kWarps * 32) {
        const int h = item / (kD / 4), c = (item % (kD / 4)) * 4;
        const size_t base = (head0 + h) * p.splits;
        const float2* ml = s_ml + h * nsp;
        float M = -INFINITY;
        for (int sp = 0; sp < nsp; ++sp) M = fmaxf(M, ml[sp].x);
        float L = 0.f;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        if (M != -INFINITY) {
            for (int sp0 = 0; sp0 < nsp; sp0 += 8) {
                float4 a[8];
                float f[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const int sp = sp0 + u;
                    f[u] = sp < nsp ? exp2f(ml[sp].x - M) : 0.f;   // exp2(-inf) = 0 for empty splits
                    a[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (f[u] != 0.f) a[u] = __ldcg(reinterpret_cast<const float4*>(p.part_acc + (base + sp) * kD + c));
                }
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    if (sp0 + u < nsp) L += f[u] * ml[sp0 + u].y;
                    acc.x += f[u] * a[u].x;
                    acc.y += f[u] * a[u].y;
                    acc.z += f[u] * a[u].z;
                    acc.w += f[u] * a[u].w;
                }
            }
        }
        const float inv = L > 0.f ? 1.f / L : 0.f;
        if (p.out_fp32) {
            *reinterpret_cast<float4*>(static_cast<float*>(p.out) + (head0 + h) * kD + c) =
                make_float4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv);
        } else {
            __nv_bfloat162* o = reinterpret_cast<__nv_bfloat162*>(static_cast<__nv_bfloat16*>(p.out) + (head0 + h) * kD + c);
            o[0] = __floats2bfloat162_rn(acc.x * inv, acc.y * inv);
            o[1] = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
        }
        if (p.lse && c == 0) p.lse[head0 + h] = L > 0.f ? (M + log2f(L)) * kLn2 : -INFINITY;
    }
}

__global__ void clear_status_kernel(uint32_t* status) { *status = 0u; }

// status word, work counters and class counts (the first 256 bytes of a workspace, with the cookie) and the arrival
// counters of the single-launch kernel that follow them: `words` 32-bit words in all
__global__ void init_header_kernel(uint32_t* header, int words) {
    pdl_launch_dependents();
    pdl_wait();
    for (int i = threadIdx.x; i < words; i += blockDim.x) header[i] = i == kHeaderCookieWord ? kHeaderCookie : 0u;
}

// ---- host side --------------------------------------------------------------------------------------------

struct Plan {
    int blocks_per_split, splits;     // dense path
    int total_items;                  // fused path
    bool small;                       // the geometry is served by the single-launch kernel
    int small_bps, small_splits;      // ... with these splits: at most one CTA per SM, never more splits than the dense path
    int wide_bps, wide_splits;        // the single-launch kernel on large geometries (deeper thumbnails): a few waves
    size_t off_arrive, off_mtilde, off_lens, off_units, off_qrec, off_ml, off_acc, off_fml, off_facc, total;
    size_t off_bmax, off_keep;
    size_t off_scores, total_residual;   // 2 + 8 bit key format: the score tiles follow everything else
};

constexpr size_t kHeaderBytes = 256;
// ffd_workspace_init does not know the geometry: it zeroes the header and as many arrival counters as any geometry can
// have (one per (sequence, KV head), fewer than 65536 of them)
constexpr size_t kInitBytes = kHeaderBytes + 65536 * sizeof(uint32_t);

// score tiles of the 2 + 8 bit format: one ring of (batch descriptors x blocks per item) tiles per CTA of the fused
// kernel, which runs one CTA per SM; sized for GPUs of up to this many SMs
constexpr int kResMaxCtas = 192;

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// SM count of the current device; 148 (B200) when no device can be asked, so that the host-only entry points still
// answer.  Asked on every call: the library caches nothing, and the answer must follow cudaSetDevice.
constexpr int kDefaultSms = 148;
static int device_sms() {
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) {
        (void)cudaGetLastError();
        return kDefaultSms;
    }
    return sms;
}

// Query heads per KV head: 1..4 directly; 6 and 8 as two groups of 3 or 4 heads that share the KV head's tiles (each
// tile is then read once per group: correct, at twice the scan and K/V traffic of a kernel with wider fragments).
static int group_shift(const ffd_config* cfg) {
    const int G = cfg->num_q_heads / cfg->num_kv_heads;
    return (G == 6 || G == 8) ? 1 : 0;
}

// Split geometry is a pure function of (batch, KV heads, max blocks, SM count) so that ffd_workspace_bytes and the
// launch agree.  Aim for at least two CTAs per SM before making splits longer than 8 blocks.
static Plan make_plan(const ffd_config* user_cfg, int batch, int max_blocks, int sms) {
    ffd_config v = *user_cfg;   // the geometry is that of the groups the kernels work on (group_shift)
    v.num_kv_heads <<= group_shift(user_cfg);
    const ffd_config* cfg = &v;
    Plan pl;
    int bps = 32;
    const long units = (long)batch * cfg->num_kv_heads;
    while (bps > 8 && units * ((max_blocks + bps - 1) / bps) < 2 * sms) bps /= 2;
    pl.blocks_per_split = bps;
    pl.splits = max_blocks > 0 ? (max_blocks + bps - 1) / bps : 1;
    const size_t heads = (size_t)batch * cfg->num_q_heads;
    pl.total_items = item_geometry(units, max_blocks, sms).item_rows * batch * cfg->num_kv_heads;
    const size_t fslots = (size_t)pl.total_items * kNA * kMaxG;
    // fewer than two full work items per SM: the single-launch kernel (a pure function of the geometry, like the rest)
    pl.small = units * ((max_blocks + kItemBlocksMax - 1) / kItemBlocksMax) < 2 * sms;
    pl.small_bps = bps;               // (every CTA repeats the scan of the sink and local blocks: few, long splits)
    while (pl.small_bps < max_blocks && units * ((max_blocks + pl.small_bps - 1) / pl.small_bps) > sms) pl.small_bps *= 2;
    pl.small_splits = (max_blocks + pl.small_bps - 1) / pl.small_bps;
    // The same kernel on large geometries (4- and 8-bit thumbnails; decisions from stored block maxima): a CTA's cost is
    // its kept blocks, which no geometry can know, so about four CTAs per SM let the hardware even them out; never
    // shorter splits than the dense path's
    {
        long per_unit = 4L * sms / units;
        if (per_unit < 1) per_unit = 1;
        pl.wide_bps = (int)((max_blocks + per_unit - 1) / per_unit);
        if (pl.wide_bps < bps) pl.wide_bps = bps;
        pl.wide_splits = max_blocks > 0 ? (max_blocks + pl.wide_bps - 1) / pl.wide_bps : 1;
    }
    pl.off_arrive = kHeaderBytes;     // one arrival counter per (sequence, KV head), zeroed with the header
    pl.off_mtilde = align_up(pl.off_arrive + (size_t)units * sizeof(uint32_t), 256);
    pl.off_lens = align_up(pl.off_mtilde + heads * sizeof(float), 256);
    pl.off_units = align_up(pl.off_lens + (size_t)batch * sizeof(int32_t), 256);
    pl.off_qrec = align_up(pl.off_units + (size_t)batch * cfg->num_kv_heads * sizeof(int2), 256);
    pl.off_ml = align_up(pl.off_qrec + (size_t)batch * cfg->num_kv_heads * kQrecBytes, 256);
    pl.off_acc = align_up(pl.off_ml + heads * pl.splits * 2 * sizeof(float), 256);
    pl.off_fml = align_up(pl.off_acc + heads * pl.splits * kD * sizeof(float), 256);
    pl.off_facc = align_up(pl.off_fml + fslots * 2 * sizeof(float), 256);
    pl.total = align_up(pl.off_facc + fslots * kD * sizeof(float), 256);
    // scan -> select -> decode: block maxima [B, Hq, max_blocks] and decision bytes [B, Hkv, max_blocks, 4]
    pl.off_bmax = pl.total;
    pl.off_keep = align_up(pl.off_bmax + heads * (size_t)max_blocks * sizeof(float), 256);
    pl.total = align_up(pl.off_keep + (size_t)units * max_blocks * kMaxG, 256);
    pl.off_scores = pl.total;
    pl.total_residual = pl.off_scores + (size_t)kResMaxCtas * kNB * kItemBlocksMax * kScoreTileFloats * sizeof(float);
    return pl;
}

// two_bit_only: the entry point exists for the 2-bit thumbnails only (the 2 + 8 bit format, the device-side append);
// wide_groups: it also serves 6 and 8 query heads per KV head
static ffd_status check_config(const ffd_config* cfg, bool two_bit_only = false, bool wide_groups = false) {
    if (!cfg) return FFD_ERR_NULL;
    if (cfg->head_dim != kD || cfg->block_tokens != kBlk) return FFD_ERR_UNSUPPORTED;
    if (cfg->quant_bits != 2 && (two_bit_only || (cfg->quant_bits != 4 && cfg->quant_bits != 8))) return FFD_ERR_UNSUPPORTED;
    if (cfg->num_q_heads <= 0 || cfg->num_kv_heads <= 0 || cfg->num_q_heads % cfg->num_kv_heads) return FFD_ERR_SHAPE;
    if (cfg->num_q_heads / cfg->num_kv_heads > kMaxG && !(wide_groups && group_shift(cfg))) return FFD_ERR_UNSUPPORTED;
    if (cfg->n_sink_blocks < 0 || cfg->n_local_blocks < 0 || cfg->n_sink_blocks + cfg->n_local_blocks < 1)
        return FFD_ERR_SHAPE;
    if (cfg->out_dtype != 0 && cfg->out_dtype != 1) return FFD_ERR_UNSUPPORTED;
    if (!(cfg->sm_scale >= 0.f) || isinf(cfg->sm_scale)) return FFD_ERR_SHAPE;
    return FFD_OK;
}

static bool misaligned(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

static ffd_status check_geometry(int batch, int max_blocks, int num_pages) {
    if (batch <= 0 || batch > 65535 || max_blocks <= 0 || num_pages <= 0) return FFD_ERR_SHAPE;
    if ((long)max_blocks * kBlk > 0x7fffffffL) return FFD_ERR_SHAPE;
    return FFD_OK;
}

// Threads per combine CTA (one CTA per head): as many as still let all CTAs be resident at once.
static int combine_threads(long heads, int sms) { return heads <= 2 * sms ? 1024 : heads <= 4 * sms ? 512 : 256; }
// CTAs per head (each takes a share of the channels): more when there are few heads with many partials each, so
// that a long sequence's partials are not summed by a handful of SMs; never so many that a CTA is left with fewer
// than 128 partials (its fixed cost would dominate) or that the grid exceeds two CTAs per SM.
static int combine_split(long heads, long max_partials, int sms) {
    for (int z = 4; z > 1; z >>= 1)
        if (heads * z <= 2 * sms + 32 && max_partials / z >= 128) return z;
    return 1;
}

static cudaEvent_t g_prof_start = nullptr, g_prof_stop = nullptr;

// Launch with programmatic stream serialization: the grid may be scheduled while its predecessor in the stream is
// still running; every kernel of this library calls pdl_wait() before it reads anything a predecessor wrote.
template <typename... KArgs, typename... Args>
static void launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    (void)cudaLaunchKernelEx(&cfg, kernel, args...);   // errors surface through cudaGetLastError in launch_status
}

static ffd_status launch_status() { return cudaGetLastError() == cudaSuccess ? FFD_OK : FFD_ERR_CUDA; }

// Everything about a decode call that can be refused on the host (nothing is launched when this fails).
static ffd_status check_decode_args(bool sparse, const ffd_config* cfg, const void* q, const void* k_cache,
                                    const void* v_cache, const void* k_quant, const void* k_scales,
                                    const int32_t* block_table, const int32_t* seq_lens, int batch, int max_blocks,
                                    int num_pages, float delta, const void* out, const float* lse,
                                    const float* block_max, const void* workspace, const void* k_res) {
    ffd_status st = check_config(cfg, false, k_res == nullptr);
    if (st) return st;
    if (!q || (!k_cache && !k_res) || !v_cache || !seq_lens || !out || !workspace) return FFD_ERR_NULL;
    if (sparse && (!k_quant || !k_scales)) return FFD_ERR_NULL;
    st = check_geometry(batch, max_blocks, num_pages);
    if (st) return st;
    if (cfg->num_kv_heads > 65535 || cfg->num_q_heads > 65535) return FFD_ERR_SHAPE;
    if ((double)num_pages * cfg->num_kv_heads >= 2147483648.0) return FFD_ERR_SHAPE;
    if (((long)batch * cfg->num_kv_heads << group_shift(cfg)) >= 65536L) return FFD_ERR_SHAPE;   // fast_div: items * units < 2^48
    if (sparse && (isnan(delta) || delta < 0.f)) return FFD_ERR_DELTA;
    const void* ptrs[] = {q, k_cache, k_res, v_cache, k_quant, k_scales, block_table, seq_lens, out, lse, block_max,
                          workspace};
    for (const void* ptr : ptrs)
        if (ptr && misaligned(ptr)) return FFD_ERR_ALIGN;
    return FFD_OK;
}

static ffd_status run_decode(bool sparse, const ffd_config* cfg, const void* q, const void* k_cache,
                             const void* v_cache, const void* k_quant, const void* k_scales,
                             const int32_t* block_table, const int32_t* seq_lens, int batch, int max_blocks,
                             int num_pages, float delta, void* out, float* lse, uint8_t* kept_mask,
                             float* block_max, void* workspace, size_t workspace_bytes, void* stream,
                             const AppendParams* append = nullptr, const void* k_res = nullptr, int rule = -1,
                             int top_k = 0) {   // rule >= 0: ffd_decode_select, always scan -> select -> decode
    const ffd_status st = check_decode_args(sparse, cfg, q, k_cache, v_cache, k_quant, k_scales, block_table, seq_lens,
                                            batch, max_blocks, num_pages, delta, out, lse, block_max, workspace, k_res);
    if (st) return st;
    const int sms = device_sms();
    const Plan pl = make_plan(cfg, batch, max_blocks, sms);
    if (workspace_bytes < (k_res ? pl.total_residual : pl.total)) return FFD_ERR_WORKSPACE;

    DecodeParams p;
    memset(&p, 0, sizeof p);
    p.q = static_cast<const __nv_bfloat16*>(q);
    p.k_cache = static_cast<const __nv_bfloat16*>(k_cache);
    p.k_res = static_cast<const int8_t*>(k_res);
    p.v_cache = static_cast<const __nv_bfloat16*>(v_cache);
    p.k_quant = static_cast<const uint8_t*>(k_quant);
    p.k_scales = static_cast<const __half*>(k_scales);
    p.block_table = block_table;
    p.seq_lens = seq_lens;
    p.batch = batch;
    p.Hq = cfg->num_q_heads;
    p.kv_shift = group_shift(cfg);
    if (p.kv_shift && (append || k_res)) return FFD_ERR_UNSUPPORTED;
    p.Hkv_phys = cfg->num_kv_heads;
    p.Hkv = cfg->num_kv_heads << p.kv_shift;
    p.G = p.Hq / p.Hkv;
    p.max_blocks = max_blocks;
    p.num_pages = num_pages;
    p.n_sink = cfg->n_sink_blocks;
    p.n_local = cfg->n_local_blocks;
    p.blocks_per_split = pl.blocks_per_split;
    p.splits = pl.splits;
    p.sm_scale = cfg->sm_scale > 0.f ? cfg->sm_scale : 1.0f / sqrtf((float)kD);
    p.delta = delta;
    char* ws = static_cast<char*>(workspace);
    p.status = reinterpret_cast<uint32_t*>(ws);
    p.mtilde = reinterpret_cast<float*>(ws + pl.off_mtilde);
    p.part_ml = reinterpret_cast<float*>(ws + pl.off_ml);
    p.part_acc = reinterpret_cast<float*>(ws + pl.off_acc);
    p.qrec = reinterpret_cast<unsigned char*>(ws + pl.off_qrec);
    p.fpart_ml = reinterpret_cast<float*>(ws + pl.off_fml);
    p.fpart_acc = reinterpret_cast<float*>(ws + pl.off_facc);
    p.total_items = pl.total_items;
    p.item_counter = reinterpret_cast<uint32_t*>(ws + 64);
    p.class_counts = reinterpret_cast<uint32_t*>(ws + 68);
    p.light_counter = reinterpret_cast<uint32_t*>(ws + 76);
    p.len_stats = reinterpret_cast<uint32_t*>(ws + 80);
    p.unit_list = reinterpret_cast<int2*>(ws + pl.off_units);
    p.res_scores = reinterpret_cast<float*>(ws + pl.off_scores);
    p.bmax = reinterpret_cast<float*>(ws + pl.off_bmax);
    p.keep_bits = reinterpret_cast<uint8_t*>(ws + pl.off_keep);
    p.units = batch * p.Hkv;
    const ItemGeom geom = item_geometry(p.units, max_blocks, sms);
    p.item_rows = geom.item_rows;
    p.rows_small = geom.rows_small;
    p.item_blocks = geom.item_blocks;
    p.units_magic = fast_div_magic((unsigned)p.units);
    p.hkv_magic = fast_div_magic((unsigned)p.Hkv);
    p.kept_mask = kept_mask;
    p.block_max = block_max;
    p.out = out;
    p.lse = lse;
    p.out_fp32 = cfg->out_dtype;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const dim3 grid(p.splits, p.Hkv, batch);
    const bool prof = g_prof_start && g_prof_stop;
    if (sparse) {
        if (cudaFuncSetAttribute(fused_sparse_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kFusedSmem) != cudaSuccess ||
            cudaFuncSetAttribute(fused_sparse_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kFusedSmem) != cudaSuccess)
            return FFD_ERR_CUDA;
        if (k_res && sms > kResMaxCtas) return FFD_ERR_UNSUPPORTED;
        // the work counters and class counts at ws + 64 are zero here: ffd_workspace_init zeroes them and the
        // combine kernel of every call leaves them zeroed for the next one (the kernels check the header's cookie)
        // 4- / 8-bit thumbnails: the single-launch kernel on small geometries, scan -> select -> decode on large ones;
        // ffd_decode_select: scan -> select -> decode at every size and depth
        const bool deeper = cfg->quant_bits != 2;
        if ((deeper || rule >= 0) && (append || k_res)) return FFD_ERR_UNSUPPORTED;
        const bool three = rule >= 0 || (deeper && !pl.small);
        if ((pl.small || three) && !append && !k_res) {   // little work: the whole step in one launch
            void (*kernel)(DecodeParams, uint32_t*) = three ? small_sparse_kernel<0>
                                                      : cfg->quant_bits == 2 ? small_sparse_kernel<2>
                                                      : cfg->quant_bits == 4 ? small_sparse_kernel<4> : small_sparse_kernel<8>;
            if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kDecodeSmem) != cudaSuccess)
                return FFD_ERR_CUDA;
            if (pl.small) {
                p.blocks_per_split = pl.small_bps;
                p.splits = pl.small_splits;
            } else {
                p.blocks_per_split = pl.wide_bps;
                p.splits = pl.wide_splits;
            }
            if (prof) cudaEventRecord(g_prof_start, s);
            if (three) {
                const dim3 scan_grid((p.max_blocks + kScanCtaBlocks - 1) / kScanCtaBlocks, p.Hkv, batch);
                launch_pdl(cfg->quant_bits == 2 ? scan_blocks_kernel<2> : cfg->quant_bits == 4 ? scan_blocks_kernel<4> : scan_blocks_kernel<8>,
                           scan_grid, dim3(256), 0, s, p);
                launch_pdl(select_kernel, dim3(p.Hq, batch), dim3(kSelectThreads), 0, s, p, rule < 0 ? (int)kRulePseudoMax : rule, top_k);
            }
            launch_pdl(kernel, dim3(p.splits, p.Hkv, batch), dim3(kWarps * 32), kDecodeSmem, s, p,
                       reinterpret_cast<uint32_t*>(ws + pl.off_arrive));
            if (prof) cudaEventRecord(g_prof_stop, s);
            return launch_status();
        }
        if (append) {
            // the kernels after the first one read the lengths it leaves in the workspace
            int32_t* new_lens = reinterpret_cast<int32_t*>(ws + pl.off_lens);
            launch_pdl(pseudomax_kernel<true>, dim3(p.Hkv, batch), dim3(kPmWarps * 32), 0, s, p, *append, new_lens);
            p.seq_lens = new_lens;
            p.bump_lens = append->seq_lens;
        } else {
            launch_pdl(pseudomax_kernel<false>, dim3(p.Hkv, batch), dim3(kPmWarps * 32), 0, s, p, AppendParams{},
                       static_cast<int32_t*>(nullptr));
        }
        if (prof) cudaEventRecord(g_prof_start, s);
        launch_pdl(k_res ? fused_sparse_kernel<true> : fused_sparse_kernel<false>, dim3(min(p.total_items, sms)),
                   dim3(kFusedThreads), kFusedSmem, s, p);
        if (prof) cudaEventRecord(g_prof_stop, s);
        launch_pdl(combine_kernel<true>, dim3(p.Hq, batch, combine_split(p.Hq * batch, (long)p.item_rows * kNA, sms)),
                   dim3(combine_threads(p.Hq * batch, sms)), 0, s, p);
    } else {
        if (cudaFuncSetAttribute(dense_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kDecodeSmem) != cudaSuccess)
            return FFD_ERR_CUDA;
        if (prof) cudaEventRecord(g_prof_start, s);
        launch_pdl(dense_kernel, grid, dim3(kWarps * 32), kDecodeSmem, s, p);
        if (prof) cudaEventRecord(g_prof_stop, s);
        launch_pdl(combine_kernel<false>, dim3(p.Hq, batch, combine_split(p.Hq * batch, p.splits, sms)),
                   dim3(combine_threads(p.Hq * batch, sms)), 0, s, p);
    }
    return launch_status();
}

}  // namespace ffd

using namespace ffd;

static ffd_status quantize_impl(const ffd_config* cfg, const void* k_cache, void* k_quant, void* k_scales, void* k_res,
                                const int32_t* block_table, const int32_t* seq_lens, const int32_t* first_token,
                                int32_t batch, int32_t max_blocks_per_seq, int32_t num_pages, void* stream);

extern "C" {

const char* ffd_status_string(ffd_status status) {
    switch (status) {
        case FFD_OK: return "ok";
        case FFD_ERR_NULL: return "required pointer is NULL";
        case FFD_ERR_SHAPE: return "shape or count out of range";
        case FFD_ERR_UNSUPPORTED: return "unsupported configuration (needs head_dim 128, block 64, 2 bits, group <= 4)";
        case FFD_ERR_ALIGN: return "device pointer not 16-byte aligned";
        case FFD_ERR_WORKSPACE: return "workspace too small";
        case FFD_ERR_DELTA: return "delta must be >= 0 or +inf";
        case FFD_ERR_CUDA: return "CUDA runtime error";
        case FFD_ERR_DEVICE_STATUS: return "a kernel recorded a problem in the status word";
        case FFD_ERR_STATIC_LIMIT:
            return "geometry needs more scratch than the built-in FFD_STATIC_SCRATCH_BYTES array of ffd_decode_static";
    }
    return "unknown status";
}

ffd_status ffd_workspace_bytes(const ffd_config* cfg, int32_t batch, int32_t max_blocks_per_seq, size_t* bytes) {
    ffd_status st = check_config(cfg, false, true);
    if (st) return st;
    if (!bytes) return FFD_ERR_NULL;
    st = check_geometry(batch, max_blocks_per_seq, 1);
    if (st) return st;
    *bytes = make_plan(cfg, batch, max_blocks_per_seq, device_sms()).total;
    return FFD_OK;
}

ffd_status ffd_workspace_bytes_residual(const ffd_config* cfg, int32_t batch, int32_t max_blocks_per_seq, size_t* bytes) {
    ffd_status st = check_config(cfg, true);
    if (st) return st;
    if (!bytes) return FFD_ERR_NULL;
    st = check_geometry(batch, max_blocks_per_seq, 1);
    if (st) return st;
    *bytes = make_plan(cfg, batch, max_blocks_per_seq, device_sms()).total_residual;
    return FFD_OK;
}

ffd_status ffd_workspace_init(void* workspace, size_t workspace_bytes, void* stream) {
    if (!workspace) return FFD_ERR_NULL;
    if (workspace_bytes < 256) return FFD_ERR_WORKSPACE;
    if (misaligned(workspace)) return FFD_ERR_ALIGN;
    const size_t bytes = workspace_bytes < kInitBytes ? workspace_bytes : kInitBytes;
    launch_pdl(init_header_kernel, dim3(1), dim3(1024), 0, static_cast<cudaStream_t>(stream),
               static_cast<uint32_t*>(workspace), (int)(bytes / sizeof(uint32_t)));
    return launch_status();
}

ffd_status ffd_quantize_keys(const ffd_config* cfg, const void* k_cache, void* k_quant, void* k_scales,
                             const int32_t* block_table, const int32_t* seq_lens, const int32_t* first_token,
                             int32_t batch, int32_t max_blocks_per_seq, int32_t num_pages, void* stream) {
    return quantize_impl(cfg, k_cache, k_quant, k_scales, nullptr, block_table, seq_lens, first_token, batch,
                         max_blocks_per_seq, num_pages, stream);
}

ffd_status ffd_quantize_keys_residual(const ffd_config* cfg, const void* k_cache, void* k_quant, void* k_scales,
                                      void* k_res, const int32_t* block_table, const int32_t* seq_lens,
                                      const int32_t* first_token, int32_t batch, int32_t max_blocks_per_seq,
                                      int32_t num_pages, void* stream) {
    if (!k_res) return FFD_ERR_NULL;
    if (misaligned(k_res)) return FFD_ERR_ALIGN;
    return quantize_impl(cfg, k_cache, k_quant, k_scales, k_res, block_table, seq_lens, first_token, batch,
                         max_blocks_per_seq, num_pages, stream);
}

}   // extern "C"

// thumbnails, and with k_res also the residuals: in the same launch when only tail blocks are redone, else by the
// streaming kernel followed by the residual kernel
static ffd_status quantize_impl(const ffd_config* cfg, const void* k_cache, void* k_quant, void* k_scales, void* k_res,
                                const int32_t* block_table, const int32_t* seq_lens, const int32_t* first_token,
                                int32_t batch, int32_t max_blocks_per_seq, int32_t num_pages, void* stream) {
    ffd_status st = check_config(cfg, false, k_res == nullptr);
    if (st) return st;
    if (!k_cache || !k_quant || !k_scales || !seq_lens) return FFD_ERR_NULL;
    st = check_geometry(batch, max_blocks_per_seq, num_pages);
    if (st) return st;
    if (cfg->num_kv_heads > 65535) return FFD_ERR_SHAPE;
    const void* ptrs[] = {k_cache, k_quant, k_scales, block_table, seq_lens, first_token};
    for (const void* ptr : ptrs)
        if (ptr && misaligned(ptr)) return FFD_ERR_ALIGN;
    if (k_res && cfg->quant_bits != 2) return FFD_ERR_UNSUPPORTED;   // the residual format is defined on the 2-bit thumbnails
    QuantParams p{static_cast<const __nv_bfloat16*>(k_cache), static_cast<uint8_t*>(k_quant),
                  static_cast<__half*>(k_scales), block_table, seq_lens, first_token,
                  cfg->num_kv_heads, max_blocks_per_seq, num_pages};
    if (cfg->quant_bits != 2) {   // 4 or 8 bits: the plain tile-at-a-time kernel for whole caches and tail blocks alike
        long x = first_token ? 2 : (16L * device_sms() + (long)batch * cfg->num_kv_heads - 1) / ((long)batch * cfg->num_kv_heads);
        x = x > max_blocks_per_seq ? max_blocks_per_seq : (x < 1 ? 1 : x);
        launch_pdl(cfg->quant_bits == 4 ? quantize_wide_kernel<4> : quantize_wide_kernel<8>,
                   dim3((unsigned)x, cfg->num_kv_heads, batch), dim3(128), 0, static_cast<cudaStream_t>(stream), p);
        return launch_status();
    }
    // CTAs per (sequence, KV head): every CTA walks its share of the blocks, so any number is correct.  With
    // first_token (decode steps re-quantize the block the new token fell into) two are plenty and a wide grid
    // would only launch thousands of CTAs that find nothing to do.
    const int wide = max_blocks_per_seq < 64 ? max_blocks_per_seq : 64;
    if (first_token) {
        launch_pdl(quantize_kernel, dim3(wide < 2 ? wide : 2, cfg->num_kv_heads, batch), dim3(128), 0,
                   static_cast<cudaStream_t>(stream), p, static_cast<int8_t*>(k_res));
    } else {   // a whole cache: the streaming kernel; twelve CTAs fit an SM, and four times as many as fit at once are
               // launched so that sequences of different lengths even out
        if (cudaFuncSetAttribute(quantize_bulk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kQbSmem) != cudaSuccess)
            return FFD_ERR_CUDA;
        const long tiles = (long)max_blocks_per_seq * cfg->num_kv_heads;
        long x = (48L * device_sms() + batch - 1) / batch;
        if (x > tiles) x = tiles;
        launch_pdl(quantize_bulk_kernel, dim3((unsigned)x, batch), dim3(kQbThreads), kQbSmem,
                   static_cast<cudaStream_t>(stream), p);
        if (k_res) {
            st = launch_status();
            if (st) return st;
            return ffd_quantize_residual(cfg, k_cache, k_scales, k_res, block_table, seq_lens, nullptr, batch,
                                         max_blocks_per_seq, num_pages, stream);
        }
    }
    return launch_status();
}

extern "C" {

ffd_status ffd_quantize_residual(const ffd_config* cfg, const void* k_cache, const void* k_scales, void* k_res,
                                 const int32_t* block_table, const int32_t* seq_lens, const int32_t* first_token,
                                 int32_t batch, int32_t max_blocks_per_seq, int32_t num_pages, void* stream) {
    ffd_status st = check_config(cfg, true);
    if (st) return st;
    if (!k_cache || !k_scales || !k_res || !seq_lens) return FFD_ERR_NULL;
    st = check_geometry(batch, max_blocks_per_seq, num_pages);
    if (st) return st;
    if (cfg->num_kv_heads > 65535) return FFD_ERR_SHAPE;
    const void* ptrs[] = {k_cache, k_scales, k_res, block_table, seq_lens, first_token};
    for (const void* ptr : ptrs)
        if (ptr && misaligned(ptr)) return FFD_ERR_ALIGN;
    ResidualParams p{static_cast<const __nv_bfloat16*>(k_cache), static_cast<const __half*>(k_scales),
                     static_cast<int8_t*>(k_res), block_table, seq_lens, first_token,
                     cfg->num_kv_heads, max_blocks_per_seq, num_pages};
    // as in ffd_quantize_keys: every CTA walks its share of the blocks; two per (sequence, KV head) when only the
    // tail block is redone, else enough to fill the GPU several times over
    long x = first_token ? 2 : (16L * device_sms() + (long)batch * cfg->num_kv_heads - 1) / ((long)batch * cfg->num_kv_heads);
    if (x > max_blocks_per_seq) x = max_blocks_per_seq;
    if (x < 1) x = 1;
    launch_pdl(residual_kernel, dim3((unsigned)x, cfg->num_kv_heads, batch), dim3(128), 0,
               static_cast<cudaStream_t>(stream), p);
    return launch_status();
}

static ffd_status append_impl(const ffd_config* cfg, const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                              void* k_quant, void* k_scales, void* k_res, const int32_t* block_table, int32_t* seq_lens,
                              int32_t batch, int32_t max_blocks_per_seq, int32_t num_pages, void* workspace,
                              size_t workspace_bytes, void* stream) {
    ffd_status st = check_config(cfg, true);
    if (st) return st;
    if (!k_new || !v_new || !k_cache || !v_cache || !k_quant || !k_scales || !seq_lens || !workspace) return FFD_ERR_NULL;
    st = check_geometry(batch, max_blocks_per_seq, num_pages);
    if (st) return st;
    if (cfg->num_kv_heads > 65535) return FFD_ERR_SHAPE;
    if (workspace_bytes < 256) return FFD_ERR_WORKSPACE;
    const void* ptrs[] = {k_new, v_new, k_cache, v_cache, k_quant, k_scales, k_res, block_table, seq_lens, workspace};
    for (const void* ptr : ptrs)
        if (ptr && misaligned(ptr)) return FFD_ERR_ALIGN;
    AppendParams p{static_cast<const __nv_bfloat16*>(k_new), static_cast<const __nv_bfloat16*>(v_new),
                   static_cast<__nv_bfloat16*>(k_cache), static_cast<__nv_bfloat16*>(v_cache),
                   static_cast<uint8_t*>(k_quant), static_cast<__half*>(k_scales), block_table, seq_lens,
                   static_cast<uint32_t*>(workspace), cfg->num_kv_heads, max_blocks_per_seq, num_pages,
                   static_cast<int8_t*>(k_res)};
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    launch_pdl(append_kernel, dim3(cfg->num_kv_heads, batch), dim3(128), 0, s, p);
    launch_pdl(bump_lengths_kernel, dim3((batch + 255) / 256), dim3(256), 0, s, seq_lens, (int)batch,
               (int)(max_blocks_per_seq * kBlk));
    return launch_status();
}

ffd_status ffd_append_kv(const ffd_config* cfg, const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                         void* k_quant, void* k_scales, const int32_t* block_table, int32_t* seq_lens, int32_t batch,
                         int32_t max_blocks_per_seq, int32_t num_pages, void* workspace, size_t workspace_bytes,
                         void* stream) {
    return append_impl(cfg, k_new, v_new, k_cache, v_cache, k_quant, k_scales, nullptr, block_table, seq_lens, batch,
                       max_blocks_per_seq, num_pages, workspace, workspace_bytes, stream);
}

ffd_status ffd_append_kv_residual(const ffd_config* cfg, const void* k_new, const void* v_new, void* k_cache,
                                  void* v_cache, void* k_quant, void* k_scales, void* k_res, const int32_t* block_table,
                                  int32_t* seq_lens, int32_t batch, int32_t max_blocks_per_seq, int32_t num_pages,
                                  void* workspace, size_t workspace_bytes, void* stream) {
    if (!k_res) return FFD_ERR_NULL;
    return append_impl(cfg, k_new, v_new, k_cache, v_cache, k_quant, k_scales, k_res, block_table, seq_lens, batch,
                       max_blocks_per_seq, num_pages, workspace, workspace_bytes, stream);
}

ffd_status ffd_decode(const ffd_config* cfg, const void* q, const void* k_cache, const void* v_cache,
                      const void* k_quant, const void* k_scales, const int32_t* block_table,
                      const int32_t* seq_lens, int32_t batch, int32_t max_blocks_per_seq, int32_t num_pages,
                      float delta, void* out, float* lse, uint8_t* kept_mask, float* block_max, void* workspace,
                      size_t workspace_bytes, void* stream) {
    return run_decode(true, cfg, q, k_cache, v_cache, k_quant, k_scales, block_table, seq_lens, batch,
                      max_blocks_per_seq, num_pages, delta, out, lse, kept_mask, block_max, workspace,
                      workspace_bytes, stream);
}

ffd_status ffd_decode_select(const ffd_config* cfg, int32_t rule, int32_t top_k, const void* q, const void* k_cache,
                             const void* v_cache, const void* k_quant, const void* k_scales, const int32_t* block_table,
                             const int32_t* seq_lens, int32_t batch, int32_t max_blocks_per_seq, int32_t num_pages,
                             float delta, void* out, float* lse, uint8_t* kept_mask, float* block_max, void* workspace,
                             size_t workspace_bytes, void* stream) {
    if (rule < FFD_RULE_PSEUDO_MAX || rule > FFD_RULE_TOP_K) return FFD_ERR_UNSUPPORTED;
    if (rule == FFD_RULE_TOP_K && top_k < 1) return FFD_ERR_SHAPE;
    return run_decode(true, cfg, q, k_cache, v_cache, k_quant, k_scales, block_table, seq_lens, batch,
                      max_blocks_per_seq, num_pages, delta, out, lse, kept_mask, block_max, workspace,
                      workspace_bytes, stream, nullptr, nullptr, rule, top_k);
}

ffd_status ffd_decode_residual(const ffd_config* cfg, const void* q, const void* k_res, const void* v_cache,
                               const void* k_quant, const void* k_scales, const int32_t* block_table,
                               const int32_t* seq_lens, int32_t batch, int32_t max_blocks_per_seq, int32_t num_pages,
                               float delta, void* out, float* lse, uint8_t* kept_mask, float* block_max,
                               void* workspace, size_t workspace_bytes, void* stream) {
    if (!k_res) return FFD_ERR_NULL;
    return run_decode(true, cfg, q, nullptr, v_cache, k_quant, k_scales, block_table, seq_lens, batch,
                      max_blocks_per_seq, num_pages, delta, out, lse, kept_mask, block_max, workspace,
                      workspace_bytes, stream, nullptr, k_res);
}

ffd_status ffd_append_decode(const ffd_config* cfg, const void* k_new, const void* v_new, const void* q, void* k_cache,
                             void* v_cache, void* k_quant, void* k_scales, const int32_t* block_table,
                             int32_t* seq_lens, int32_t batch, int32_t max_blocks_per_seq, int32_t num_pages,
                             float delta, void* out, float* lse, uint8_t* kept_mask, float* block_max, void* workspace,
                             size_t workspace_bytes, void* stream) {
    if (!k_new || !v_new) return FFD_ERR_NULL;
    if (misaligned(k_new) || misaligned(v_new)) return FFD_ERR_ALIGN;
    AppendParams ap{static_cast<const __nv_bfloat16*>(k_new), static_cast<const __nv_bfloat16*>(v_new),
                    static_cast<__nv_bfloat16*>(k_cache), static_cast<__nv_bfloat16*>(v_cache),
                    static_cast<uint8_t*>(k_quant), static_cast<__half*>(k_scales), block_table, seq_lens,
                    static_cast<uint32_t*>(workspace), cfg ? cfg->num_kv_heads : 0, max_blocks_per_seq, num_pages};
    return run_decode(true, cfg, q, k_cache, v_cache, k_quant, k_scales, block_table, seq_lens, batch,
                      max_blocks_per_seq, num_pages, delta, out, lse, kept_mask, block_max, workspace, workspace_bytes,
                      stream, &ap);
}

ffd_status ffd_decode_dense(const ffd_config* cfg, const void* q, const void* k_cache, const void* v_cache,
                            const int32_t* block_table, const int32_t* seq_lens, int32_t batch,
                            int32_t max_blocks_per_seq, int32_t num_pages, void* out, float* lse, void* workspace,
                            size_t workspace_bytes, void* stream) {
    return run_decode(false, cfg, q, k_cache, v_cache, nullptr, nullptr, block_table, seq_lens, batch,
                      max_blocks_per_seq, num_pages, INFINITY, out, lse, nullptr, nullptr, workspace,
                      workspace_bytes, stream);
}

ffd_status ffd_unpack_codes(const ffd_config* cfg, const void* k_quant, uint8_t* codes, int32_t num_pages,
                            void* stream) {
    ffd_status st = check_config(cfg, false, true);
    if (st) return st;
    if (!k_quant || !codes) return FFD_ERR_NULL;
    if (num_pages <= 0) return FFD_ERR_SHAPE;
    if (misaligned(k_quant) || misaligned(codes)) return FFD_ERR_ALIGN;
    const size_t tiles = (size_t)num_pages * cfg->num_kv_heads;
    if (tiles > 0x7fffffffu) return FFD_ERR_SHAPE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cfg->quant_bits == 2) unpack_kernel<<<(unsigned)tiles, 128, 0, s>>>(static_cast<const uint8_t*>(k_quant), codes, tiles);
    else if (cfg->quant_bits == 4) unpack_wide_kernel<4><<<(unsigned)tiles, 128, 0, s>>>(static_cast<const uint8_t*>(k_quant), codes, tiles);
    else unpack_wide_kernel<8><<<(unsigned)tiles, 128, 0, s>>>(static_cast<const uint8_t*>(k_quant), codes, tiles);
    return launch_status();
}

// ---- ffd_decode_static: the decode step for callers that cannot allocate ------------------------------------
//
// The scratch that ffd_decode takes from its caller lives here instead, in the library image.  In host code the
// name `g_static_scratch` is only a handle for the symbol, not a device address: the address the kernels need comes
// from cudaGetSymbolAddress, asked once per device (with that device current) and cached.
static __device__ __align__(256) unsigned char g_static_scratch[FFD_STATIC_SCRATCH_BYTES];

static ffd_status static_scratch_address(void** out) {
    constexpr int kMaxDevices = 64;
    static std::mutex lock;
    static void* cache[kMaxDevices] = {nullptr};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return FFD_ERR_CUDA;
    std::lock_guard<std::mutex> guard(lock);
    if (!cache[dev]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) {
            (void)cudaGetLastError();
            return FFD_ERR_CUDA;
        }
        cache[dev] = ptr;
    }
    *out = cache[dev];
    return FFD_OK;
}

ffd_status ffd_decode_static(const ffd_config* cfg, const void* q, const void* k_cache, const void* v_cache,
                             const void* k_quant, const void* k_scales, const int32_t* block_table,
                             const int32_t* seq_lens, int32_t batch, int32_t max_blocks_per_seq, int32_t num_pages,
                             float delta, void* out, float* lse, void* stream) {
    // everything that can be refused on the host is refused before the device is touched
    ffd_status st = check_config(cfg, true);   // (the built-in scratch is sized for the 2-bit path)
    if (st) return st;
    st = check_geometry(batch, max_blocks_per_seq, num_pages);
    if (st) return st;
    if (make_plan(cfg, batch, max_blocks_per_seq, device_sms()).total > FFD_STATIC_SCRATCH_BYTES) return FFD_ERR_STATIC_LIMIT;
    void* scratch = nullptr;
    st = static_scratch_address(&scratch);
    if (st) return st;
    st = check_decode_args(true, cfg, q, k_cache, v_cache, k_quant, k_scales, block_table, seq_lens, batch,
                           max_blocks_per_seq, num_pages, delta, out, lse, nullptr, scratch, nullptr);
    if (st) return st;
    // The array still holds whatever the previous call left there, and nobody else can initialise it: the whole
    // header (status word, work counters, cookie) is rewritten at the start of every call.
    const Plan spl = make_plan(cfg, batch, max_blocks_per_seq, device_sms());
    launch_pdl(init_header_kernel, dim3(1), dim3(1024), 0, static_cast<cudaStream_t>(stream), static_cast<uint32_t*>(scratch),
               (int)(spl.off_mtilde / sizeof(uint32_t)));
    if (cudaGetLastError() != cudaSuccess) return FFD_ERR_CUDA;
    return run_decode(true, cfg, q, k_cache, v_cache, k_quant, k_scales, block_table, seq_lens, batch,
                      max_blocks_per_seq, num_pages, delta, out, lse, nullptr, nullptr, scratch,
                      FFD_STATIC_SCRATCH_BYTES, stream);
}

ffd_status ffd_profile_events(void* start_event, void* stop_event) {
    if ((start_event == nullptr) != (stop_event == nullptr)) return FFD_ERR_NULL;
    g_prof_start = static_cast<cudaEvent_t>(start_event);
    g_prof_stop = static_cast<cudaEvent_t>(stop_event);
    return FFD_OK;
}

ffd_status ffd_read_device_status(void* workspace, void* stream, uint32_t* status_bits) {
    if (!workspace || !status_bits) return FFD_ERR_NULL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(status_bits, workspace, sizeof(uint32_t), cudaMemcpyDeviceToHost, s) != cudaSuccess)
        return FFD_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return FFD_ERR_CUDA;
    if (*status_bits) {
        clear_status_kernel<<<1, 1, 0, s>>>(static_cast<uint32_t*>(workspace));
        if (cudaGetLastError() != cudaSuccess) return FFD_ERR_CUDA;
        return FFD_ERR_DEVICE_STATUS;
    }
    return FFD_OK;
}

}  // extern "C"
