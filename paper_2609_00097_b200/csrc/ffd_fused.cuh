// The fused sparse kernel: scan -> top-delta select -> exact attention over kept blocks, in one persistent launch.
//
// One CTA per SM, 12 warps in two roles that run concurrently:
//   8 scan warps    stream the 2-bit codes and scales of every block through a private 3-stage cp.async ring
//                   (3 blocks = 6.9 KB in flight per warp), compute the block maxima of the approximate scores
//                   on the tensor cores and publish the keep decisions of one work item in a batch descriptor;
//   4 attend warps  take the kept blocks of a published batch, stage their K and V tiles (16 KB each) through
//                   private swizzled slots with cp.async + mbarrier and run the exact online-softmax attention.
// A work item is 32 consecutive blocks of one (sequence, KV head).  Items are handed out dynamically: lane 0 of scan
// warp 0 draws item numbers from a global counter two items ahead and shares them with the other scan warps
// through a small ring and one named barrier per item; attend warps learn the item from the batch descriptor.
// Scan warps run up to two items ahead of the attend warps (two batch descriptors, full/empty mbarriers).
// Every mbarrier wait is bounded; on expiry the warp records kDevTimeout and the CTA winds down.
#pragma once
#include "ffd_kernels.cuh"

namespace ffd {

constexpr int kNS = 8;                 // scan warps
constexpr int kNA = 4;                 // attend warps
constexpr int kFusedThreads = (kNS + kNA) * 32;
constexpr int kItemBlocks = 32;        // blocks per work item
constexpr int kRing = 3;               // code-ring stages per scan warp
constexpr int kStageBytes = kCodeBytes + kD * 2;   // 2048 B codes + 256 B scales
constexpr int kNB = 2;                 // batch descriptors in flight

struct BatchDesc {
    int item;                          // work item of this batch; < 0: no more work
    int pad[3];
    uint32_t tile[kItemBlocks];        // (page, KV head) tile of each block of the item
    uint8_t keep4[kItemBlocks];        // bit h: query head h of the group keeps the block; 0 = skipped
    uint8_t rows[kItemBlocks];         // valid tokens
};

constexpr int kOffSlots = 0;
constexpr int kOffRing = kOffSlots + kNA * 2 * kSlotBytes;
constexpr int kOffDesc = kOffRing + kNS * kRing * kStageBytes;
constexpr int kOffBars = kOffDesc + kNB * (int)sizeof(BatchDesc);
constexpr int kOffIds = kOffBars + (2 * kNB + 2 * kNA) * 8;      // ring of 4 item numbers + abort flag
constexpr int kFusedSmem = kOffIds + 8 * 4;
static_assert(kOffBars % 8 == 0 && kOffRing % 16 == 0 && kOffDesc % 16 == 0, "alignment");

struct Item {
    int b, g, blk0, nblk, n;           // nblk <= 0: nothing to do
};

__device__ __forceinline__ Item decode_item(const DecodeParams& p, int item) {
    Item it;
    const int units = p.batch * p.Hkv;
    const int bg = item % units, split = item / units;
    it.b = bg / p.Hkv;
    it.g = bg % p.Hkv;
    it.n = clamped_seq_len(p, it.b);
    const int nb = (it.n + kBlk - 1) / kBlk;
    it.blk0 = split * kItemBlocks;
    it.nblk = min(nb - it.blk0, kItemBlocks);
    return it;
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" ::"r"(bar) : "memory");
}

__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n .reg .pred p;\n mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
                 : "=r"(ok)
                 : "r"(bar), "r"(parity)
                 : "memory");
    return ok != 0;
}

// ---- scan role ---------------------------------------------------------------------------------------------

__device__ __forceinline__ void scan_warps_barrier() { asm volatile("bar.sync 1, %0;\n" ::"n"(kNS * 32) : "memory"); }

// Draw the next non-empty work item from the global counter (one thread); p.total_items when none is left.
__device__ __forceinline__ int draw_item(const DecodeParams& p) {
    for (;;) {
        const int item = (int)atomicAdd(p.item_counter, 1u);
        if (item >= p.total_items) return p.total_items;
        if (decode_item(p, item).nblk > 0) return item;
    }
}

// Position of a scan warp in its stream of blocks: batch after batch, local blocks w, w+8, w+16, w+24.
struct ScanCursor {
    int bi;        // batch the cursor is in
    Item it;       // nblk = 0 before the first batch
    int lb;
    bool end;      // ran into the end of the work
};

// Advance to this warp's next block.  Returns false when that block lies beyond the batches whose item numbers
// are known (bi <= horizon) or beyond the end of the work; the cursor then stays where it can resume.
__device__ __forceinline__ bool cursor_next(ScanCursor& c, const DecodeParams& p, const volatile int* ids, int horizon,
                                            int w) {
    if (c.end) return false;
    int lb = c.lb + kNS;
    while (lb >= c.it.nblk) {
        if (c.bi + 1 > horizon) { c.lb = lb - kNS; return false; }   // resume here later (lb is re-derived)
        const int item = ids[(c.bi + 1) & 3];
        ++c.bi;
        if (item >= p.total_items) { c.end = true; c.it.nblk = 0; return false; }
        c.it = decode_item(p, item);
        lb = w;
    }
    c.lb = lb;
    return true;
}

// start the copy of one block's codes + scales into a ring stage (one commit group)
__device__ __forceinline__ void ring_issue(const DecodeParams& p, const ScanCursor& c, uint32_t stage, int lane) {
    const int page = page_of(p, c.it.b, c.it.blk0 + c.lb);
    if (page >= 0) {
        const size_t tile = (size_t)page * p.Hkv + c.it.g;
        const uint4* codes = reinterpret_cast<const uint4*>(p.k_quant + tile * kCodeBytes);
#pragma unroll
        for (int x = 0; x < 4; ++x) cp_async16(stage + (x * 32 + lane) * 16, codes + x * 32 + lane);
        if (lane < 16)
            cp_async16(stage + kCodeBytes + lane * 16, reinterpret_cast<const uint4*>(p.k_scales + tile * kD) + lane);
    }
    asm volatile("cp.async.commit_group;\n" ::: "memory");
}

__device__ __forceinline__ void ring_wait(int younger) {
    if (younger >= 2) asm volatile("cp.async.wait_group 2;\n" ::: "memory");
    else if (younger == 1) asm volatile("cp.async.wait_group 1;\n" ::: "memory");
    else asm volatile("cp.async.wait_group 0;\n" ::: "memory");
}

__device__ __forceinline__ void scan_role(const DecodeParams& p, unsigned char* smem, int w, int lane) {
    const int r = lane >> 2, j = lane & 3;
    const uint32_t ring = smem_u32(smem) + kOffRing + w * kRing * kStageBytes;
    const uint32_t bars = smem_u32(smem) + kOffBars;
    BatchDesc* descs = reinterpret_cast<BatchDesc*>(smem + kOffDesc);
    volatile int* ids = reinterpret_cast<volatile int*>(smem + kOffIds);
    volatile int* abort_flag = ids + 4;

    if (w == 0 && lane == 0) {
        ids[0] = draw_item(p);
        ids[1] = ids[0] < p.total_items ? draw_item(p) : p.total_items;
    }
    ScanCursor ic;
    ic.bi = -1;
    ic.it.nblk = 0;
    ic.lb = w - kNS;
    ic.end = false;
    int issued = 0, consumed = 0;   // this warp's blocks whose copies were started / whose data was taken
    ScanQuery sq;
    sq.piece = r & 1;

    for (int bi = 0;; ++bi) {
        const int slot = bi & 1, use = bi >> 1;
        // the attend warps must have released this descriptor (two batches ago)
        if (use > 0 && !mbar_wait(bars + (kNB + slot) * 8, (use - 1) & 1)) *abort_flag = 1;
        if (w == 0 && lane == 0) {
            const int prev = ids[(bi + 1) & 3];
            ids[(bi + 2) & 3] = prev < p.total_items ? draw_item(p) : p.total_items;
        }
        __syncwarp();
        scan_warps_barrier();          // item numbers of batches bi, bi+1, bi+2 are visible to all scan warps
        const int horizon = bi + 2;
        const int item = ids[bi & 3];
        BatchDesc& d = descs[slot];
        if (item >= p.total_items || *abort_flag) {   // no more work: tell the attend warps
            if (lane == 0) {
                if (w == 0) d.item = -1;
                mbar_arrive(bars + slot * 8);
            }
            break;
        }
        const Item it = decode_item(p, item);
        const size_t head0 = (size_t)it.b * p.Hq + (size_t)it.g * p.G;
        {   // pre-scaled fp16 query fragments written by the pseudo-max kernel
            const uint4* qf = reinterpret_cast<const uint4*>(p.qfrag) + ((size_t)(it.b * p.Hkv + it.g) * 32 + lane) * 4;
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                const uint4 v = __ldg(qf + x);
                sq.qh[4 * x] = v.x; sq.qh[4 * x + 1] = v.y; sq.qh[4 * x + 2] = v.z; sq.qh[4 * x + 3] = v.w;
            }
        }
        const float thr = (j < p.G) ? p.mtilde[head0 + j] - p.delta : -INFINITY;   // delta = +inf: all pass
        if (w == 0 && lane == 0) d.item = item;
        for (int lb = w; lb < it.nblk; lb += kNS) {
            // keep the ring full: blocks consumed .. consumed + kRing - 1 of this warp's stream
            while (issued < consumed + kRing && cursor_next(ic, p, ids, horizon, w)) {
                ring_issue(p, ic, ring + (issued % kRing) * kStageBytes, lane);
                ++issued;
            }
            const uint32_t stage = ring + (consumed % kRing) * kStageBytes;
            ring_wait(issued - consumed - 1);
            __syncwarp();
            ScanRegs sr;
#pragma unroll
            for (int mt = 0; mt < 4; ++mt) sr.w[mt] = lds128(stage + (mt * 32 + lane) * 16);
#pragma unroll
            for (int x = 0; x < 4; ++x) sr.s[x] = lds128(stage + kCodeBytes + (4 * j + x) * 16);
            __syncwarp();   // the stage is free again
            ++consumed;
            if (issued < consumed + kRing && cursor_next(ic, p, ids, horizon, w)) {
                ring_issue(p, ic, ring + (issued % kRing) * kStageBytes, lane);
                ++issued;
            }

            const int blk = it.blk0 + lb;
            const int page = page_of(p, it.b, blk);
            const int rows = min(kBlk, it.n - blk * kBlk);
            unsigned keep4 = 0;
            if (page >= 0) {
                float band;
                float bm = scan_compute<false>(sr, sq, lane, rows, p.sm_scale, band);
                // too close to call with the fast accumulation: redo with the arithmetic m_tilde was computed in
                if (__any_sync(kFull, (j < p.G) && fabsf(bm - thr) <= band))
                    bm = scan_compute<true>(sr, sq, lane, rows, p.sm_scale, band);
                const bool keep = (j < p.G) && (bm >= thr);
                keep4 = __ballot_sync(kFull, keep) & 0xFu;
                if (r == 0 && j < p.G) {
                    const size_t o = (head0 + j) * p.max_blocks + blk;
                    if (p.kept_mask) p.kept_mask[o] = keep ? 1 : 0;
                    if (p.block_max) p.block_max[o] = bm;
                }
            }
            if (lane == 0) {
                d.tile[lb] = page >= 0 ? (uint32_t)((size_t)page * p.Hkv + it.g) : 0u;
                d.keep4[lb] = (uint8_t)keep4;
                d.rows[lb] = (uint8_t)rows;
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(bars + slot * 8);   // this warp's share of the batch is published
    }
    cp_async_drain();
    if (*abort_flag && w == 0 && lane == 0) atomicOr(p.status, kDevTimeout);
}

// ---- attend role -------------------------------------------------------------------------------------------

// bits of the blocks of a published batch that attend warp `a` processes: every kNA-th kept block
__device__ __forceinline__ unsigned my_entries(const BatchDesc& d, int nblk, int a, int lane) {
    const unsigned kept = __ballot_sync(kFull, lane < nblk && d.keep4[lane] != 0);
    unsigned mine = 0;
    int rank = 0;
    for (unsigned m = kept; m; m &= m - 1, ++rank)
        if (rank % kNA == a) mine |= m & (0u - m);
    return mine;
}

__device__ __forceinline__ void attend_role(const DecodeParams& p, unsigned char* smem, int a, int lane) {
    const int r = lane >> 2, j = lane & 3;
    const uint32_t kslot = smem_u32(smem) + kOffSlots + a * 2 * kSlotBytes;
    const uint32_t vslot = kslot + kSlotBytes;
    const uint32_t bars = smem_u32(smem) + kOffBars;
    const uint32_t kbar = bars + (2 * kNB + 2 * a) * 8, vbar = kbar + 8;
    const BatchDesc* descs = reinterpret_cast<const BatchDesc*>(smem + kOffDesc);
    const uint4* kbase = reinterpret_cast<const uint4*>(p.k_cache);
    const uint4* vbase = reinterpret_cast<const uint4*>(p.v_cache);
    constexpr size_t kTileVec = kTileBytes / 16;
    const float logit_scale_log2 = p.sm_scale * kLog2e;

    uint32_t phase = 0;
    int issued_bi = -1, issued_lb = -1;   // block whose K/V copies are already in flight
    bool ok = true;
    AttendState st;
    for (int bi = 0; ok; ++bi) {
        const int slot = bi & 1, use = bi >> 1;
        if (!mbar_wait(bars + slot * 8, use & 1)) { ok = false; break; }
        const BatchDesc& d = descs[slot];
        const int item = d.item;
        if (item < 0) break;
        const Item it = decode_item(p, item);
        unsigned mine = my_entries(d, it.nblk, a, lane);
        const bool any = mine != 0;
        if (any) attend_setup(st, p.q + ((size_t)it.b * p.Hq + (size_t)it.g * p.G) * kD, p.G, lane);
        while (mine && ok) {
            const int lb = __ffs(mine) - 1;
            mine &= mine - 1;
            if (!(issued_bi == bi && issued_lb == lb)) {
                tile_copy_async(kslot, kbase + (size_t)d.tile[lb] * kTileVec, lane, kbar);
                tile_copy_async(vslot, vbase + (size_t)d.tile[lb] * kTileVec, lane, vbar);
            }
            // the next block this warp will attend: in this batch, else in the next one if it is already published
            const uint4 *next_k = nullptr, *next_v = nullptr;
            if (mine) {
                const int nlb = __ffs(mine) - 1;
                next_k = kbase + (size_t)d.tile[nlb] * kTileVec;
                next_v = vbase + (size_t)d.tile[nlb] * kTileVec;
                issued_bi = bi;
                issued_lb = nlb;
            } else {
                const int bi2 = bi + 1;
                if (mbar_test(bars + (bi2 & 1) * 8, (bi2 >> 1) & 1)) {
                    const BatchDesc& d2 = descs[bi2 & 1];
                    if (d2.item >= 0) {
                        const unsigned mine2 = my_entries(d2, decode_item(p, d2.item).nblk, a, lane);
                        if (mine2) {
                            const int nlb = __ffs(mine2) - 1;
                            next_k = kbase + (size_t)d2.tile[nlb] * kTileVec;
                            next_v = vbase + (size_t)d2.tile[nlb] * kTileVec;
                            issued_bi = bi2;
                            issued_lb = nlb;
                        }
                    }
                }
            }
            ok = attend_block(st, kslot, vslot, kbar, vbar, phase, next_k, next_v, lane, d.rows[lb], d.keep4[lb],
                              logit_scale_log2);
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(bars + (kNB + slot) * 8);   // done with this batch descriptor
        // this warp's partial (m, l, acc) of the item; heads in rows r < 4 (r + 4 holds the bf16 remainder sums)
        const size_t pslot = ((size_t)item * kNA + a) * kMaxG;
        if (any && ok) {
            float l = st.l;
            l += __shfl_xor_sync(kFull, l, 1);
            l += __shfl_xor_sync(kFull, l, 2);
#pragma unroll
            for (int nt = 0; nt < 16; ++nt) {
                st.acc[nt][0] += __shfl_xor_sync(kFull, st.acc[nt][0], 16);
                st.acc[nt][1] += __shfl_xor_sync(kFull, st.acc[nt][1], 16);
            }
            if (r < p.G) {
                if (j == 0) *reinterpret_cast<float2*>(p.fpart_ml + (pslot + r) * 2) = make_float2(st.m, l);
                float* dst = p.fpart_acc + (pslot + r) * kD;
                // O fragment (nt, column n) is channel 64*(nt/8) + 8n + nt%8: two runs of 16 floats per lane
#pragma unroll
                for (int hf = 0; hf < 2; ++hf)
#pragma unroll
                    for (int x = 0; x < 2; ++x) {
                        float* run = dst + 64 * hf + 8 * (2 * j + x);
                        *reinterpret_cast<float4*>(run) = make_float4(st.acc[8 * hf + 0][x], st.acc[8 * hf + 1][x],
                                                                      st.acc[8 * hf + 2][x], st.acc[8 * hf + 3][x]);
                        *reinterpret_cast<float4*>(run + 4) = make_float4(st.acc[8 * hf + 4][x], st.acc[8 * hf + 5][x],
                                                                          st.acc[8 * hf + 6][x], st.acc[8 * hf + 7][x]);
                    }
            }
        } else if (r < p.G && j == 0) {
            *reinterpret_cast<float2*>(p.fpart_ml + (pslot + r) * 2) = make_float2(-INFINITY, 0.f);
        }
    }
    cp_async_drain();
    if (!ok && lane == 0) atomicOr(p.status, kDevTimeout);
}

__global__ void __launch_bounds__(kFusedThreads, 1) fused_sparse_kernel(DecodeParams p) {
    extern __shared__ __align__(1024) unsigned char smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        const uint32_t bars = smem_u32(smem) + kOffBars;
        for (int s = 0; s < kNB; ++s) {
            mbar_init(bars + s * 8, kNS);             // full: one arrival per scan warp
            mbar_init(bars + (kNB + s) * 8, kNA);     // empty: one arrival per attend warp
        }
        for (int a = 0; a < 2 * kNA; ++a) mbar_init(bars + (2 * kNB + a) * 8, 32);
        reinterpret_cast<volatile int*>(smem + kOffIds)[4] = 0;   // abort flag
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    __syncthreads();
    if (warp < kNS) scan_role(p, smem, warp, lane);
    else attend_role(p, smem, warp - kNS, lane);
}

// ---- combine for the fused kernel's partials ---------------------------------------------------------------
// One CTA of 128 threads per (query head, sequence); partial e = (split, attend warp).
__global__ void __launch_bounds__(kD) fused_combine_kernel(DecodeParams p) {
    const int h = blockIdx.x, b = blockIdx.y, c = threadIdx.x;
    const size_t head = (size_t)b * p.Hq + h;
    const int g = h / p.G, hl = h % p.G;
    const int n = min(max(p.seq_lens[b], 0), p.max_blocks * kBlk);
    const int nsplit = ((n + kBlk - 1) / kBlk + kItemBlocks - 1) / kItemBlocks;
    const int units = p.batch * p.Hkv, bg = b * p.Hkv + g;
    const int entries = nsplit * kNA;
    __shared__ float wgt[kD];
    __shared__ float red[kD / 32];
    float M = -INFINITY, L = 0.f, acc = 0.f;
    // pass 1: global max over all partials
    for (int e = c; e < entries; e += kD) {
        const size_t slot = (((size_t)(e / kNA) * units + bg) * kNA + (e % kNA)) * kMaxG + hl;
        const float2 ml = *reinterpret_cast<const float2*>(p.fpart_ml + slot * 2);
        if (ml.y > 0.f) M = fmaxf(M, ml.x);
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) M = fmaxf(M, __shfl_xor_sync(kFull, M, o));
    if ((c & 31) == 0) red[c >> 5] = M;
    __syncthreads();
    M = fmaxf(fmaxf(red[0], red[1]), fmaxf(red[2], red[3]));
    // pass 2: weights in chunks of 128 partials, then the weighted sum of their accumulators
    for (int base = 0; base < entries && M != -INFINITY; base += kD) {
        __syncthreads();
        const int e = base + c;
        float wv = 0.f;
        if (e < entries) {
            const size_t slot = (((size_t)(e / kNA) * units + bg) * kNA + (e % kNA)) * kMaxG + hl;
            const float2 ml = *reinterpret_cast<const float2*>(p.fpart_ml + slot * 2);
            if (ml.y > 0.f) {
                wv = exp2f(ml.x - M);
                L += wv * ml.y;
            }
        }
        wgt[c] = wv;
        __syncthreads();
        const int cnt = min(kD, entries - base);
        for (int x0 = 0; x0 < cnt; x0 += 8) {   // eight independent (predicated) loads in flight per thread
            float v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int x = x0 + u;
                const int e2 = base + x;
                const size_t slot = (((size_t)(e2 / kNA) * units + bg) * kNA + (e2 % kNA)) * kMaxG + hl;
                v[u] = (x < cnt && wgt[x] != 0.f) ? p.fpart_acc[slot * kD + c] : 0.f;
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) acc += (x0 + u < cnt ? wgt[x0 + u] : 0.f) * v[u];
        }
    }
    // total L: every thread holds the share of the partials it weighted
#pragma unroll
    for (int o = 16; o; o >>= 1) L += __shfl_xor_sync(kFull, L, o);
    __syncthreads();
    if ((c & 31) == 0) red[c >> 5] = L;
    __syncthreads();
    L = red[0] + red[1] + red[2] + red[3];
    const float o = L > 0.f ? acc / L : 0.f;
    if (p.out_fp32) reinterpret_cast<float*>(p.out)[head * kD + c] = o;
    else reinterpret_cast<__nv_bfloat16*>(p.out)[head * kD + c] = __float2bfloat16_rn(o);
    if (p.lse && c == 0) p.lse[head] = L > 0.f ? (M + log2f(L)) * kLn2 : -INFINITY;
}

}  // namespace ffd
