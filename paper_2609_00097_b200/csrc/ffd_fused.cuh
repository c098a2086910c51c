// The fused sparse kernel: scan -> top-delta select -> exact attention over kept blocks, in one persistent launch.
//
// One CTA per SM, 16 warps in two roles that run concurrently (register budgets set with setmaxnreg):
//   12 scan warps   stream the 2-bit codes and scales of every block through a private 3-stage cp.async ring
//                   (3 blocks = 6.9 KB in flight per warp), compute the block maxima of the approximate scores
//                   on the tensor cores and publish the keep decisions of one work item in a batch descriptor;
//   4 attend warps  take the kept blocks of a published batch, stage their K and V tiles (16 KB each) through
//                   private swizzled slots with cp.async + mbarrier and run the exact online-softmax attention.
// A work item is 24 consecutive blocks of one (sequence, KV head).  Items are handed out dynamically: lane 0 of scan
// warp 0 draws item numbers from a global counter (the atomic for the next draw is always in flight, so its latency
// is not waited for), skips items without blocks, decodes the item once and publishes it two items ahead in a tagged
// ring in shared memory; it also starts the copy of the item's query record (pre-scaled fp16 query fragments +
// thresholds, written by the pseudo-max kernel).  Readers check the tag; nobody divides or reloads sequence
// lengths on the per-block path.  Scan warps run up to two batches ahead of the attend warps (two descriptors,
// full/empty mbarriers), which also keeps all scan warps within one batch of each other.
// Every wait is bounded; on expiry the warp records kDevTimeout and the CTA winds down.
#pragma once
#include "ffd_kernels.cuh"

namespace ffd {

constexpr int kNS = 12;                // scan warps (three warpgroups)
constexpr int kNA = 4;                 // attend warps (one warpgroup)
constexpr int kFusedThreads = (kNS + kNA) * 32;
constexpr int kScanRegs = 112;         // 12*32*112 + 4*32*176 = 65536 registers
constexpr int kAttendRegs = (65536 - kNS * 32 * kScanRegs) / (kNA * 32);
static_assert(kAttendRegs % 8 == 0 && kScanRegs % 8 == 0, "setmaxnreg takes multiples of 8");
constexpr int kItemBlocks = 24;        // blocks per work item: two per scan warp
constexpr int kRing = 3;               // code-ring stages per scan warp
constexpr int kStageBytes = kCodeBytes + kD * 2;   // 2048 B codes + 256 B scales
constexpr int kNB = 2;                 // batch descriptors in flight
constexpr int kItemRing = 8;           // decoded items published ahead
constexpr int kQrecRing = 4;           // query records staged ahead
constexpr int kQrecBytes = 2048 + 32;  // [4][32 lanes] uint4 of fp16 query fragments, then 4 thresholds (+ pad)

struct Item {
    int item;                          // work item number; < 0: no more work
    int b, g, blk0, nblk, n;           // sequence, KV head, first block, blocks (1..24), tokens of the sequence
};

struct ItemSlot {                      // entry `seq` of the published-item ring is valid when tag == seq
    volatile int tag;
    volatile int item, b, g, blk0, nblk, n;
    int pad;
};

struct BatchDesc {
    int item, b, g, nblk;              // work item of this batch; item < 0: no more work
    uint32_t tile[kItemBlocks];        // (page, KV head) tile of each block of the item
    uint8_t keep4[kItemBlocks];        // bit h: query head h of the group keeps the block; 0 = skipped
    uint8_t rows[kItemBlocks];         // valid tokens
};

constexpr int kOffSlots = 0;
constexpr int kOffRing = kOffSlots + kNA * 2 * kSlotBytes;
constexpr int kOffQrec = kOffRing + kNS * kRing * kStageBytes;
constexpr int kOffDesc = kOffQrec + kQrecRing * kQrecBytes;
constexpr int kOffBars = kOffDesc + kNB * (int)sizeof(BatchDesc);
constexpr int kNumBars = 2 * kNB + 2 * kNA + kQrecRing;          // full, empty, K/V slots, query records
constexpr int kOffItems = kOffBars + kNumBars * 8;               // ring of decoded items
constexpr int kOffStageTile = kOffItems + kItemRing * (int)sizeof(ItemSlot);   // tile index of each ring stage
constexpr int kOffAbort = kOffStageTile + kNS * 4 * 4;
constexpr int kFusedSmem = kOffAbort + 16;
static_assert(kOffBars % 8 == 0 && kOffRing % 16 == 0 && kOffDesc % 16 == 0 && kOffQrec % 16 == 0, "alignment");
static_assert(sizeof(BatchDesc) % 16 == 0 && sizeof(ItemSlot) == 32, "descriptor sizes");
static_assert(kFusedSmem <= 227 * 1024, "shared memory budget");

// Items are numbered from the END of the sequences backwards: the local window, whose blocks are the most likely
// to be kept (and therefore the most expensive), is handed out first.
__device__ __forceinline__ Item decode_item(const DecodeParams& p, int item) {
    Item it;
    const int units = p.batch * p.Hkv;
    const int bg = item % units, split = p.total_items / units - 1 - item / units;
    it.item = item;
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

// ---- published items ---------------------------------------------------------------------------------------

__device__ __forceinline__ bool item_ready(const ItemSlot* ring, int seq) { return ring[seq & (kItemRing - 1)].tag == seq; }

__device__ __forceinline__ Item item_read(const ItemSlot* ring, int seq) {
    const ItemSlot& e = ring[seq & (kItemRing - 1)];
    __threadfence_block();
    Item it;
    it.item = e.item; it.b = e.b; it.g = e.g; it.blk0 = e.blk0; it.nblk = e.nblk; it.n = e.n;
    return it;
}

// bounded wait for entry `seq` (it is normally there long before it is needed)
__device__ __forceinline__ bool item_wait(const ItemSlot* ring, int seq) {
    if (item_ready(ring, seq)) return true;
    const long long t0 = clock64();
    while (!item_ready(ring, seq)) {
        __nanosleep(64);
        if (clock64() - t0 > kSpinCycles) return false;
    }
    return true;
}

// Lane 0 of scan warp 0: draw the next item that has blocks and publish it as entry `seq`.
// `pend` holds the result of an atomicAdd issued earlier; `done` is set once the counter ran past the last item.
__device__ __forceinline__ Item item_publish(const DecodeParams& p, ItemSlot* ring, int seq, int& pend, bool& done) {
    Item it;
    it.item = -1; it.b = it.g = it.blk0 = it.nblk = it.n = 0;
    while (!done) {
        const int cand = pend;
        if (cand >= p.total_items) { done = true; break; }
        pend = (int)atomicAdd(p.item_counter, 1u);   // keep the next draw in flight
        const Item c = decode_item(p, cand);
        if (c.nblk > 0) { it = c; break; }
    }
    ItemSlot& e = ring[seq & (kItemRing - 1)];
    e.item = it.item; e.b = it.b; e.g = it.g; e.blk0 = it.blk0; e.nblk = it.nblk; e.n = it.n;
    __threadfence_block();
    e.tag = seq;
    return it;
}

// ---- scan role ---------------------------------------------------------------------------------------------

// Position of a scan warp in its stream of blocks: published item after published item, local blocks w and w + 12.
struct ScanCursor {
    int seq;       // published item the cursor is in (-1 before the first)
    Item it;
    int lb;
    bool end;      // ran into the end of the work
};

// Advance to this warp's next block; false when the item it lies in has not been published yet (the cursor then
// stays where it can resume) or when there is no more work.
__device__ __forceinline__ bool cursor_next(ScanCursor& c, const ItemSlot* items, int w) {
    if (c.end) return false;
    int lb = c.lb + kNS;
    while (lb >= c.it.nblk) {
        if (!item_ready(items, c.seq + 1)) { c.lb = lb - kNS; return false; }
        c.it = item_read(items, c.seq + 1);
        ++c.seq;
        if (c.it.item < 0) { c.end = true; c.it.nblk = 0; return false; }
        lb = w;
    }
    c.lb = lb;
    return true;
}

// start the copy of one block's codes + scales into a ring stage (one commit group); remembers the block's tile
__device__ __forceinline__ void ring_issue(const DecodeParams& p, const ScanCursor& c, uint32_t stage,
                                           volatile int* stage_tile, int lane) {
    const int page = page_of(p, c.it.b, c.it.blk0 + c.lb);
    const int tile = page >= 0 ? page * p.Hkv + c.it.g : -1;
    if (tile >= 0) {
        const uint4* codes = reinterpret_cast<const uint4*>(p.k_quant + (size_t)tile * kCodeBytes);
#pragma unroll
        for (int x = 0; x < 4; ++x) cp_async16(stage + (x * 32 + lane) * 16, codes + x * 32 + lane);
        // scales: 16-byte chunk 4j + x lands at position 4x + j, so the four chunks read together are adjacent
        if (lane < 16)
            cp_async16(stage + kCodeBytes + ((lane & 3) * 4 + (lane >> 2)) * 16,
                       reinterpret_cast<const uint4*>(p.k_scales + (size_t)tile * kD) + lane);
    }
    if (lane == 0) *stage_tile = tile;
    asm volatile("cp.async.commit_group;\n" ::: "memory");
}

__device__ __forceinline__ void ring_wait(int younger) {
    if (younger >= 2) asm volatile("cp.async.wait_group 2;\n" ::: "memory");
    else if (younger == 1) asm volatile("cp.async.wait_group 1;\n" ::: "memory");
    else asm volatile("cp.async.wait_group 0;\n" ::: "memory");
}

// Warp 0 only: copy the query record of published item `seq` into slot seq % 4 of the record ring and report
// completion on that slot's mbarrier.  Every scan warp waits for every record, in order, so a parity wait can
// never see a stale phase.
__device__ __forceinline__ void qrec_issue(const DecodeParams& p, int seq, int bg, uint32_t qrecs, uint32_t qbars,
                                           int lane) {
    const int slot = seq & (kQrecRing - 1);
    const uint4* src = reinterpret_cast<const uint4*>(p.qrec + (size_t)bg * kQrecBytes);
    for (int c = lane; c < kQrecBytes / 16; c += 32) cp_async16(qrecs + slot * kQrecBytes + c * 16, src + c);
    cp_async_arrive(qbars + slot * 8);
}

// The precise variant of the scan for one block, with the arithmetic m_tilde was computed in.  Kept out of line so
// that its registers do not weigh on the fast path; it re-reads the block's codes and scales from global memory.
__device__ __noinline__ float scan_block_precise(const uint4* codes_tile, const uint4* scales_tile, uint32_t qrec,
                                                 int lane, int rows, float sm_scale) {
    ScanRegs sr;
    scan_load(sr, codes_tile, scales_tile, lane);
    ScanQuery sq;
    sq.piece = (lane >> 2) & 1;
#pragma unroll
    for (int x = 0; x < 4; ++x) {
        const uint4 v = lds128(qrec + (x * 32 + lane) * 16);
        sq.qh[4 * x] = v.x; sq.qh[4 * x + 1] = v.y; sq.qh[4 * x + 2] = v.z; sq.qh[4 * x + 3] = v.w;
    }
    float band;
    return scan_compute<true>(sr, sq, lane, rows, sm_scale, band);
}

__device__ __forceinline__ void scan_role(const DecodeParams& p, unsigned char* smem, int w, int lane) {
    const int r = lane >> 2, j = lane & 3;
    const uint32_t ring = smem_u32(smem) + kOffRing + w * kRing * kStageBytes;
    const uint32_t qrecs = smem_u32(smem) + kOffQrec;
    const uint32_t bars = smem_u32(smem) + kOffBars;
    const uint32_t qbars = bars + (2 * kNB + 2 * kNA) * 8;
    BatchDesc* descs = reinterpret_cast<BatchDesc*>(smem + kOffDesc);
    ItemSlot* items = reinterpret_cast<ItemSlot*>(smem + kOffItems);
    volatile int* stage_tile = reinterpret_cast<volatile int*>(smem + kOffStageTile) + w * 4;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kOffAbort);
    const int units = p.batch * p.Hkv;

    // warp 0 publishes items 0 and 1 (and stages their records) before anybody starts
    int pend = p.total_items;
    bool done = false;
    if (w == 0) {
        int item0 = -1, item1 = -1;
        if (lane == 0) {
            pend = (int)atomicAdd(p.item_counter, 1u);
            item0 = item_publish(p, items, 0, pend, done).item;
            item1 = item_publish(p, items, 1, pend, done).item;
        }
        item0 = __shfl_sync(kFull, item0, 0);
        item1 = __shfl_sync(kFull, item1, 0);
        if (item0 >= 0) qrec_issue(p, 0, item0 % units, qrecs, qbars, lane);
        if (item1 >= 0) qrec_issue(p, 1, item1 % units, qrecs, qbars, lane);
    }
    ScanCursor ic;
    ic.seq = -1;
    ic.it.nblk = 0;
    ic.lb = w - kNS;
    ic.end = false;
    int issued = 0, consumed = 0;   // this warp's blocks whose copies were started / whose data was taken

#pragma unroll 1
    for (int seq = 0;; ++seq) {     // published item seq = batch seq
        if (w == 0) {               // publish item seq + 2 and stage its record
            int item2 = -1;
            if (lane == 0) item2 = item_publish(p, items, seq + 2, pend, done).item;
            item2 = __shfl_sync(kFull, item2, 0);
            if (item2 >= 0) qrec_issue(p, seq + 2, item2 % units, qrecs, qbars, lane);
        }
        if (!item_wait(items, seq)) *abort_flag = 1;
        const Item it = item_read(items, seq);
        const int slot = seq & 1, use = seq >> 1;
        // the attend warps must have released this descriptor (two batches ago)
        if (use > 0 && !mbar_wait(bars + (kNB + slot) * 8, (use - 1) & 1)) *abort_flag = 1;
        BatchDesc& d = descs[slot];
        if (it.item < 0 || *abort_flag) {   // no more work: tell the attend warps
            if (lane == 0) {
                if (w == 0) d.item = -1;
                mbar_arrive(bars + slot * 8);
            }
            break;
        }
        // the item's query record must have landed
        if (!mbar_wait(qbars + (seq & (kQrecRing - 1)) * 8, (seq / kQrecRing) & 1)) *abort_flag = 1;
        const uint32_t qrec = qrecs + (seq & (kQrecRing - 1)) * kQrecBytes;
        const size_t head0 = (size_t)it.b * p.Hq + (size_t)it.g * p.G;
        float thr;
        asm volatile("ld.shared.f32 %0, [%1];\n" : "=f"(thr) : "r"(qrec + 2048 + j * 4));
        if (w == 0 && lane == 0) { d.item = it.item; d.b = it.b; d.g = it.g; d.nblk = it.nblk; }
#pragma unroll 1
        for (int lb = w; lb < it.nblk; lb += kNS) {
            // keep the ring full: blocks consumed .. consumed + kRing - 1 of this warp's stream
            while (issued < consumed + kRing && cursor_next(ic, items, w)) {
                ring_issue(p, ic, ring + (issued % kRing) * kStageBytes, stage_tile + issued % kRing, lane);
                ++issued;
            }
            const int st = consumed % kRing;
            const uint32_t stage = ring + st * kStageBytes;
            ring_wait(issued - consumed - 1);
            __syncwarp();
            // codes into registers; B operand straight from the staged scales and the item's query record
            uint4 wv[4];
#pragma unroll
            for (int mt = 0; mt < 4; ++mt) wv[mt] = lds128(stage + (mt * 32 + lane) * 16);
            uint32_t bfrag[16];
#pragma unroll
            for (int x = 0; x < 4; ++x)
                scan_bfrag4(bfrag + 4 * x, lds128(qrec + (x * 32 + lane) * 16),
                            lds128(stage + kCodeBytes + (4 * x + j) * 16), r & 1);
            const int tile = stage_tile[st];
            __syncwarp();   // the stage is free again
            ++consumed;
            if (issued < consumed + kRing && cursor_next(ic, items, w)) {
                ring_issue(p, ic, ring + (issued % kRing) * kStageBytes, stage_tile + issued % kRing, lane);
                ++issued;
            }

            const int blk = it.blk0 + lb;
            const int rows = min(kBlk, it.n - blk * kBlk);
            unsigned keep4 = 0;
            if (tile >= 0) {
                float band;
                float bm = scan_mma<false>(wv, bfrag, lane, rows, p.sm_scale, band);
                // too close to call (rare): a separate, non-inlined routine re-reads the block and redoes it precisely
                if (__any_sync(kFull, (j < p.G) && fabsf(bm - thr) <= band))
                    bm = scan_block_precise(reinterpret_cast<const uint4*>(p.k_quant + (size_t)tile * kCodeBytes),
                                            reinterpret_cast<const uint4*>(p.k_scales + (size_t)tile * kD), qrec, lane,
                                            rows, p.sm_scale);
                const bool keep = (j < p.G) && (bm >= thr);
                keep4 = __ballot_sync(kFull, keep) & 0xFu;
                if (r == 0 && j < p.G) {
                    const size_t o = (head0 + j) * p.max_blocks + blk;
                    if (p.kept_mask) p.kept_mask[o] = keep ? 1 : 0;
                    if (p.block_max) p.block_max[o] = bm;
                }
            }
            if (lane == 0) {
                d.tile[lb] = tile >= 0 ? (uint32_t)tile : 0u;
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
        Item it;
        it.item = item; it.b = d.b; it.g = d.g; it.nblk = d.nblk;
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
                        const unsigned mine2 = my_entries(d2, d2.nblk, a, lane);
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
        for (int a = 0; a < 2 * kNA + kQrecRing; ++a) mbar_init(bars + (2 * kNB + a) * 8, 32);
        for (int s = 0; s < kItemRing; ++s) reinterpret_cast<ItemSlot*>(smem + kOffItems)[s].tag = -1;
        *reinterpret_cast<volatile int*>(smem + kOffAbort) = 0;
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    __syncthreads();
    if (warp < kNS) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;\n" ::"n"(kScanRegs));
        scan_role(p, smem, warp, lane);
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;\n" ::"n"(kAttendRegs));
        attend_role(p, smem, warp - kNS, lane);
    }
}

// ---- split combine (FlashDecoding-style log-sum-exp merge) -------------------------------------------------
// One CTA of 1024 threads per (query head, sequence).  FUSED: partial e = (work item, attend warp) of the fused
// kernel; otherwise partial e = split of the dense kernel.  The (m, l) pairs are read once into shared memory;
// thread (el, cg) = (tid / 32, tid % 32) sums the partials e = el, el + 32, ... for channels 4cg .. 4cg+3 with
// eight independent loads in flight; the 32 partial sums meet in shared memory.  Summation order is fixed, so
// results are reproducible.
constexpr int kCombineThreads = 1024;
constexpr int kCombineLanes = kCombineThreads / 32;   // partials summed side by side
constexpr int kCombineChunk = 1024;

template <bool FUSED>
__device__ __forceinline__ size_t combine_slot(const DecodeParams& p, size_t head, int bg, int hl, int e) {
    if (FUSED) {   // item number of split e / kNA (see decode_item), then the attend warp
        const int units = p.batch * p.Hkv;
        const int item = (p.total_items / units - 1 - e / kNA) * units + bg;
        return ((size_t)item * kNA + (e % kNA)) * kMaxG + hl;
    }
    return head * p.splits + e;
}

template <bool FUSED>
__global__ void __launch_bounds__(kCombineThreads) combine_kernel(DecodeParams p) {
    const int h = blockIdx.x, b = blockIdx.y, tid = threadIdx.x;
    const int el = tid >> 5, cg = tid & 31;
    const size_t head = (size_t)b * p.Hq + h;
    const int g = h / p.G, hl = h % p.G, bg = b * p.Hkv + g;
    const int n = min(max(p.seq_lens[b], 0), p.max_blocks * kBlk);
    const int nb = (n + kBlk - 1) / kBlk;
    const int entries = FUSED ? ((nb + kItemBlocks - 1) / kItemBlocks) * kNA
                              : min((nb + p.blocks_per_split - 1) / p.blocks_per_split, p.splits);
    const float* ml = FUSED ? p.fpart_ml : p.part_ml;
    const float* pacc = FUSED ? p.fpart_acc : p.part_acc;
    __shared__ float s_m[kCombineChunk];   // m of the partial, then its weight
    __shared__ float s_l[kCombineChunk];
    __shared__ float s_red[kCombineLanes];
    __shared__ float4 s_part[kCombineLanes][32];

    float Mrun = -INFINITY, L = 0.f;       // running max / sum across chunks (one chunk unless > 1024 partials)
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int base = 0; base < entries; base += kCombineChunk) {
        const int cnt = min(kCombineChunk, entries - base);
        __syncthreads();
        float M = -INFINITY;
        for (int x = tid; x < cnt; x += kCombineThreads) {
            const float2 v = *reinterpret_cast<const float2*>(ml + combine_slot<FUSED>(p, head, bg, hl, base + x) * 2);
            s_m[x] = v.y > 0.f ? v.x : -INFINITY;
            s_l[x] = v.y;
            M = fmaxf(M, s_m[x]);
        }
#pragma unroll
        for (int o = 16; o; o >>= 1) M = fmaxf(M, __shfl_xor_sync(kFull, M, o));
        if (cg == 0) s_red[el] = M;
        __syncthreads();
        M = Mrun;
#pragma unroll
        for (int x = 0; x < kCombineLanes; ++x) M = fmaxf(M, s_red[x]);
        if (M == -INFINITY) continue;      // uniform: nothing in this chunk or before it
        const float rescale = exp2f(Mrun - M);   // 0 for the first non-empty chunk
        acc.x *= rescale; acc.y *= rescale; acc.z *= rescale; acc.w *= rescale;
        L *= rescale;
        Mrun = M;
        for (int x = tid; x < cnt; x += kCombineThreads) {
            const float wv = exp2f(s_m[x] - M);  // exp2(-inf) = 0 for empty partials
            L += wv * s_l[x];
            s_m[x] = wv;
        }
        __syncthreads();
        for (int x0 = el; x0 < cnt; x0 += kCombineLanes * 8) {
            float4 v[8];
            float wv[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int x = x0 + kCombineLanes * u;
                wv[u] = x < cnt ? s_m[x] : 0.f;
                v[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (wv[u] != 0.f)
                    v[u] = *reinterpret_cast<const float4*>(pacc + combine_slot<FUSED>(p, head, bg, hl, base + x) * kD +
                                                            4 * cg);
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                acc.x += wv[u] * v[u].x; acc.y += wv[u] * v[u].y; acc.z += wv[u] * v[u].z; acc.w += wv[u] * v[u].w;
            }
        }
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) L += __shfl_xor_sync(kFull, L, o);
    __syncthreads();
    if (cg == 0) s_red[el] = L;
    s_part[el][cg] = acc;
    __syncthreads();
    if (tid < 32) {
        L = 0.f;
        float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int x = 0; x < kCombineLanes; ++x) {
            L += s_red[x];
            const float4 v = s_part[x][tid];
            t.x += v.x; t.y += v.y; t.z += v.z; t.w += v.w;
        }
        const float inv = L > 0.f ? 1.f / L : 0.f;
        const float4 o = make_float4(t.x * inv, t.y * inv, t.z * inv, t.w * inv);
        if (p.out_fp32) {
            reinterpret_cast<float4*>(p.out)[head * (kD / 4) + tid] = o;
        } else {
            __nv_bfloat162 lo = __floats2bfloat162_rn(o.x, o.y), hi = __floats2bfloat162_rn(o.z, o.w);
            uint2 pk;
            pk.x = *reinterpret_cast<uint32_t*>(&lo);
            pk.y = *reinterpret_cast<uint32_t*>(&hi);
            reinterpret_cast<uint2*>(p.out)[head * (kD / 4) + tid] = pk;
        }
        if (p.lse && tid == 0) p.lse[head] = L > 0.f ? (Mrun + log2f(L)) * kLn2 : -INFINITY;
    }
}

}  // namespace ffd
