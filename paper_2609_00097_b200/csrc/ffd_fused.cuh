// The fused sparse kernel: scan -> top-delta select -> exact attention over kept blocks, in one persistent launch.
//
// One CTA per SM, 16 warps in three jobs that run concurrently (register budgets set with setmaxnreg):
//   1 scheduling warp  (warp 0) draws work items from two global counters, decodes them once and publishes them up to
//                      four entries ahead in a ring in shared memory (one mbarrier per entry) together with the
//                      item's page-table entries and the header of its batch descriptor; it also starts the copy
//                      of the item's query record (pre-scaled fp16 query fragments, |q| fragments and thresholds,
//                      written by the pseudo-max kernel).  The atomic for the next draw of each class is always in
//                      flight.
//   11 scan warps      stream the 2-bit codes and scales of every block through a private 2-stage cp.async ring,
//                      bound the block's scores from its scales alone and, unless that already rules the block out,
//                      compute the block maxima of the approximate scores on the tensor cores; they publish the
//                      keep decisions of one work item in a batch descriptor.
//   4 attend warps     take the kept blocks of a published batch, stage their K and V tiles (16 KB each) through
//                      private swizzled slots with cp.async + mbarrier and run the exact online-softmax attention.
// A work item is 32 consecutive blocks of one (sequence, KV head), two or three per scan warp (11 for the small items
// at the start of a sequence, which are handed out last).  Scan warps may run up to eight batches ahead of the attend
// warps (eight descriptors, full/empty mbarriers).  Units that the pseudo-max kernel's
// hint marks as dense ("heavy") are scheduled so that at most a few heavy batches are outstanding per CTA and the
// scan warps' spare time goes to light items (see ItemSched).
// Nobody divides or reloads sequence lengths on the per-block path.  Every wait is bounded; on expiry the warp
// records kDevTimeout and the CTA winds down.
#pragma once
#include "ffd_kernels.cuh"

namespace ffd {

constexpr int kNS = 12;                // warps of the scheduling + scan roles (three warpgroups)
constexpr int kSched = 1;              // warp 0 only draws and publishes items, warps 1..11 scan
constexpr int kScanners = kNS - kSched;
static_assert(kSched == 1, "warp 0 schedules, warps 1 .. kNS - 1 scan");
constexpr int kNA = 4;                 // attend warps (one warpgroup)
constexpr int kFusedThreads = (kNS + kNA) * 32;
constexpr int kScanRegs = 112;         // 12*32*112 + 4*32*176 = 65536 registers
constexpr int kAttendRegs = (65536 - kNS * 32 * kScanRegs) / (kNA * 32);
static_assert(kAttendRegs % 8 == 0 && kScanRegs % 8 == 0, "setmaxnreg takes multiples of 8");
// Blocks per full work item: 32 — as many as the one-lane-per-block ballots allow — when the launch has plenty of
// items per SM, else 22.  Every batch costs its scan warps a round of waits (item, query record, ring refill), so
// big batches are cheaper per block (C5: 9 % faster with 32 than with 22); but with only a few items per SM the
// coarser items leave the SMs unevenly loaded (C3 at context 32768: 10 % slower).  Scan warp w takes blocks w,
// w + 11, w + 22.
constexpr int kItemBlocksMax = 32;
constexpr int kItemBlocksMin = 2 * kScanners;
static_assert(kItemBlocksMax <= 32, "batch descriptor arrays; one lane per block in the ballots");
// The sequence is cut into items from block 0 upwards: first rows_small small items (one block per scanning
// warp), then full items.  Items are drawn from the sequence END backwards, so the small ones are drawn last and
// the CTAs run out of work within a small item's time of each other.
constexpr int kSmallBlocks = kScanners;

struct ItemGeom { int rows_small, item_rows, item_blocks; };

// pure function of the launch geometry and the GPU's SM count (the workspace layout depends on it)
__host__ __device__ inline ItemGeom item_geometry(long units, int max_blocks, int sms) {
    ItemGeom g;
    g.item_blocks = units * ((max_blocks + kItemBlocksMax - 1) / kItemBlocksMax) >= 6 * sms ? kItemBlocksMax : kItemBlocksMin;
    const int kItemBlocks = g.item_blocks;
    const int full_rows = (max_blocks + kItemBlocks - 1) / kItemBlocks;
    const int all_small = (max_blocks + kSmallBlocks - 1) / kSmallBlocks;
    if (units * full_rows < 2 * sms) {
        g.rows_small = all_small;        // few items per SM: halve them all
    } else {
        const long want = (6 * sms + units - 1) / units;             // about three small heavy items per SM
        const long cap = all_small / 3;                              // at most a third of the blocks
        g.rows_small = (int)(want < cap ? want : cap);
    }
    const int rest = max_blocks - g.rows_small * kSmallBlocks;
    g.item_rows = g.rows_small + (rest > 0 ? (rest + kItemBlocks - 1) / kItemBlocks : 0);
    return g;
}

// item number idx of a sequence, counted from block 0: first block and capacity
__device__ __forceinline__ void item_span(const DecodeParams& p, int idx, int& blk0, int& cap) {
    if (idx < p.rows_small) { blk0 = idx * kSmallBlocks; cap = kSmallBlocks; }
    else { blk0 = p.rows_small * kSmallBlocks + (idx - p.rows_small) * p.item_blocks; cap = p.item_blocks; }
}

// items a sequence of nb blocks is cut into
__device__ __forceinline__ int item_count(const DecodeParams& p, int nb) {
    const int s = p.rows_small * kSmallBlocks;
    return nb <= s ? (nb + kSmallBlocks - 1) / kSmallBlocks : p.rows_small + (nb - s + p.item_blocks - 1) / p.item_blocks;
}
constexpr int kRing = 2;               // code-ring stages per scan warp (a third stage measured no faster)
constexpr int kStageBytes = kCodeBytes + kD * 2;   // 2048 B codes + 256 B scales
constexpr int kNB = 8;                 // batch descriptors: how far the scan warps may run ahead of the attend warps
constexpr int kHeavyAhead = 2;         // heavy batches outstanding at most once the attend warps are the bottleneck
constexpr int kUnitCache = 512;        // entries of each end of the unit list kept in shared memory
constexpr int kRowCap = 512;           // item rows up to which the table of existing items is built (ragged batches)
constexpr int kItemRing = 8;           // decoded items published ahead
constexpr int kQrecRing = 4;           // query records staged ahead
constexpr int kQrecAbs = 2048;         // query record: [4][32 lanes] uint4 of pre-scaled fp16 query fragments, ...
constexpr int kQrecThr = 4096;         // ... the same fragments of |q| (not pre-scaled), then per head (4 floats each): the
                                       // threshold, the accumulator unit, the bound's multiplier and its slack
constexpr int kQrecBytes = kQrecThr + 64;

struct Item {
    int slot;                          // canonical number row * units + bg (names the partial slots); < 0: no more work
    int b, g, bg, blk0, nblk, n;       // sequence, KV head, b * Hkv + g, first block, blocks (1..24), tokens
};

struct ItemSlot {                      // entry seq % 8 of the published-item ring; readiness: one mbarrier per entry
    volatile int slot, b, g, bg, blk0, nblk, n;
    int pad;
    volatile int pages[32];            // physical page of each block of the item (-1: bad page-table entry)
};

struct BatchDesc {
    int item, b, g, nblk;              // canonical item number (row * units + bg) of this batch; < 0: no more work
    uint32_t tile[32];                 // (page, KV head) tile of each block of the item (at most kItemBlocksMax used)
    uint8_t keep4[32];                 // bit h: query head h of the group keeps the block; 0 = skipped
    uint8_t rows[32];                  // valid tokens
};

constexpr int kOffSlots = 0;
constexpr int kOffRing = kOffSlots + kNA * 2 * kSlotBytes;
constexpr int kOffQrec = kOffRing + kScanners * kRing * kStageBytes;
constexpr int kOffDesc = kOffQrec + kQrecRing * kQrecBytes;
constexpr int kOffBars = kOffDesc + kNB * (int)sizeof(BatchDesc);
constexpr int kNumBars = 2 * kNB + 2 * kNA + kQrecRing + kItemRing;   // full, empty, K/V slots, records, items
constexpr int kOffItems = kOffBars + kNumBars * 8;               // ring of decoded items
constexpr int kOffStageTile = kOffItems + kItemRing * (int)sizeof(ItemSlot);   // tile index of each ring stage
constexpr int kOffAbort = kOffStageTile + kNS * 4 * 4;
constexpr int kOffAttendDone = kOffAbort + 16;                   // batches finished by each attend warp
constexpr int kOffUnits = kOffAttendDone + 16;                   // first kUnitCache entries of each end of the unit list
constexpr int kOffStart = kOffUnits + 2 * kUnitCache * 8;        // first row (16 bit) in which each cached unit has an item
constexpr int kOffRowPref = kOffStart + 2 * kUnitCache * 2;      // per class: draws before each row, then the total
constexpr int kFusedSmem = kOffRowPref + 2 * (kRowCap + 1) * 4;
static_assert(kOffBars % 8 == 0 && kOffRing % 16 == 0 && kOffDesc % 16 == 0 && kOffQrec % 16 == 0, "alignment");
static_assert(sizeof(BatchDesc) % 16 == 0 && sizeof(ItemSlot) == 160, "descriptor sizes");
static_assert(kFusedSmem <= 227 * 1024, "shared memory budget");

// Work is handed out from two global counters, one per class of (sequence, KV head) units.  "Heavy" units are the
// ones the pseudo-max kernel's hint expects to keep most of their blocks (expensive for the attend warps, memory
// bound), "light" units the rest (almost pure scan work).  The drawing thread keeps at most kHeavyAhead heavy batches
// queued ahead of the attend warps and fills the scan warps' remaining time with light items, so the two kinds of
// work overlap on every SM.  Within a class,
// rows count from the END of the sequences backwards (the local window first, the small items last).
struct ItemSched {                                        // lives in the registers of the scheduling warp's lane 0
    int n_heavy, n_light, total_heavy, total_light;      // units and items per class
    unsigned long long magic_heavy, magic_light;          // reciprocals of the unit counts
    int row_off;                                          // leading rows that no sequence of the batch reaches
    int table;                                            // 1: draws go through the row tables (see plan_tables)
    int pend_heavy, pend_light;                           // draw of each class already fetched (>= total: none left)
    int released;                                         // batches the attend warps have finished, in order
    int heavy_queued;                                     // heavy batches published and not yet released
    unsigned long long heavy_hist;                        // bit s % 64: batch s is heavy
};

// Row tables for batches whose sequences differ much in length.  A sequence shorter than the longest one has no
// item in the first rows; when more than half of the (row, unit) grid is empty (and the batch fits: kUnitCache
// units per class, kRowCap rows) the scheduling warp builds, per class, the number of draws before each row
// counting only items that exist, so that no ticket is spent on a missing item.  Kept out of line: the scheduling
// loop of the common case stays small.
__device__ __noinline__ int2 plan_tables(int units, int rows_small, int item_blocks, unsigned char* smem, int n_heavy,
                                         int rows, int lane) {
    int total_heavy = 0, total_light = 0;
    const int2* cache = reinterpret_cast<const int2*>(smem + kOffUnits);
    unsigned short* ustart = reinterpret_cast<unsigned short*>(smem + kOffStart);
    int* pref = reinterpret_cast<int*>(smem + kOffRowPref);
    for (int x = lane; x <= rows; x += 32) pref[x] = pref[kRowCap + 1 + x] = 0;
    __syncwarp();
    for (int c = 0; c < 2; ++c) {
        const int n_class = c == 0 ? n_heavy : units - n_heavy;
        for (int u = lane; u < n_class; u += 32) {
            const int nb = (cache[c * kUnitCache + u].y + kBlk - 1) / kBlk;
            const int s = rows_small * kSmallBlocks;
            const int items = nb <= s ? (nb + kSmallBlocks - 1) / kSmallBlocks
                                      : rows_small + (nb - s + item_blocks - 1) / item_blocks;   // item_count
            const int start = max(rows - items, 0);   // == rows: the sequence is empty
            ustart[c * kUnitCache + u] = (unsigned short)start;
            if (start < rows) atomicAdd(&pref[c * (kRowCap + 1) + start], 1);
        }
    }
    __syncwarp();
    for (int c = 0; c < 2; ++c) {   // units starting in row r -> units present in row r -> draws before row r
        int* pc = pref + c * (kRowCap + 1);
        int started = 0, before = 0;
        for (int base = 0; base < rows; base += 32) {
            const int r = base + lane;
            int v = r < rows ? pc[r] : 0;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int t = __shfl_up_sync(kFull, v, o);
                if (lane >= o) v += t;
            }
            const int here = r < rows ? started + v : 0;
            int w = here;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int t = __shfl_up_sync(kFull, w, o);
                if (lane >= o) w += t;
            }
            if (r < rows) pc[r] = before + w - here;
            started += __shfl_sync(kFull, v, 31);
            before += __shfl_sync(kFull, w, 31);
        }
        if (lane == 0) pc[rows] = before;
        if (c == 0) total_heavy = before; else total_light = before;
    }
    __syncwarp();
    return make_int2(total_heavy, total_light);
}

// draw number k of a class -> row (among the rows in use) and index within the class, through the row tables;
// all lanes, same arguments
__device__ __forceinline__ int2 table_lookup(const unsigned char* smem, int c, int n_class, int rows, int k, int lane) {
    const int* pc = reinterpret_cast<const int*>(smem + kOffRowPref) + c * (kRowCap + 1);
    const unsigned short* ustart = reinterpret_cast<const unsigned short*>(smem + kOffStart) + c * kUnitCache;
    // the last row whose first draw is <= k: 32-way search, the lanes probing evenly spaced rows (pc is monotone and
    // pc[0] = 0 <= k, so the lanes that pass form a prefix)
    int lo = 0, span = rows;
    while (span > 1) {
        const int step = (span + 31) >> 5;
        const int r = lo + lane * step;
        const unsigned pass = __ballot_sync(kFull, r < lo + span && pc[r] <= k);
        const int seg = __popc(pass) - 1;
        span = min(step, span - seg * step);
        lo += seg * step;
    }
    int j = k - pc[lo], sel = 0;               // the j-th unit, in list order, that has an item in this row
    for (int i0 = 0; i0 < n_class; i0 += 32) {
        const int i = i0 + lane;
        const bool present = i < n_class && (int)ustart[i] <= lo;
        const unsigned m = __ballot_sync(kFull, present);
        const int cnt = __popc(m);
        if (j < cnt) {   // the lane whose unit is present and has exactly j present units before it
            const unsigned hit = __ballot_sync(kFull, present && __popc(m & ((1u << lane) - 1u)) == j);
            sel = i0 + __ffs(hit) - 1;
            break;
        }
        j -= cnt;
    }
    return make_int2(lo, sel);
}

// draw number k of a class -> work item
// (a unit-list entry is the pair (unit, clamped sequence length), so no length is fetched per item)
__device__ __forceinline__ Item decode_item(const DecodeParams& p, const ItemSched& sc, const int2* unit_cache,
                                            bool heavy, int k, int2 via_table) {
    Item it;
    int row;
    int2 un;
    if (sc.table) {
        row = via_table.x;
        un = unit_cache[(heavy ? 0 : kUnitCache) + via_table.y];
    } else if (heavy) {   // heavy units sit at the front of the list, light units at its back (first ones cached in smem)
        row = (int)fast_div((unsigned)k, sc.magic_heavy);
        const int u = k - row * sc.n_heavy;
        un = u < kUnitCache ? unit_cache[u] : p.unit_list[u];
    } else {
        row = (int)fast_div((unsigned)k, sc.magic_light);
        const int u = k - row * sc.n_light;
        un = u < kUnitCache ? unit_cache[kUnitCache + u] : p.unit_list[p.units - 1 - u];
    }
    // (entries are written by the pseudo-max kernel of this call; the clamps only matter on a workspace whose
    // counters an interrupted call left behind, where a stale entry of another geometry could be drawn)
    const int bg = min(max(un.x, 0), p.units - 1);
    un.y = min(max(un.y, 0), p.max_blocks * kBlk);
    row += sc.row_off;
    it.slot = row * p.units + bg;
    it.bg = bg;
    it.b = (int)fast_div((unsigned)bg, p.hkv_magic);
    it.g = bg - it.b * p.Hkv;
    it.n = un.y;
    const int nb = (it.n + kBlk - 1) / kBlk;
    int cap;
    item_span(p, p.item_rows - 1 - row, it.blk0, cap);
    it.nblk = min(nb - it.blk0, cap);
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
// Entry seq lives in slot seq % 8 and is announced by one arrival on that slot's mbarrier (phase seq / 8): the
// arrive releases the entry's fields, a successful test / wait acquires them.  No fence is used on purpose: a CTA
// fence would also wait for the reader's in-flight cp.async copies and serialise the prefetch ring.  Every scan warp
// visits every entry in order and the publisher is never more than four entries ahead of the slowest of them (it
// waits for the full barrier of entry e - 4 before publishing e), so a parity test can not alias.

__device__ __forceinline__ uint32_t item_bar(uint32_t ibars, int seq) { return ibars + (seq & (kItemRing - 1)) * 8; }

__device__ __forceinline__ bool item_ready(uint32_t ibars, int seq) {
    return mbar_test(item_bar(ibars, seq), (seq / kItemRing) & 1);
}

__device__ __forceinline__ bool item_wait(uint32_t ibars, int seq) {
    return mbar_wait(item_bar(ibars, seq), (seq / kItemRing) & 1);
}

__device__ __forceinline__ Item item_read(const ItemSlot* ring, int seq) {
    const ItemSlot& e = ring[seq & (kItemRing - 1)];
    Item it;
    it.slot = e.slot; it.b = e.b; it.g = e.g; it.bg = e.bg; it.blk0 = e.blk0; it.nblk = e.nblk; it.n = e.n;
    return it;
}

// batches every attend warp has finished (they take the batches in order); a plain monotonic count, because a
// parity test on the empty barriers could be fooled when a slot completes two phases between two looks
__device__ __forceinline__ int attend_finished(const volatile int* attend_done) {
    return min(min(attend_done[0], attend_done[1]), min(attend_done[2], attend_done[3]));
}
static_assert(kNA == 4, "attend_finished reads four counters");

__device__ __forceinline__ void qrec_issue(const DecodeParams& p, int seq, int bg, uint32_t qrecs, uint32_t qbars,
                                           int lane);

// ---- scheduling role (warp 0) ------------------------------------------------------------------------------
// Publishes ring entry after ring entry: chooses the class, takes the class's pending ticket (the next one is
// fetched at once and not looked at until the next entry, so the atomic's latency is hidden), decodes it, looks the
// item's pages up, writes the item and the header of its batch descriptor, announces it and starts the copy of its
// query record.  Entry e reuses the record slot of entry e - 4 and the item slot of entry e - 8, so every scan warp
// must have finished batch e - 4 (its full barrier) and the attend warps batch e - 8 (its empty barrier) first.
// pend_heavy / pend_light: the first tickets, drawn by the caller.
__device__ __forceinline__ void sched_role(const DecodeParams& p, unsigned char* smem, int lane, int pend_heavy,
                                           int pend_light) {
    const uint32_t qrecs = smem_u32(smem) + kOffQrec;
    const uint32_t bars = smem_u32(smem) + kOffBars;
    const uint32_t qbars = bars + (2 * kNB + 2 * kNA) * 8;
    const uint32_t ibars = qbars + kQrecRing * 8;
    BatchDesc* descs = reinterpret_cast<BatchDesc*>(smem + kOffDesc);
    ItemSlot* items = reinterpret_cast<ItemSlot*>(smem + kOffItems);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kOffAbort);
    const volatile int* attend_done = reinterpret_cast<const volatile int*>(smem + kOffAttendDone);
    const int2* unit_cache = reinterpret_cast<const int2*>(smem + kOffUnits);
    ItemSched sc;
    // (a workspace whose header was never initialised hands out no work: the pseudo-max kernel has reported it)
    const bool header_ok = p.status[kHeaderCookieWord] == kHeaderCookie;
    sc.n_heavy = header_ok ? min((int)p.class_counts[0], p.units) : 0;
    sc.n_light = header_ok ? p.units - sc.n_heavy : 0;
    // Rows in use: up to the longest sequence of the batch (a cache sized for longer contexts than it holds would
    // otherwise spend most tickets on rows no sequence reaches).
    const int rows = item_count(p, min((int)p.len_stats[0], p.max_blocks));
    sc.row_off = p.item_rows - rows;
    sc.total_heavy = sc.n_heavy * rows;
    sc.total_light = sc.n_light * rows;
    sc.table = 2ll * (long long)p.len_stats[2] < (long long)p.units * rows && rows <= kRowCap &&
               sc.n_heavy <= kUnitCache && sc.n_light <= kUnitCache;
    if (sc.table) {
        const int2 totals = plan_tables(p.units, p.rows_small, p.item_blocks, smem, sc.n_heavy, rows, lane);
        sc.total_heavy = totals.x;
        sc.total_light = totals.y;
    }
    sc.magic_heavy = fast_div_magic((unsigned)max(sc.n_heavy, 1));
    sc.magic_light = fast_div_magic((unsigned)max(sc.n_light, 1));
    // (draws from counters that were never zeroed are not draws: a negative one would pass for "work left")
    sc.pend_heavy = header_ok && pend_heavy >= 0 ? pend_heavy : 0x7fffffff;
    sc.pend_light = header_ok && pend_light >= 0 ? pend_light : 0x7fffffff;
    sc.released = 0;
    sc.heavy_queued = 0;
    sc.heavy_hist = 0ull;
#pragma unroll 1
    for (int pub = 0;; ++pub) {
        bool ok = true;
        if (pub >= 4) ok = mbar_wait(bars + ((pub - 4) & (kNB - 1)) * 8, ((pub - 4) / kNB) & 1);
        if (ok && pub >= kNB) ok = mbar_wait(bars + (kNB + (pub & (kNB - 1))) * 8, (pub / kNB - 1) & 1);
        ItemSlot& e = items[pub & (kItemRing - 1)];
        BatchDesc& d = descs[pub & (kNB - 1)];
        if (!ok) *abort_flag = 1;
        Item it;
        it.slot = -1; it.b = it.g = it.bg = it.blk0 = it.nblk = it.n = 0;
#pragma unroll 1
        while (!*abort_flag) {
            int kind = -1, cand = 0;      // -1: no work left, 0: light, 1: heavy
            if (lane == 0) {
                // batches the attend warps have released since the last look
                for (const int rel = min(attend_finished(attend_done), pub); sc.released < rel; ++sc.released)
                    if ((sc.heavy_hist >> (sc.released & 63)) & 1ull) --sc.heavy_queued;
                const bool heavy_left = sc.pend_heavy < sc.total_heavy, light_left = sc.pend_light < sc.total_light;
                // Heavy batches published and not yet released: at most four.  Near the end of the heavy work, when
                // the attend warps are the bottleneck, at most kHeavyAhead, so that no CTA sits on heavy work others
                // could have taken.  Beyond the limit the scan warps spend their spare time on light items.
                const int limit = sc.total_heavy - sc.pend_heavy > 2 * (int)gridDim.x ? 4 : kHeavyAhead;
                if (heavy_left && sc.heavy_queued < limit) kind = 1;
                else if (light_left) kind = 0;
                else if (heavy_left) {   // only heavy work is left and enough of it is queued: wait for the attend warps
                    kind = 2;
                    const long long t0 = clock64();
                    while (attend_finished(attend_done) <= sc.released) {
                        __nanosleep(256);
                        if (clock64() - t0 > kSpinCycles) { *abort_flag = 1; break; }
                    }
                }
                if (kind == 1) { cand = sc.pend_heavy; sc.pend_heavy = (int)min(atomicAdd(p.item_counter, 1u), 0x7fffffffu); }
                if (kind == 0) { cand = sc.pend_light; sc.pend_light = (int)min(atomicAdd(p.light_counter, 1u), 0x7fffffffu); }
            }
            kind = __shfl_sync(kFull, kind, 0);
            cand = __shfl_sync(kFull, cand, 0);
            if (kind == 2) continue;
            if (kind < 0) break;
            // every lane decodes the same item (the class sizes and reciprocals are the same in all lanes)
            int2 via_table = make_int2(0, 0);
            if (sc.table) via_table = table_lookup(smem, kind == 1 ? 0 : 1, kind == 1 ? sc.n_heavy : sc.n_light, rows, cand, lane);
            const Item c = decode_item(p, sc, unit_cache, kind == 1, cand, via_table);
            if (c.nblk <= 0) continue;   // the sequence is shorter than the longest one: nothing in this item
            it = c;
            if (lane == 0) {
                if (kind == 1) { sc.heavy_hist |= 1ull << (pub & 63); ++sc.heavy_queued; }
                else sc.heavy_hist &= ~(1ull << (pub & 63));
            }
            break;
        }
        if (it.slot >= 0) qrec_issue(p, pub, it.bg, qrecs, qbars, lane);   // lands while the pages are looked up
        if (it.slot >= 0 && lane < it.nblk) {   // the item's page-table entries: one coalesced read
            const int blk = it.blk0 + lane;
            int page = p.block_table ? p.block_table[(size_t)it.b * p.max_blocks + blk] : it.b * p.max_blocks + blk;
            if (page < 0 || page >= p.num_pages) { atomicOr(p.status, kDevBadPage); page = -1; }
            e.pages[lane] = page;
        }
        if (lane == 0) {
            e.slot = it.slot; e.b = it.b; e.g = it.g; e.bg = it.bg; e.blk0 = it.blk0; e.nblk = it.nblk; e.n = it.n;
            d.item = it.slot; d.b = it.b; d.g = it.g; d.nblk = it.nblk;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(item_bar(ibars, pub));
        if (it.slot < 0) break;
    }
    cp_async_drain();
    if (*abort_flag && lane == 0) atomicOr(p.status, kDevTimeout);
}

// ---- scan role ---------------------------------------------------------------------------------------------

// Position of a scan warp in its stream of blocks: published item after published item, local blocks w, w + 11, w + 22.
struct ScanCursor {
    int seq;       // published item the cursor is in (-1 before the first)
    Item it;
    int lb;
    int pages;     // lane l: physical page of block l of the item (loaded once per item, not per block)
    bool end;      // ran into the end of the work
};

// Advance to this warp's next block; false when the item it lies in has not been published yet (the cursor then
// stays where it can resume) or when there is no more work.
__device__ __forceinline__ bool cursor_next(const DecodeParams& p, ScanCursor& c, const ItemSlot* items,
                                            uint32_t ibars, int w, int lane) {
    if (c.end) return false;
    int lb = c.lb + kScanners;
    while (lb >= c.it.nblk) {
        if (!item_ready(ibars, c.seq + 1)) { c.lb = lb - kScanners; return false; }
        c.it = item_read(items, c.seq + 1);
        ++c.seq;
        if (c.it.slot < 0) { c.end = true; c.it.nblk = 0; return false; }
        lb = w;
        if (lb < c.it.nblk) c.pages = lane < c.it.nblk ? items[c.seq & (kItemRing - 1)].pages[lane] : -1;
    }
    c.lb = lb;
    return true;
}

// start the copy of one block's codes + scales into a ring stage (one commit group); remembers the block's tile
__device__ __forceinline__ void ring_issue(const DecodeParams& p, const ScanCursor& c, uint32_t stage,
                                           volatile int* stage_tile, int lane) {
    const int page = __shfl_sync(kFull, c.pages, c.lb);   // -1: bad table entry (reported by the scheduler), skipped
    const int tile = page >= 0 ? (int)tile_index(p, page, c.it.g) : -1;
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

// Scheduling warp: copy the query record of published item `seq` into slot seq % 4 of the record ring and report
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
                                                 int lane, int rows, float unit) {
    ScanRegs sr;
    scan_load(sr, codes_tile, scales_tile, lane);
    ScanQuery sq;
    sq.piece = (lane >> 2) & 1;
#pragma unroll
    for (int x = 0; x < 4; ++x) {
        const uint4 v = lds128(qrec + (x * 32 + lane) * 16);
        sq.qh[4 * x] = v.x; sq.qh[4 * x + 1] = v.y; sq.qh[4 * x + 2] = v.z; sq.qh[4 * x + 3] = v.w;
    }
    sq.unit = unit;
    float band;
    return scan_compute<true>(sr, sq, lane, rows, band);
}

// RES (2 + 8 bit key format): the per-token approximate logits of every block that may be kept are left in the
// CTA's ring of score tiles in global memory (tile (batch slot, block) -- free again when the attend warps have
// released the batch slot, which the scheduler waits for before it publishes into it).  Writer and reader are threads
// of this CTA: the release of the full barrier's arrive and the acquire of the attend warp's wait order the stores
// before the reader's copies (a device-scope fence in between measured 1 - 3 us per step and buys nothing).
template <bool RES>
__device__ __forceinline__ void scan_role(const DecodeParams& p, unsigned char* smem, int w, int lane) {
    const int r = lane >> 2, j = lane & 3;
    const int w0 = w - kSched;      // index among the scanning warps
    const uint32_t ring = smem_u32(smem) + kOffRing + w0 * kRing * kStageBytes;
    const uint32_t qrecs = smem_u32(smem) + kOffQrec;
    const uint32_t bars = smem_u32(smem) + kOffBars;
    const uint32_t qbars = bars + (2 * kNB + 2 * kNA) * 8;
    const uint32_t ibars = qbars + kQrecRing * 8;
    BatchDesc* descs = reinterpret_cast<BatchDesc*>(smem + kOffDesc);
    ItemSlot* items = reinterpret_cast<ItemSlot*>(smem + kOffItems);
    volatile int* stage_tile = reinterpret_cast<volatile int*>(smem + kOffStageTile) + w * 4;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kOffAbort);
    ScanCursor ic;
    ic.seq = -1;
    ic.it.nblk = 0;
    ic.lb = w0 - kScanners;
    ic.end = false;
    ic.pages = -1;
    int issued = 0, consumed = 0;   // this warp's blocks whose copies were started / whose data was taken
    int bound_state = 0;            // >= 0: failures of the scale-only bound in a row; < 0: blocks until it is tried again

#pragma unroll 1
    for (int seq = 0;; ++seq) {     // published item seq = batch seq
        if (!item_wait(ibars, seq)) *abort_flag = 1;
        const Item it = item_read(items, seq);
        // (the scheduling warp made sure, before it published the item, that the attend warps have released this
        // descriptor and wrote its header)
        const int slot = seq & (kNB - 1);
        BatchDesc& d = descs[slot];
        if (it.slot < 0 || *abort_flag) {   // no more work: tell the attend warps
            if (lane == 0) {
                if (w0 == 0) d.item = -1;
                mbar_arrive(bars + slot * 8);
            }
            break;
        }
        // The prefetch cursor only moves when this warp has a block to fetch, so after items too short to reach the
        // warp it lags behind; an entry more than a ring behind has been overwritten.  Everything of this warp's
        // stream before this item has been issued, so the cursor may jump to the item's start.
        if (ic.seq < seq) {
            ic.seq = seq;
            ic.it = it;
            ic.lb = w0 - kScanners;
            if (w0 < it.nblk) ic.pages = lane < it.nblk ? items[seq & (kItemRing - 1)].pages[lane] : -1;
        }
        // start this warp's copies of the item's blocks, then wait for the item's query record
        if (w0 < it.nblk)
            while (issued < consumed + kRing && cursor_next(p, ic, items, ibars, w0, lane)) {
                ring_issue(p, ic, ring + (issued % kRing) * kStageBytes, stage_tile + issued % kRing, lane);
                ++issued;
            }
        if (!mbar_wait(qbars + (seq & (kQrecRing - 1)) * 8, (seq / kQrecRing) & 1)) *abort_flag = 1;
        const uint32_t qrec = qrecs + (seq & (kQrecRing - 1)) * kQrecBytes;
        const size_t head0 = (size_t)it.b * p.Hq + (size_t)it.g * p.G;
        // threshold and accumulator unit of head lane % 4 (block-max layout); threshold, bound multiplier and bound
        // slack of head lane / 8 (B-column layout)
        float thr, unit, thr_col, bmul_col, badd_col;
        asm volatile("ld.shared.f32 %0, [%1];\n" : "=f"(thr) : "r"(qrec + kQrecThr + j * 4));
        asm volatile("ld.shared.f32 %0, [%1];\n" : "=f"(unit) : "r"(qrec + kQrecThr + 16 + j * 4));
        asm volatile("ld.shared.f32 %0, [%1];\n" : "=f"(thr_col) : "r"(qrec + kQrecThr + (lane >> 3) * 4));
        asm volatile("ld.shared.f32 %0, [%1];\n" : "=f"(bmul_col) : "r"(qrec + kQrecThr + 32 + (lane >> 3) * 4));
        asm volatile("ld.shared.f32 %0, [%1];\n" : "=f"(badd_col) : "r"(qrec + kQrecThr + 48 + (lane >> 3) * 4));
#pragma unroll 1
        for (int lb = w0; lb < it.nblk; lb += kScanners) {
            // keep the ring full: blocks consumed .. consumed + kRing - 1 of this warp's stream
            while (issued < consumed + kRing && cursor_next(p, ic, items, ibars, w0, lane)) {
                ring_issue(p, ic, ring + (issued % kRing) * kStageBytes, stage_tile + issued % kRing, lane);
                ++issued;
            }
            const int st = consumed % kRing;
            const uint32_t stage = ring + st * kStageBytes;
            ring_wait(issued - consumed - 1);
            __syncwarp();
            // No token of the block can score above 1.5 * sum |q s| (every level is at most 1.5 in magnitude).  If
            // that bound stays below the threshold for every head of the group, no head can keep the block: its
            // codes are not even read from shared memory, and the decision is the same as the full scan's.  (Not when
            // the caller asked for the block maxima themselves, and not while the bound keeps failing.)
            uint4 sv[4];
#pragma unroll
            for (int x = 0; x < 4; ++x) sv[x] = lds128(stage + kCodeBytes + (4 * x + j) * 16);
            const int tile = stage_tile[st];
            bool cannot_keep = false;
            if (p.block_max == nullptr && bound_state >= 0) {
                __half2 sum_a = __floats2half2_rn(0.f, 0.f), sum_b = sum_a;
#pragma unroll
                for (int x = 0; x < 4; ++x) scan_abs_sum(lds128(qrec + kQrecAbs + (x * 32 + lane) * 16), sv[x], sum_a, sum_b);
                cannot_keep = __all_sync(kFull, scan_bound(sum_a, sum_b, bmul_col, badd_col) < thr_col);
                // a bound that fails 16 times in a row (a dense head) is left out for the next 48 blocks
                bound_state = cannot_keep ? 0 : bound_state + 1;
                if (bound_state == 16) bound_state = -48;
            } else if (bound_state < 0) {
                ++bound_state;
            }
            const int blk = it.blk0 + lb;
            const int rows = min(kBlk, it.n - blk * kBlk);
            unsigned keep4 = 0;
            bool refilled = false;
            if (tile >= 0 && !cannot_keep) {   // codes into registers; B operand from the staged scales and the record
                uint4 wv[4];
                uint32_t bfrag[16];
#pragma unroll
                for (int mt = 0; mt < 4; ++mt) wv[mt] = lds128(stage + (mt * 32 + lane) * 16);
#pragma unroll
                for (int x = 0; x < 4; ++x) scan_bfrag4(bfrag + 4 * x, lds128(qrec + (x * 32 + lane) * 16), sv[x], r & 1);
                __syncwarp();   // the stage is free again: refill it before the tensor-core work, not after
                ++consumed;
                if (issued < consumed + kRing && cursor_next(p, ic, items, ibars, w0, lane)) {
                    ring_issue(p, ic, ring + (issued % kRing) * kStageBytes, stage_tile + issued % kRing, lane);
                    ++issued;
                }
                refilled = true;
                float band;
                float tok[8];
                float bm = scan_mma<false>(wv, bfrag, lane, rows, unit, band, RES ? tok : nullptr);
                bool force_keep = false;
                if (bm != bm) {   // (uniform, rare) a scale too large for the fp16 operand: binary32 on the ordinary lanes
                    float* scores = nullptr;
                    if constexpr (RES)
                        scores = p.res_scores + ((size_t)(blockIdx.x * kNB + slot) * kItemBlocksMax + lb) * kScoreTileFloats;
                    bm = scan_block_wide(reinterpret_cast<const uint4*>(p.k_quant + (size_t)tile * kCodeBytes),
                                         p.k_scales + (size_t)tile * kD, p.q + head0 * kD, p.G, lane, rows, p.sm_scale,
                                         scores, kScoreStride);
                    if (__any_sync(kFull, (j < p.G) && !(fabsf(bm) < INFINITY))) {   // beyond binary32 too: reported, kept
                        if (lane == 0) atomicOr(p.status, kDevRange);
                        force_keep = true;
                    }
                } else {
                    if constexpr (RES) {
                        if (__any_sync(kFull, (j < p.G) && bm >= thr - band)) {
                            float* dst = p.res_scores + ((size_t)(blockIdx.x * kNB + slot) * kItemBlocksMax + lb) * kScoreTileFloats +
                                         j * kScoreStride + r;
#pragma unroll
                            for (int mt = 0; mt < 4; ++mt) {
                                dst[16 * mt] = tok[2 * mt];
                                dst[16 * mt + 8] = tok[2 * mt + 1];
                            }
                        }
                    }
                    // too close to call (rare): a separate, non-inlined routine re-reads the block and redoes it precisely
                    if (__any_sync(kFull, (j < p.G) && fabsf(bm - thr) <= band))
                        bm = scan_block_precise(reinterpret_cast<const uint4*>(p.k_quant + (size_t)tile * kCodeBytes),
                                                reinterpret_cast<const uint4*>(p.k_scales + (size_t)tile * kD), qrec, lane,
                                                rows, unit);
                }
                const bool keep = (j < p.G) && (force_keep || bm >= thr);
                keep4 = __ballot_sync(kFull, keep) & 0xFu;
                if (r == 0 && j < p.G) {
                    const size_t o = (head0 + j) * p.max_blocks + blk;
                    if (p.kept_mask) p.kept_mask[o] = keep ? 1 : 0;
                    if (p.block_max) p.block_max[o] = bm;
                }
            }
            __syncwarp();
            if (!refilled) ++consumed;   // the stage is free again (what was read from it has been used)
            if (!refilled && issued < consumed + kRing && cursor_next(p, ic, items, ibars, w0, lane)) {
                ring_issue(p, ic, ring + (issued % kRing) * kStageBytes, stage_tile + issued % kRing, lane);
                ++issued;
            }
            if (cannot_keep && tile >= 0 && p.kept_mask && r == 0 && j < p.G)
                p.kept_mask[(head0 + j) * p.max_blocks + blk] = 0;
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
    if (*abort_flag && w0 == 0 && lane == 0) atomicOr(p.status, kDevTimeout);
}

// ---- attend role -------------------------------------------------------------------------------------------

// bits of the blocks of a published batch that attend warp `a` processes: every kNA-th kept block
__device__ __forceinline__ unsigned my_entries(const BatchDesc& d, int nblk, int a, int lane) {
    const bool is_kept = lane < nblk && d.keep4[lane] != 0;
    const unsigned kept = __ballot_sync(kFull, is_kept);
    const int rank = __popc(kept & ((1u << lane) - 1u));   // kept blocks before this lane's
    return __ballot_sync(kFull, is_kept && (rank & (kNA - 1)) == a);
}

// score tile of block lb of the batch in descriptor slot `slot` of this CTA
__device__ __forceinline__ float* score_tile(const DecodeParams& p, int slot, int lb) {
    return p.res_scores + ((size_t)(blockIdx.x * kNB + slot) * kItemBlocksMax + lb) * kScoreTileFloats;
}

// RES: the 2 + 8 bit key format -- the K slot receives the block's residual tile, codes and scales instead of its
// 16-bit keys
template <bool RES>
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
    uint32_t qb[RES ? 8 : 1];
    for (int bi = 0; ok; ++bi) {
        const int slot = bi & (kNB - 1), use = bi / kNB;
        if (!mbar_wait(bars + slot * 8, use & 1)) { ok = false; break; }
        const BatchDesc& d = descs[slot];
        const int item = d.item;
        if (item < 0) break;
        Item it;
        it.slot = item; it.b = d.b; it.g = d.g; it.nblk = d.nblk;
        // the share rotates with the batch number: when the kept count is not a multiple of four, the extra blocks
        // go to a different warp each time
        unsigned mine = my_entries(d, it.nblk, (a + bi) & (kNA - 1), lane);
        const bool any = mine != 0;
        if (any) {
            if constexpr (RES) attend_setup_res(st, qb, p, it.b, it.g, lane);
            else attend_setup(st, p.q + ((size_t)it.b * p.Hq + (size_t)it.g * p.G) * kD, p.G, lane);
        }
        while (mine && ok) {
            const int lb = __ffs(mine) - 1;
            mine &= mine - 1;
            if (!(issued_bi == bi && issued_lb == lb)) {
                if constexpr (RES) res_copy_async(kslot, p, d.tile[lb], score_tile(p, slot, lb), lane, kbar);
                else tile_copy_async(kslot, kbase + (size_t)d.tile[lb] * kTileVec, lane, kbar);
                tile_copy_async(vslot, vbase + (size_t)d.tile[lb] * kTileVec, lane, vbar);
            }
            // the next block this warp will attend: in this batch, else in the next one if it is already published
            const uint4 *next_k = nullptr, *next_v = nullptr;
            int next_tile = -1;
            const float* next_scores = nullptr;
            if (mine) {
                const int nlb = __ffs(mine) - 1;
                next_tile = (int)d.tile[nlb];
                if constexpr (RES) next_scores = score_tile(p, slot, nlb);
                next_k = kbase + (size_t)d.tile[nlb] * kTileVec;
                next_v = vbase + (size_t)d.tile[nlb] * kTileVec;
                issued_bi = bi;
                issued_lb = nlb;
            } else {
                const int bi2 = bi + 1;
                if (mbar_test(bars + (bi2 & (kNB - 1)) * 8, (bi2 / kNB) & 1)) {
                    const BatchDesc& d2 = descs[bi2 & (kNB - 1)];
                    if (d2.item >= 0) {
                        const unsigned mine2 = my_entries(d2, d2.nblk, (a + bi2) & (kNA - 1), lane);
                        if (mine2) {
                            const int nlb = __ffs(mine2) - 1;
                            next_tile = (int)d2.tile[nlb];
                            if constexpr (RES) next_scores = score_tile(p, bi2 & (kNB - 1), nlb);
                            next_k = kbase + (size_t)d2.tile[nlb] * kTileVec;
                            next_v = vbase + (size_t)d2.tile[nlb] * kTileVec;
                            issued_bi = bi2;
                            issued_lb = nlb;
                        }
                    }
                }
            }
            if constexpr (RES)
                ok = attend_block_res(st, qb, p, kslot, vslot, kbar, vbar, phase, next_tile, next_scores, next_v, lane,
                                      d.rows[lb], d.keep4[lb]);
            else
                ok = attend_block(st, kslot, vslot, kbar, vbar, phase, next_k, next_v, lane, d.rows[lb], d.keep4[lb],
                                  logit_scale_log2);
        }
        __syncwarp();
        if (lane == 0) {
            mbar_arrive(bars + (kNB + slot) * 8);   // done with this batch descriptor
            reinterpret_cast<volatile int*>(smem + kOffAttendDone)[a] = bi + 1;
        }
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

template <bool RES>
__global__ void __launch_bounds__(kFusedThreads, 1) fused_sparse_kernel(DecodeParams p) {
    extern __shared__ __align__(1024) unsigned char smem[];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        const uint32_t bars = smem_u32(smem) + kOffBars;
        for (int s = 0; s < kNB; ++s) {
            mbar_init(bars + s * 8, kScanners);       // full: one arrival per scanning warp
            mbar_init(bars + (kNB + s) * 8, kNA);     // empty: one arrival per attend warp
        }
        for (int a = 0; a < 2 * kNA + kQrecRing; ++a) mbar_init(bars + (2 * kNB + a) * 8, 32);
        for (int s = 0; s < kItemRing; ++s) mbar_init(bars + (2 * kNB + 2 * kNA + kQrecRing + s) * 8, 1);
        *reinterpret_cast<volatile int*>(smem + kOffAbort) = 0;
        for (int a = 0; a < kNA; ++a) reinterpret_cast<volatile int*>(smem + kOffAttendDone)[a] = 0;
    }
    pdl_launch_dependents();
    // First draw of each class.  The counters were reset by the previous call's combine kernel, and the pseudo-max
    // kernel lets this kernel start only once everything before it has finished, so this need not wait.
    int pend_heavy = 0, pend_light = 0;
    if (threadIdx.x == 0) {
        pend_heavy = (int)atomicAdd(p.item_counter, 1u);
        pend_light = (int)atomicAdd(p.light_counter, 1u);
    }
    pdl_wait();   // the pseudo-max kernel's outputs (unit list, class counts, query records) are needed from here on
    {   // shared-memory copy of both ends of the unit list (heavy units from the front, light units from the back)
        int2* cache = reinterpret_cast<int2*>(smem + kOffUnits);
        for (int u = threadIdx.x; u < min(p.units, kUnitCache); u += kFusedThreads) {
            cache[u] = p.unit_list[u];
            cache[kUnitCache + u] = p.unit_list[p.units - 1 - u];
        }
    }
    if (threadIdx.x == 0) {
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    __syncthreads();
    if (warp < kNS) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;\n" ::"n"(kScanRegs));
        if (warp < kSched) sched_role(p, smem, lane, pend_heavy, pend_light);
        else scan_role<RES>(p, smem, warp, lane);
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;\n" ::"n"(kAttendRegs));
        attend_role<RES>(p, smem, warp - kNS, lane);
    }
}

// ---- split combine (FlashDecoding-style log-sum-exp merge) -------------------------------------------------
// One, two or four CTAs of 256 .. 1024 threads per (query head, sequence), each taking a share of the channels.
// FUSED: partial e = (work item, attend warp) of the fused kernel; otherwise partial e = split of the dense kernel.
// The (m, l) pairs are read once into shared memory; thread (el, cg) sums the partials e = el, el + lanes, ... for
// four channels with eight independent loads in flight; the partial sums meet in shared memory.  For a given launch
// shape the summation order is fixed.
constexpr int kCombineThreads = 1024;
constexpr int kCombineLanes = kCombineThreads / 32;   // partials summed side by side (at most: the launch may use fewer threads)
constexpr int kCombineChunk = 1024;

template <bool FUSED>
__device__ __forceinline__ size_t combine_slot(const DecodeParams& p, size_t head, int bg, int hl, int e) {
    if (FUSED) {   // item number of split e / kNA (items count from block 0, see item_span), then the attend warp
        const int item = (p.item_rows - 1 - e / kNA) * p.units + bg;
        return ((size_t)item * kNA + (e % kNA)) * kMaxG + hl;
    }
    return head * p.splits + e;
}

template <bool FUSED>
__global__ void __launch_bounds__(kCombineThreads) combine_kernel(DecodeParams p) {
    // gridDim.z = 1, 2 or 4 CTAs share a head, each taking 128 / gridDim.z channels (few heads: more CTAs)
    const int h = blockIdx.x, b = blockIdx.y, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int cgn = 32 / (int)gridDim.z;          // groups of four channels per CTA
    const int el = tid / cgn, cg = tid % cgn;
    const int threads = blockDim.x, warps = threads >> 5, lanes = threads / cgn;
    const int chan0 = (int)blockIdx.z * 4 * cgn;
    pdl_launch_dependents();
    pdl_wait();
    if (FUSED && h == 0 && b == 0 && blockIdx.z == 0 && tid == 0) {   // the next call's draws and class lists start from zero
        *p.item_counter = 0u;
        p.class_counts[0] = 0u;
        p.class_counts[1] = 0u;
        *p.light_counter = 0u;
        p.len_stats[0] = 0u;
        p.len_stats[1] = 0u;
        p.len_stats[2] = 0u;
    }
    // append + decode: the caller's lengths take the new values now that nothing of this call reads them any more
    if (FUSED && p.bump_lens && h == 0 && blockIdx.z == 0 && tid == 0) p.bump_lens[b] = p.seq_lens[b];
    const size_t head = (size_t)b * p.Hq + h;
    const int g = h / p.G, hl = h % p.G, bg = b * p.Hkv + g;
    const int n = min(max(p.seq_lens[b], 0), p.max_blocks * kBlk);
    const int nb = (n + kBlk - 1) / kBlk;
    const int entries = FUSED ? item_count(p, nb) * kNA
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
        for (int x = tid; x < cnt; x += threads) {
            const float2 v = *reinterpret_cast<const float2*>(ml + combine_slot<FUSED>(p, head, bg, hl, base + x) * 2);
            s_m[x] = v.y > 0.f ? v.x : -INFINITY;
            s_l[x] = v.y;
            M = fmaxf(M, s_m[x]);
        }
#pragma unroll
        for (int o = 16; o; o >>= 1) M = fmaxf(M, __shfl_xor_sync(kFull, M, o));
        if (lane == 0) s_red[warp] = M;
        __syncthreads();
        M = Mrun;
#pragma unroll
        for (int x = 0; x < kCombineLanes; ++x)
            if (x < warps) M = fmaxf(M, s_red[x]);
        if (M == -INFINITY) continue;      // uniform: nothing in this chunk or before it
        const float rescale = exp2f(Mrun - M);   // 0 for the first non-empty chunk
        acc.x *= rescale; acc.y *= rescale; acc.z *= rescale; acc.w *= rescale;
        L *= rescale;
        Mrun = M;
        for (int x = tid; x < cnt; x += threads) {
            const float wv = exp2f(s_m[x] - M);  // exp2(-inf) = 0 for empty partials
            L += wv * s_l[x];
            s_m[x] = wv;
        }
        __syncthreads();
        for (int x0 = el; x0 < cnt; x0 += lanes * 8) {
            float4 v[8];
            float wv[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int x = x0 + lanes * u;
                wv[u] = x < cnt ? s_m[x] : 0.f;
                v[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (wv[u] != 0.f)
                    v[u] = *reinterpret_cast<const float4*>(pacc + combine_slot<FUSED>(p, head, bg, hl, base + x) * kD +
                                                            chan0 + 4 * cg);
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                acc.x += wv[u] * v[u].x; acc.y += wv[u] * v[u].y; acc.z += wv[u] * v[u].z; acc.w += wv[u] * v[u].w;
            }
        }
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) L += __shfl_xor_sync(kFull, L, o);
    for (int o = cgn; o < 32; o <<= 1) {   // the partial lanes that share a warp
        acc.x += __shfl_xor_sync(kFull, acc.x, o); acc.y += __shfl_xor_sync(kFull, acc.y, o);
        acc.z += __shfl_xor_sync(kFull, acc.z, o); acc.w += __shfl_xor_sync(kFull, acc.w, o);
    }
    __syncthreads();
    if (lane == 0) s_red[warp] = L;
    if (lane < cgn) s_part[warp][lane] = acc;
    __syncthreads();
    if (tid < cgn) {
        L = 0.f;
        float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int x = 0; x < warps; ++x) {
            L += s_red[x];
            const float4 v = s_part[x][tid];
            t.x += v.x; t.y += v.y; t.z += v.z; t.w += v.w;
        }
        const float inv = L > 0.f ? 1.f / L : 0.f;
        const float4 o = make_float4(t.x * inv, t.y * inv, t.z * inv, t.w * inv);
        if (p.out_fp32) {
            reinterpret_cast<float4*>(p.out)[head * (kD / 4) + chan0 / 4 + tid] = o;
        } else {
            __nv_bfloat162 lo = __floats2bfloat162_rn(o.x, o.y), hi = __floats2bfloat162_rn(o.z, o.w);
            uint2 pk;
            pk.x = *reinterpret_cast<uint32_t*>(&lo);
            pk.y = *reinterpret_cast<uint32_t*>(&hi);
            reinterpret_cast<uint2*>(p.out)[head * (kD / 4) + chan0 / 4 + tid] = pk;
        }
        if (p.lse && tid == 0 && blockIdx.z == 0) p.lse[head] = L > 0.f ? (Mrun + log2f(L)) * kLn2 : -INFINITY;
    }
}

}  // namespace ffd
