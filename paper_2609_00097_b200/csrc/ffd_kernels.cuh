// Device code of the FFD sparse decode-attention path for sm_100a.
//
// Work unit: one (sequence b, KV head g) pair owns the G <= 4 query heads of its GQA group; its cache is a
// list of 64-token blocks, each a contiguous 16 KB K tile, 16 KB V tile, 2 KB of packed 2-bit codes and
// 256 B of fp16 scales.  One warp processes one block at a time:
//   scan   : 2-bit codes -> fp16 subnormal integers (one AND per register), per-block B operand
//            q*scale split in two fp16 pieces, 40 mma.sync.m16n8k16 (tokens x (head,piece) x channels)
//   select : block max per head vs (m_tilde - delta)                                   (Eq. 1, Alg. 1)
//   attend : S^T = Q K^T and O = P V with mma.sync bf16, online softmax in registers   (Alg. 1 refinement)
// Only kept blocks move their K and V: each warp owns one 16 KB K slot and one 16 KB V slot in shared memory,
// filled by 16-byte cp.async copies into an XOR-swizzled layout and tracked by one mbarrier per slot.  The warp
// scans one block ahead, so the next kept block's K (V) copy is issued as soon as the current block's Q K^T
// (P V) has released the slot and overlaps the rest of the work.
// A CTA merges its warps' partial (m, l, acc) in shared memory; a combine kernel merges the splits.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>

namespace ffd {

constexpr int kD = 128;            // head_dim
constexpr int kBlk = 64;           // tokens per block
constexpr int kTileBytes = kBlk * kD * 2;
constexpr int kCodeBytes = kBlk * kD / 4;
constexpr int kWarps = 7;          // warps per decode CTA: 7 x (16 KB K slot + 16 KB V slot) of shared memory
constexpr int kSlotBytes = kTileBytes;
constexpr int kDecodeSmem = kWarps * 2 * kSlotBytes + 128;   // + mbarriers
constexpr uint32_t kSuspendHintNs = 200000u;       // upper bound of one hardware-suspended try_wait
constexpr long long kSpinCycles = 2000000000LL;   // bounded mbarrier wait (~1 s of SM clocks); then report and stop
constexpr int kMaxG = 4;           // query heads per KV head handled by one warp
constexpr unsigned kFull = 0xffffffffu;

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// bound on the relative error of the chained tensor-core accumulation in the fast scan (measured ~2.3e-6)
constexpr float kScanBandRel = 1.2e-5f;

constexpr uint32_t kDevBadPage = 1u;
constexpr uint32_t kDevBadSeqLen = 2u;
constexpr uint32_t kDevTimeout = 4u;
constexpr uint32_t kDevRange = 8u;          // an approximate score left the binary32 range; that block was kept
constexpr uint32_t kDevBadWorkspace = 16u;  // the workspace header was not initialised (or a call was interrupted)

// The workspace header (first 256 bytes): word 0 status, words 16 .. 22 work counters and batch statistics, word 24 a
// cookie that ffd_workspace_init writes.  A kernel that finds another value there knows that the counters were never
// zeroed: it reports kDevBadWorkspace and hands out no work instead of indexing with them.
constexpr uint32_t kHeaderCookie = 0xFFD0B200u;
constexpr int kHeaderCookieWord = 24;

struct DecodeParams {
    const __nv_bfloat16* q;
    const __nv_bfloat16* k_cache;
    const int8_t* k_res;      // 2 + 8 bit key format: residuals of the keys (k_cache is then unused)
    float* res_scores;        // 2 + 8 bit key format: per-token approximate scores of maybe-kept blocks, scan -> attend
    const __nv_bfloat16* v_cache;
    const uint8_t* k_quant;
    const __half* k_scales;
    const int32_t* block_table;
    const int32_t* seq_lens;
    int batch, Hq, Hkv, G, max_blocks, num_pages;   // Hkv, G: the groups the kernels work on (see kv_shift)
    int Hkv_phys, kv_shift;  // KV heads of the caches; a KV head with 6 or 8 query heads is served as 2^kv_shift = 2 groups of
                             // 3 or 4 heads that read the same tiles: group g uses KV head g >> kv_shift
    int n_sink, n_local;
    int blocks_per_split, splits;
    float sm_scale;          // logit scale
    float delta;             // +inf allowed
    uint32_t* status;        // workspace status word
    float* mtilde;           // [B, Hq]   (workspace)
    float* part_ml;          // dense path: [B, Hq, S, 2]   m (log2 domain), l
    float* part_acc;         // dense path: [B, Hq, S, 128]
    unsigned char* qrec;     // [B, Hkv] query records of the scan: fp16 fragments + thresholds (workspace)
    float* fpart_ml;         // fused path: [items, attend warps, 4 heads, 2]
    float* fpart_acc;        // fused path: [items, attend warps, 4 heads, 128]
    int total_items;         // fused path: work items = ceil(max_blocks / 32) * B * Hkv
    uint32_t* item_counter;  // fused path: next heavy-class draw (workspace; zeroed at the start of every call)
    uint32_t* light_counter; // fused path: next light-class draw
    uint32_t* class_counts;  // fused path: [0] heavy units, [1] light units found by the pseudo-max kernel (workspace)
    int32_t* bump_lens;      // append + decode: the caller's seq_lens, set to the new lengths by the combine kernel
    uint32_t* len_stats;     // fused path: [0] largest block count of the batch, [1] largest (max_blocks - block count), [2] items
    int2* unit_list;         // fused path: (unit, its clamped sequence length); heavy units from the front, light units
                             // from the back (workspace)
    int units;               // batch * Hkv
    int item_rows;           // fused path: work items per (sequence, KV head)
    int item_blocks;         // fused path: blocks per full-size item (22 or 32)
    int rows_small;          // fused path: how many of them, counted from block 0, are half-size items
    unsigned long long units_magic, hkv_magic;   // reciprocals for fast_div
    uint8_t* kept_mask;      // nullable [B, Hq, max_blocks]
    float* block_max;        // nullable [B, Hq, max_blocks]
    float* bmax;             // scan kernel -> select kernel: [B, Hq, max_blocks] block maxima of the approximate logits (workspace)
    uint8_t* keep_bits;      // select kernel -> decode kernel: [B, Hkv, max_blocks, 4] bytes, byte h = head h of the group keeps the block (workspace)
    void* out;               // [B, Hq, 128] bf16 or fp32
    float* lse;              // nullable [B, Hq]
    int out_fp32;
};

// ---- small helpers --------------------------------------------------------------------------------------

// Programmatic dependent launch: every kernel of the library lets its successor in the stream be scheduled early
// (pdl_launch_dependents) and itself waits, before it touches anything a predecessor may have written, until the
// predecessor grid has completed and its writes are visible (pdl_wait).  This only hides launch latency.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;\n" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory"); }

__device__ __forceinline__ void mma_f16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                        uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// rows 8..15 of A are zero and rows 8..15 of the result are never used
__device__ __forceinline__ void mma_bf16_top(float& c0, float& c1, uint32_t a0, uint32_t a2, uint32_t b0,
                                             uint32_t b1) {
    float z0 = 0.f, z1 = 0.f;
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(c0), "+f"(c1), "+f"(z0), "+f"(z1)
        : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b0), "r"(b1));
}

// the same with fp16 operands
__device__ __forceinline__ void mma_f16_top(float& c0, float& c1, uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1) {
    float z0 = 0.f, z1 = 0.f;
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(c0), "+f"(c1), "+f"(z0), "+f"(z1)
        : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b0), "r"(b1));
}

// signed 8-bit operands, K = 32, 32-bit integer accumulation; rows 8..15 of A are zero
__device__ __forceinline__ void mma_s8_top(int& c0, int& c1, uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1) {
    int z0 = 0, z1 = 0;
    asm volatile(
        "mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+r"(c0), "+r"(c1), "+r"(z0), "+r"(z1)
        : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b0), "r"(b1));
}

// an ordinary (coherent) 16-byte global load
__device__ __forceinline__ uint4 ldg_plain(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.v4.u32 {%0,%1,%2,%3}, [%4];\n" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ uint4 ldg_stream(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];\n" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(dst), "l"(src) : "memory");
}

// the mbarrier receives one arrival from this thread once all its earlier cp.async copies have landed
__device__ __forceinline__ void cp_async_arrive(uint32_t bar) {
    asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];\n" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void cp_async_drain() { asm volatile("cp.async.wait_all;\n" ::: "memory"); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count) : "memory");
}

// Bounded wait for the phase with the given parity; false when the limit ran out.  The suspend-time hint lets the
// hardware park the warp until the phase completes instead of polling: a waiting warp must not eat the issue
// slots of the warps it is waiting for.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    long long t0 = 0;
    for (;;) {
        uint32_t ok;
        asm volatile(
            "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n selp.u32 %0, 1, 0, p;\n}\n"
            : "=r"(ok)
            : "r"(bar), "r"(parity), "r"(kSuspendHintNs)
            : "memory");
        if (ok) return true;
        const long long now = clock64();
        if (t0 == 0) t0 = now;
        else if (now - t0 > kSpinCycles) return false;
    }
}

// Shared-memory tile layout: token T's 256-byte row keeps its place, its sixteen 16-byte chunks are XOR-ed with
// swz(T) (bits 0..2 only).  With this every quarter-warp of the K and V fragment reads below, and of the copy
// that fills the slot, touches eight different 16-byte bank groups.
__device__ __forceinline__ uint32_t swz(uint32_t token) { return (((token >> 1) & 3u) << 1) ^ ((token & 1u) << 2); }

// Copy one 16 KB (64 tokens x 256 B) tile into a slot: 32 coalesced 512-byte warp copies.
__device__ __forceinline__ void tile_copy_async(uint32_t slot, const uint4* __restrict__ src, int lane, uint32_t bar) {
    const uint32_t half = lane >> 4, c = lane & 15;
#pragma unroll
    for (int it = 0; it < 32; ++it) {
        const uint32_t token = 2 * it + half;
        cp_async16(slot + token * 256 + ((c ^ swz(token)) << 4), src + it * 32 + lane);
    }
    cp_async_arrive(bar);
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

__device__ __forceinline__ float bf16_round(float x) { return __bfloat162float(__float2bfloat16_rn(x)); }

// n / d for n < 2^32 with magic = 2^48 / d + 1 (host-computed): exact while n * d < 2^48
__host__ __device__ __forceinline__ unsigned long long fast_div_magic(unsigned d) {
    return (1ull << 48) / d + 1ull;
}
__device__ __forceinline__ unsigned fast_div(unsigned n, unsigned long long magic) {
    return (unsigned)__umul64hi((unsigned long long)n << 16, magic);
}

// physical page of logical block `blk`; returns -1 (and flags) when the table entry is out of range
__device__ __forceinline__ int page_of(const DecodeParams& p, int b, int blk) {
    int page = p.block_table ? p.block_table[(size_t)b * p.max_blocks + blk] : b * p.max_blocks + blk;
    if (page < 0 || page >= p.num_pages) {
        atomicOr(p.status, kDevBadPage);
        return -1;
    }
    return page;
}

// (page, KV head) tile of group g
__device__ __forceinline__ size_t tile_index(const DecodeParams& p, int page, int g) {
    return (size_t)page * p.Hkv_phys + (g >> p.kv_shift);
}

__device__ __forceinline__ int clamped_seq_len(const DecodeParams& p, int b) {
    int n = p.seq_lens[b];
    int cap = p.max_blocks * kBlk;
    if (n < 0 || n > cap) {
        atomicOr(p.status, kDevBadSeqLen);
        n = n < 0 ? 0 : cap;
    }
    return n;
}

// ---- scan: approximate scores of one block from its 2-bit codes -----------------------------------------
//
// MMA shape: M = 16 tokens, N = 8 = 4 heads x {hi, lo} piece of q*scale, K = 16 channels.
// Lane = 4*r + j.  As a B-fragment owner the lane serves column n = lane/4 = 2*head + piece and the 32
// channels 32j..32j+31; k-step i (0..7) uses channels 32j+4i..32j+4i+3.
//
// A operand: the two code bits of a channel stay where they are in the packed word; masking them out leaves
// the fp16 subnormal code * 4^e * 2^-24 with e = i (i < 5) or i - 5 (after a shift by 10 bits).  The factor
// 4^e is undone by pre-scaling q with 4^(2-e); the level offset -1.5 is applied afterwards from
// sum_c q*scale, which one extra MMA per k-step with A = 4^e * 2^-24 provides.
//
// B operand: v = (q * 4^(2-e)) * scale has at most 8 + 11 significant bits; hi = fp16(v) and
// lo = fma(q, scale, -hi) represent it exactly (barring underflow), so the products are exact and only the
// fp32 accumulation rounds.

struct ScanQuery {
    uint32_t qh[16];  // half2: q of head (lane/8), channels 32j+4i+{0,1} (qh[2i]) and +{2,3} (qh[2i+1]), pre-scaled
    int piece;        // (lane/4) & 1
    float unit;       // accumulator units -> logits for head lane % 4: 2^20 * sm_scale * 2^k of that head
};

__device__ __forceinline__ float scan_pos_scale(int i) {
    const int e = i < 5 ? i : i - 5;
    return e == 0 ? 16.f : e == 1 ? 4.f : e == 2 ? 1.f : e == 3 ? 0.25f : 0.0625f;
}

// Range of the fp16 B operand.  The query of every head is brought into range by an exact power of two before it is
// converted to fp16: k = the smallest integer >= 0 with 16 * max_c |q_c| * 2^-k <= 32, undone in `unit`.  The B operand
// (16 q 2^-k) * s then overflows fp16 only for scales above 2047 (keys beyond +-3000); such a block shows up as a
// non-finite level-offset sum and is redone by scan_block_wide in binary32.  Small products lose low bits to fp16
// underflow, at most 2^-25 absolute per product, i.e. below 2^-30 of the head's largest |q_c| * s_c.
// Returns 2^-k for the head lane / 8; all lanes of that head agree.
__device__ __forceinline__ float scan_query_scale(const uint4 (&raw)[4]) {
    float m = 0.f;
#pragma unroll
    for (int x = 0; x < 4; ++x) {
        const uint32_t wds[4] = {raw[x].x, raw[x].y, raw[x].z, raw[x].w};
#pragma unroll
        for (int y = 0; y < 4; ++y)
            m = fmaxf(m, fmaxf(fabsf(__uint_as_float(wds[y] << 16)), fabsf(__uint_as_float(wds[y] & 0xffff0000u))));
    }
    m = fmaxf(m, __shfl_xor_sync(kFull, m, 1));
    m = fmaxf(m, __shfl_xor_sync(kFull, m, 2));
    int e = 0;
    (void)frexpf(m, &e);                 // m = f * 2^e, f in [0.5, 1): m * 2^-(e-1) < 2
    const int k = min(max(e - 1, 0), 100);
    return __uint_as_float((uint32_t)(127 - k) << 23);
}

// raw: this lane's 32 query values (bf16) of head lane / 8, channels 32j .. 32j + 31 (zero for heads >= G);
// inv = 2^-k of that head
__device__ __forceinline__ void scan_setup_scaled(ScanQuery& sq, const uint4 (&raw)[4], float inv, int lane) {
    sq.piece = (lane >> 2) & 1;
#pragma unroll
    for (int x = 0; x < 4; ++x) {   // 8 contiguous channels 32j + 8x .. + 7 = k-steps 2x and 2x + 1
        const uint32_t wds[4] = {raw[x].x, raw[x].y, raw[x].z, raw[x].w};
#pragma unroll
        for (int y = 0; y < 4; ++y) {
            const float sc = scan_pos_scale(2 * x + (y >> 1)) * inv;
            const float lo = __uint_as_float(wds[y] << 16), hi = __uint_as_float(wds[y] & 0xffff0000u);
            const __half2 v = __floats2half2_rn(lo * sc, hi * sc);
            sq.qh[4 * x + y] = *reinterpret_cast<const uint32_t*>(&v);
        }
    }
}

// Loads the group's queries, picks the power of two per head and builds the fragments.  Returns 2^-k of head lane / 8.
__device__ __forceinline__ float scan_setup(ScanQuery& sq, const __nv_bfloat16* q_group /* [G][128] */, int G,
                                            int lane, float sm_scale) {
    const int head = lane >> 3, j = lane & 3;
    uint4 raw[4];
#pragma unroll
    for (int x = 0; x < 4; ++x) {
        raw[x] = make_uint4(0u, 0u, 0u, 0u);
        if (head < G) raw[x] = *reinterpret_cast<const uint4*>(q_group + head * kD + 32 * j + 8 * x);
    }
    const float inv = scan_query_scale(raw);
    scan_setup_scaled(sq, raw, inv, lane);
    // results come out for head lane % 4: its 2^k sits in the lanes of column head lane % 4, e.g. lane 8 * (lane % 4)
    const float inv_res = __shfl_sync(kFull, inv, 8 * (lane & 3));
    sq.unit = 1048576.0f * sm_scale / inv_res;
    return inv;
}

// Returns, in every lane, the block maximum of the approximate logits (sm_scale applied) of head lane%4
// over the first `rows` tokens of the block.
//
// PRECISE = false chains the 8 k-steps through the tensor-core accumulator.  That accumulation truncates every
// addend when it aligns it, which costs up to a few 1e-5 of a logit at |logit| ~ 40; `band` returns a bound on
// that error.  PRECISE = true starts every k-step from a zero accumulator (alignment then happens at the size of
// single products) and adds the eight partial sums with round-to-nearest fp32 adds; it is used for the
// pseudo-max and for blocks whose fast result lands within `band` of the threshold, so that both decisions rest
// on the same, deterministic, ~1e-5-accurate arithmetic.
struct ScanRegs {
    uint4 w[4];   // packed codes of the four 16-token groups
    uint4 s[4];   // this lane's 32 scales
};

// the same through ordinary loads: for a tile this kernel has itself just written
__device__ __forceinline__ void scan_load_plain(ScanRegs& sr, const uint4* codes_tile, const uint4* scales_tile,
                                                int lane) {
#pragma unroll
    for (int mt = 0; mt < 4; ++mt) sr.w[mt] = ldg_plain(codes_tile + mt * 32 + lane);
#pragma unroll
    for (int x = 0; x < 4; ++x) sr.s[x] = ldg_plain(scales_tile + 4 * (lane & 3) + x);
}

__device__ __forceinline__ void scan_load(ScanRegs& sr, const uint4* __restrict__ codes_tile,
                                          const uint4* __restrict__ scales_tile, int lane) {
#pragma unroll
    for (int mt = 0; mt < 4; ++mt) sr.w[mt] = ldg_stream(codes_tile + mt * 32 + lane);
#pragma unroll
    for (int x = 0; x < 4; ++x) sr.s[x] = __ldg(scales_tile + 4 * (lane & 3) + x);
}

// B operand of four k-step halves: hi / lo piece of (pre-scaled q) * scale for this lane's column
__device__ __forceinline__ void scan_bfrag4(uint32_t* bfrag, const uint4& qv, const uint4& sv, int piece) {
    const uint32_t q[4] = {qv.x, qv.y, qv.z, qv.w};
    const uint32_t sc[4] = {sv.x, sv.y, sv.z, sv.w};
#pragma unroll
    for (int x = 0; x < 4; ++x) {
        const __half2 a = *reinterpret_cast<const __half2*>(&q[x]);
        const __half2 b = *reinterpret_cast<const __half2*>(&sc[x]);
        const __half2 hi = __hmul2(a, b);
        const __half2 lo = __hfma2(a, b, __hneg2(hi));
        const __half2 pick = piece ? lo : hi;
        bfrag[x] = *reinterpret_cast<const uint32_t*>(&pick);
    }
}

// The same, and also sum_c |q_c * s_c| over the lane's channels (fp16, two running pairs): the ingredient of an
// upper bound on every approximate score of the block.  base = index of the first of the four registers (0, 4, 8, 12):
// register idx belongs to k-step idx / 2, whose pre-scaling of q is undone here.
__device__ __forceinline__ void scan_bfrag4_bound(uint32_t* bfrag, const uint4& qv, const uint4& sv, int piece,
                                                  int base, __half2& sum_a, __half2& sum_b) {
    const uint32_t q[4] = {qv.x, qv.y, qv.z, qv.w};
    const uint32_t sc[4] = {sv.x, sv.y, sv.z, sv.w};
#pragma unroll
    for (int x = 0; x < 4; ++x) {
        const __half2 a = *reinterpret_cast<const __half2*>(&q[x]);
        const __half2 b = *reinterpret_cast<const __half2*>(&sc[x]);
        const __half2 hi = __hmul2(a, b);
        const __half2 lo = __hfma2(a, b, __hneg2(hi));
        const __half2 pick = piece ? lo : hi;
        bfrag[x] = *reinterpret_cast<const uint32_t*>(&pick);
        const float undo = 1.0f / scan_pos_scale((base + x) >> 1);
        const __half2 u = __floats2half2_rn(undo, undo);
        if (x & 1) sum_b = __hfma2(__habs2(hi), u, sum_b);
        else sum_a = __hfma2(__habs2(hi), u, sum_a);
    }
}

// sum_c |q_c| s_c over four registers of the lane's channels (fp16, two running pairs; the products are exact
// inside the fused multiply-add)
__device__ __forceinline__ void scan_abs_sum(const uint4& qabs, const uint4& sv, __half2& sum_a, __half2& sum_b) {
    const uint32_t q[4] = {qabs.x, qabs.y, qabs.z, qabs.w};
    const uint32_t sc[4] = {sv.x, sv.y, sv.z, sv.w};
#pragma unroll
    for (int x = 0; x < 4; ++x) {
        const __half2 a = *reinterpret_cast<const __half2*>(&q[x]);
        const __half2 b = *reinterpret_cast<const __half2*>(&sc[x]);
        if (x & 1) sum_b = __hfma2(a, b, sum_b);
        else sum_a = __hfma2(a, b, sum_a);
    }
}

// Upper bound (in logits) on the approximate score of every token of the block for the head this lane's column
// belongs to: |sum_c q_c s_c level_c| <= 1.5 sum_c |q_c s_c|.  The factor 1.02 and the constant cover the fp16
// roundings of the products and of the 16-term running sums (each below 2^-11 relative) and the lo pieces.
// bmul = 1.5 * 1.02 * sm_scale * 2^k of the head, badd = 1e-3 + bmul * 2^-17 (the second term covers products that
// underflowed in fp16: 128 of them, each rounded by at most 2^-25).
__device__ __forceinline__ float scan_bound(__half2 sum_a, __half2 sum_b, float bmul, float badd) {
    const float2 a = __half22float2(sum_a), b = __half22float2(sum_b);
    float s = (a.x + a.y) + (b.x + b.y);
    s += __shfl_xor_sync(kFull, s, 1);
    s += __shfl_xor_sync(kFull, s, 2);
    return fmaf(bmul, s, badd);
}

// unit: accumulator units -> logits for head lane % 4 (ScanQuery::unit).  The result is NaN in every lane when the
// fp16 B operand overflowed for any head of the group (the caller then redoes the block with scan_block_wide).
template <bool PRECISE>
__device__ __forceinline__ float scan_mma(const uint4 (&w)[4], const uint32_t (&bfrag)[16], int lane, int rows,
                                          float unit, float& band, float* tok = nullptr);

template <bool PRECISE>
__device__ __forceinline__ float scan_compute(const ScanRegs& sr, const ScanQuery& sq, int lane, int rows,
                                              float& band) {
    uint32_t bfrag[16];
#pragma unroll
    for (int x = 0; x < 4; ++x)
        scan_bfrag4(bfrag + 4 * x, make_uint4(sq.qh[4 * x], sq.qh[4 * x + 1], sq.qh[4 * x + 2], sq.qh[4 * x + 3]),
                    sr.s[x], sq.piece);
    return scan_mma<PRECISE>(sr.w, bfrag, lane, rows, sq.unit, band);
}

// tok (optional): the approximate logits themselves, tok[2 mt] for token 16 mt + lane/4 and tok[2 mt + 1] for the
// token eight further on, head lane % 4 (rows past `rows` included: the caller masks them).
template <bool PRECISE>
__device__ __forceinline__ float scan_mma(const uint4 (&w)[4], const uint32_t (&bfrag)[16], int lane, int rows,
                                          float unit, float& band, float* tok) {
    const int r = lane >> 2;
    float acc[4][4];
    float off[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int mt = 0; mt < 4; ++mt)
#pragma unroll
        for (int x = 0; x < 4; ++x) acc[mt][x] = 0.f;
    uint4 t[4];   // bits 10..15 of every half moved down to 0..5 (k-steps 5..7)
#pragma unroll
    for (int mt = 0; mt < 4; ++mt) t[mt] = make_uint4(w[mt].x >> 10, w[mt].y >> 10, w[mt].z >> 10, w[mt].w >> 10);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int e = i < 5 ? i : i - 5;
        const uint32_t mask = 0x00030003u << (2 * e);
        const uint32_t one = 0x00010001u << (2 * e);
#pragma unroll
        for (int mt = 0; mt < 4; ++mt) {
            const uint4 src = i < 5 ? w[mt] : t[mt];
            const uint32_t x0 = src.x, x1 = src.y, x2 = src.z, x3 = src.w;
            if (PRECISE) {
                float part[4] = {0.f, 0.f, 0.f, 0.f};
                mma_f16(part, x0 & mask, x1 & mask, x2 & mask, x3 & mask, bfrag[2 * i], bfrag[2 * i + 1]);
#pragma unroll
                for (int x = 0; x < 4; ++x) acc[mt][x] += part[x];
            } else {
                mma_f16(acc[mt], x0 & mask, x1 & mask, x2 & mask, x3 & mask, bfrag[2 * i], bfrag[2 * i + 1]);
            }
        }
        if (PRECISE) {
            float part[4] = {0.f, 0.f, 0.f, 0.f};
            mma_f16(part, one, one, one, one, bfrag[2 * i], bfrag[2 * i + 1]);
            off[0] += part[0];
            off[1] += part[1];
        } else {
            mma_f16(off, one, one, one, one, bfrag[2 * i], bfrag[2 * i + 1]);
        }
    }
    float best = -INFINITY;
    if (rows == kBlk) {
#pragma unroll
        for (int mt = 0; mt < 4; ++mt)
            best = fmaxf(best, fmaxf(acc[mt][0] + acc[mt][1], acc[mt][2] + acc[mt][3]));
    } else {
#pragma unroll
        for (int mt = 0; mt < 4; ++mt) {
            float t0 = acc[mt][0] + acc[mt][1];
            float t1 = acc[mt][2] + acc[mt][3];
            if (16 * mt + r < rows) best = fmaxf(best, t0);
            if (16 * mt + r + 8 < rows) best = fmaxf(best, t1);
        }
    }
    best = fmaxf(best, __shfl_xor_sync(kFull, best, 4));
    best = fmaxf(best, __shfl_xor_sync(kFull, best, 8));
    best = fmaxf(best, __shfl_xor_sync(kFull, best, 16));
    // sum_c (code - 1.5) q s = 2^20 * (acc - 1.5 * off)
    const float o = 1.5f * (off[0] + off[1]);
    band = kScanBandRel * (fabsf(best) + fabsf(o)) * unit;
    // an overflowed B operand (+-inf) makes the level-offset sum of its head infinite or NaN
    if (__any_sync(kFull, !(fabsf(o) < INFINITY))) return __int_as_float(0x7fc00000);
    if (tok) {
#pragma unroll
        for (int mt = 0; mt < 4; ++mt) {
            tok[2 * mt] = (acc[mt][0] + acc[mt][1] - o) * unit;
            tok[2 * mt + 1] = (acc[mt][2] + acc[mt][3] - o) * unit;
        }
    }
    return (best - o) * unit;
}

// ---- deeper thumbnails (4 and 8 bits; App. "Bandwidth Proportionality of Quantization Depth") -------------------
// The same mid-rise construction with 2^b levels +-(k + 1/2).  Physical order of a (page, head) tile: 4 groups of 16
// tokens; inside a group lane = 4 r + j owns 2 b words of 32 bits, k-step after k-step (i = 0 .. 7) the eight codes of its
// MMA A fragment.  The k index of the contraction is a permutation of the channels chosen so that lane j's B operand
// covers the 32 consecutive channels 32 j .. 32 j + 31: k-step i, A register x (x & 1: token r or r + 8; x >> 1: lower or
// upper half of the k-step), element e  <->  token 16 mt + r + 8 (x & 1), channel 32 j + 4 i + 2 (x >> 1) + e.
//   4 bits: one word per k-step; nibble x of the low / high half-word = A register x, element 0 / 1
//   8 bits: two words per k-step; byte n of the low / high half-word of word h = A register 2 h + n, element 0 / 1
// Word n of a lane sits in 16-byte vector n / 4 of the group, the vectors of the 32 lanes side by side (a warp's load
// of one vector is one contiguous 512 bytes): byte offset (((mt V + n / 4) 32 + lane) 4 + n % 4) 4 with V = b / 2.
// A code c stands for level c - (2^b - 1) / 2.  Shifted into the mantissa of fp16 16 (4 bits: unit in the last place
// 1/64, the code at bits 6..9) or 256 (8 bits: 1/4, bits 2..9) a code becomes the number 16 + c or 256 + c exactly, and
// one half2 subtraction of 23.5 or 383.5 (both representable next to those bases, which 1024 + 7.5 would not be) gives
// the level, the A operand; with B = (q 2^-k) * s split in two fp16 pieces the products are exact as in the 2-bit scan.
template <int BITS>
struct WideScan {
    static constexpr int kTileBytes = kBlk * kD * BITS / 8;
    static constexpr int kVec = BITS / 2;              // 16-byte vectors per lane and group of 16 tokens
    __device__ static constexpr int word(int mt, int lane, int n) { return ((mt * kVec + n / 4) * 32 + lane) * 4 + n % 4; }
};

// q of head lane / 8, channels 32 j .. 32 j + 31, scaled by 2^-k only (the deeper scans need no per-k-step factor);
// sq.unit turns accumulator units into logits for head lane % 4
__device__ __forceinline__ void scan_setup_wide(ScanQuery& sq, const __nv_bfloat16* q_group, int G, int lane, float sm_scale) {
    const int head = lane >> 3, j = lane & 3;
    uint4 raw[4];   // channels 32 j .. 32 j + 31 of the head: the four lanes j of a column cover all 128
#pragma unroll
    for (int x = 0; x < 4; ++x) {
        raw[x] = make_uint4(0u, 0u, 0u, 0u);
        if (head < G) raw[x] = *reinterpret_cast<const uint4*>(q_group + head * kD + 32 * j + 8 * x);
    }
    const uint32_t* wds = reinterpret_cast<const uint32_t*>(raw);
    // scale: the same power of two as the 2-bit scan (max over the head's channels)
    float m = 0.f;
#pragma unroll
    for (int y = 0; y < 16; ++y)
        m = fmaxf(m, fmaxf(fabsf(__uint_as_float(wds[y] << 16)), fabsf(__uint_as_float(wds[y] & 0xffff0000u))));
    m = fmaxf(m, __shfl_xor_sync(kFull, m, 1));
    m = fmaxf(m, __shfl_xor_sync(kFull, m, 2));
    int e = 0;
    (void)frexpf(m, &e);
    const int k = min(max(e - 1, 0), 100);
    const float inv = __uint_as_float((uint32_t)(127 - k) << 23);
    sq.piece = (lane >> 2) & 1;
    // B fragment of k-step i for column lane / 4 = (head, piece): registers 2 i and 2 i + 1 = channels 32 j + 4 i .. + 3
#pragma unroll
    for (int y = 0; y < 16; ++y) {
        const __half2 h2 = __floats2half2_rn(__uint_as_float(wds[y] << 16) * inv, __uint_as_float(wds[y] & 0xffff0000u) * inv);
        sq.qh[y] = *reinterpret_cast<const uint32_t*>(&h2);
    }
    const float inv_res = __shfl_sync(kFull, inv, 8 * (lane & 3));
    sq.unit = sm_scale / inv_res;
}

// hint: bring a tile's codes and scales into L2 (one 128-byte line per lane and instruction)
template <int BITS>
__device__ __forceinline__ void wide_prefetch_l2(const unsigned char* codes_tile, const __half* scales_tile, int lane) {
#pragma unroll
    for (int o = 0; o < WideScan<BITS>::kTileBytes; o += 4096)
        asm volatile("prefetch.global.L2 [%0];\n" ::"l"(codes_tile + o + lane * 128));
    if (lane < 2) asm volatile("prefetch.global.L2 [%0];\n" ::"l"(reinterpret_cast<const unsigned char*>(scales_tile) + lane * 128));
}

// Block maximum of the approximate logits of head lane % 4 over the first `rows` tokens, codes and scales read straight
// from global memory (the caller has prefetched the tile into L2), 32 tokens' worth of codes per round of loads.
// PRECISE as in scan_mma.
template <int BITS, bool PRECISE>
__device__ __forceinline__ float scan_wide(const unsigned char* codes_tile, const __half* scales_tile, const ScanQuery& sq,
                                           int lane, int rows, float& band) {
    const int r = lane >> 2, j = lane & 3;
    constexpr int kVec = WideScan<BITS>::kVec;
    constexpr int kGroupsPerRound = 8 / kVec;            // 8 vectors per lane in flight: 4 groups (4 bits) or 2 (8 bits)
    const uint4* src = reinterpret_cast<const uint4*>(codes_tile) + lane;
    uint4 cv[8];
#pragma unroll
    for (int v = 0; v < 8; ++v) cv[v] = ldg_stream(src + v * 32);
    // B operand: hi / lo piece of (q 2^-k) * s for this lane's column, k-step by k-step
    uint32_t bfrag[16];
    {
        uint4 sv[4];
#pragma unroll
        for (int x = 0; x < 4; ++x) sv[x] = __ldg(reinterpret_cast<const uint4*>(scales_tile) + 4 * j + x);
        const uint32_t* sc = reinterpret_cast<const uint32_t*>(sv);
#pragma unroll
        for (int y = 0; y < 16; ++y) {
            const __half2 s2 = *reinterpret_cast<const __half2*>(&sc[y]);
            const __half2 a = *reinterpret_cast<const __half2*>(&sq.qh[y]);
            const __half2 hi = __hmul2(a, s2);
            const __half2 lo = __hfma2(a, s2, __hneg2(hi));
            const __half2 pick = sq.piece ? lo : hi;
            bfrag[y] = *reinterpret_cast<const uint32_t*>(&pick);
        }
    }
    float best = -INFINITY, amax = 0.f;
    bool bad = false;
#pragma unroll
    for (int round = 0; round < 4 / kGroupsPerRound; ++round) {
        if (round > 0) {
#pragma unroll
            for (int v = 0; v < 8; ++v) cv[v] = ldg_stream(src + (round * 8 + v) * 32);
        }
        const uint32_t* wr = reinterpret_cast<const uint32_t*>(cv);
#pragma unroll
        for (int gi = 0; gi < kGroupsPerRound; ++gi) {
            const int mt = round * kGroupsPerRound + gi;
            const uint32_t* w = wr + gi * kVec * 4;
            float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                uint32_t a[4];
                if (BITS == 4) {
                    const __half2 bias = __floats2half2_rn(23.5f, 23.5f);          // 16 + 7.5
#pragma unroll
                    for (int x = 0; x < 4; ++x) {
                        const uint32_t sh = 4 * x <= 6 ? w[i] << (6 - 4 * x) : w[i] >> (4 * x - 6);
                        const uint32_t v = (sh & 0x03C003C0u) | 0x4C004C00u;     // 16 + c
                        const __half2 lv = __hsub2(*reinterpret_cast<const __half2*>(&v), bias);
                        a[x] = *reinterpret_cast<const uint32_t*>(&lv);
                    }
                } else {
                    const __half2 bias = __floats2half2_rn(383.5f, 383.5f);        // 256 + 127.5
#pragma unroll
                    for (int x = 0; x < 4; ++x) {
                        const uint32_t word = w[2 * i + (x >> 1)];
                        const uint32_t sh = (x & 1) ? word >> 6 : word << 2;
                        const uint32_t v = (sh & 0x03FC03FCu) | 0x5C005C00u;     // 256 + c
                        const __half2 lv = __hsub2(*reinterpret_cast<const __half2*>(&v), bias);
                        a[x] = *reinterpret_cast<const uint32_t*>(&lv);
                    }
                }
                if (PRECISE) {
                    float part[4] = {0.f, 0.f, 0.f, 0.f};
                    mma_f16(part, a[0], a[1], a[2], a[3], bfrag[2 * i], bfrag[2 * i + 1]);
#pragma unroll
                    for (int x = 0; x < 4; ++x) acc[x] += part[x];
                } else {
                    mma_f16(acc, a[0], a[1], a[2], a[3], bfrag[2 * i], bfrag[2 * i + 1]);
                }
            }
            const float t0 = acc[0] + acc[1], t1 = acc[2] + acc[3];    // hi + lo piece: token r, token r + 8
            bad |= !(fabsf(t0) < INFINITY) || !(fabsf(t1) < INFINITY);
            if (16 * mt + r < rows) { best = fmaxf(best, t0); amax = fmaxf(amax, fabsf(t0)); }
            if (16 * mt + r + 8 < rows) { best = fmaxf(best, t1); amax = fmaxf(amax, fabsf(t1)); }
        }
    }
    best = fmaxf(best, __shfl_xor_sync(kFull, best, 4));
    best = fmaxf(best, __shfl_xor_sync(kFull, best, 8));
    best = fmaxf(best, __shfl_xor_sync(kFull, best, 16));
    amax = fmaxf(amax, __shfl_xor_sync(kFull, amax, 4));
    amax = fmaxf(amax, __shfl_xor_sync(kFull, amax, 8));
    amax = fmaxf(amax, __shfl_xor_sync(kFull, amax, 16));
    // The level sums are centred (no offset term as in the 2-bit scan), so the accumulators are of the size of the
    // scores themselves; the band follows the largest of them.
    band = 4.f * kScanBandRel * amax * sq.unit;
    if (__any_sync(kFull, bad)) return __int_as_float(0x7fc00000);
    return best * sq.unit;
}

// The scan of one block in plain binary32 on the ordinary lanes, for blocks whose fp16 B operand overflowed (scales
// above ~2000): approx[h][t] = sm_scale * sum_c q[h][c] * s[c] * (code[t][c] - 1.5), fused multiply-adds in channel
// order.  Lane L takes tokens 16 (L / 8) + L % 8 and eight further on.  Returns the block maximum of head lane % 4
// over the first `rows` tokens (NaN or +-inf if binary32 overflowed as well); score_dst (optional): the per-token
// logits, head h token t at score_dst[h * score_stride + t].  Rare by construction, so kept out of line and small.
__device__ __noinline__ float scan_block_wide(const uint4* codes_tile, const __half* scales_tile,
                                              const __nv_bfloat16* q_group, int G, int lane, int rows, float sm_scale,
                                              float* score_dst, int score_stride) {
    const int mt = lane >> 3, r = lane & 7;
    float acc[kMaxG][2];
#pragma unroll
    for (int h = 0; h < kMaxG; ++h) acc[h][0] = acc[h][1] = 0.f;
#pragma unroll 1
    for (int j = 0; j < 4; ++j) {
        const uint4 wv = ldg_plain(codes_tile + mt * 32 + 4 * r + j);
        const uint32_t w[4] = {wv.x, wv.y, wv.z, wv.w};
#pragma unroll 1
        for (int i = 0; i < 8; ++i) {
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int c = 32 * j + 4 * i + u, shift = 2 * i + 16 * (u & 1);
                const float sc = __half2float(scales_tile[c]);
                const float k0 = sc * ((float)((w[(u >> 1) * 2] >> shift) & 3u) - 1.5f);
                const float k1 = sc * ((float)((w[(u >> 1) * 2 + 1] >> shift) & 3u) - 1.5f);
#pragma unroll
                for (int h = 0; h < kMaxG; ++h) {
                    const float qv = h < G ? __bfloat162float(q_group[h * kD + c]) : 0.f;
                    acc[h][0] = fmaf(qv, k0, acc[h][0]);
                    acc[h][1] = fmaf(qv, k1, acc[h][1]);
                }
            }
        }
    }
    const int t0 = 16 * mt + r, t1 = t0 + 8;
    float mine = 0.f;
#pragma unroll
    for (int h = 0; h < kMaxG; ++h) {
        const float a0 = acc[h][0] * sm_scale, a1 = acc[h][1] * sm_scale;
        if (score_dst) {
            score_dst[h * score_stride + t0] = a0;
            score_dst[h * score_stride + t1] = a1;
        }
        float best = -INFINITY;
        bool bad = false;
        if (t0 < rows) { best = fmaxf(best, a0); bad |= !(fabsf(a0) < INFINITY); }
        if (t1 < rows) { best = fmaxf(best, a1); bad |= !(fabsf(a1) < INFINITY); }
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) best = fmaxf(best, __shfl_xor_sync(kFull, best, o));
        if (__any_sync(kFull, bad)) best = __int_as_float(0x7fc00000);   // fmaxf drops a NaN: say so explicitly
        if ((lane & 3) == h) mine = best;
    }
    return mine;
}

// ---- attend: exact attention of one block, online softmax state in registers ------------------------------
//
// S^T = Q K^T : M = 16 rows (row r < 4: head r, row r + 4: the same head again, rows 8..15 zero), N = 8 tokens,
//               K = 16 channels.  A lane (n = lane/4, j) reads 16 contiguous bytes of token n's key per read.
// O = P V     : M = same rows (r < 4 carries the bf16 rounding of P, r + 4 the remainder), N = 8 channels,
//               K = 16 tokens.  V rows are paired in registers with byte permutes.
// Channel order inside the contractions is a fixed permutation chosen so that every shared-memory read is a
// full 16-byte vector of one token row.

struct AttendState {
    uint32_t qa[16];   // A fragments of Q: qa[2s] (k = 2j..2j+1), qa[2s+1] (k = 2j+8..2j+9) of k-step s
    float m;           // running max of row r%4 in the log2 domain (-inf when nothing seen)
    float l;           // this lane's share of the running sum
    float acc[16][2];  // O fragments: n-tile nt, columns 2j, 2j+1
};

// A fragments of the group's queries (rows r < 4 and their duplicates r + 4; heads >= G are zero)
__device__ __forceinline__ void attend_load_q(uint32_t (&qa)[16], const __nv_bfloat16* q_group, int G, int lane) {
    const int r = lane >> 2, j = lane & 3;
    const int head = r & 3;
#pragma unroll
    for (int l4 = 0; l4 < 4; ++l4) {
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (head < G) v = *reinterpret_cast<const uint4*>(q_group + head * kD + 32 * l4 + 8 * j);
        qa[4 * l4 + 0] = v.x; qa[4 * l4 + 1] = v.y; qa[4 * l4 + 2] = v.z; qa[4 * l4 + 3] = v.w;
    }
}

__device__ __forceinline__ void attend_reset(AttendState& st) {
    st.m = -INFINITY;
    st.l = 0.f;
#pragma unroll
    for (int nt = 0; nt < 16; ++nt) st.acc[nt][0] = st.acc[nt][1] = 0.f;
}

__device__ __forceinline__ void attend_setup(AttendState& st, const __nv_bfloat16* q_group, int G, int lane) {
    attend_load_q(st.qa, q_group, G, lane);
    attend_reset(st);
}

__device__ __forceinline__ bool attend_finish(AttendState& st, float (&s)[8][2], uint32_t vslot, uint32_t vbar,
                                              uint32_t& phase, const uint4* next_v, int lane, int rows, bool mine,
                                              float logit_scale_log2);

// keep4: bit h set when head h attends to this block.  rows: valid tokens in the block (1..64).
// The block's K and V tiles are (being) copied into kslot / vslot; kbar / vbar complete when they have landed.
// next_k / next_v: global tiles of the next kept block (nullptr = none); their copies are issued as soon as
// this block has finished reading the respective slot.  Returns false if a wait ran out.
__device__ __forceinline__ bool attend_block(AttendState& st, uint32_t kslot, uint32_t vslot, uint32_t kbar,
                                             uint32_t vbar, uint32_t& phase, const uint4* next_k, const uint4* next_v,
                                             int lane, int rows, unsigned keep4, float logit_scale_log2) {
    const int r = lane >> 2, j = lane & 3;
    const bool mine = (keep4 >> (r & 3)) & 1u;
    if (!mbar_wait(kbar, phase & 1u)) return false;
    float s[8][2];
    {
        const uint32_t swz_k = swz(r);   // token 8*nt + r: the swizzle depends on r only
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            s[nt][0] = s[nt][1] = 0.f;
            const uint32_t row = kslot + (8 * nt + r) * 256;
#pragma unroll
            for (int l4 = 0; l4 < 4; ++l4) {
                const uint4 kv = lds128(row + (((4 * l4 + j) ^ swz_k) << 4));
                mma_bf16_top(s[nt][0], s[nt][1], st.qa[4 * l4 + 0], st.qa[4 * l4 + 1], kv.x, kv.y);
                mma_bf16_top(s[nt][0], s[nt][1], st.qa[4 * l4 + 2], st.qa[4 * l4 + 3], kv.z, kv.w);
            }
        }
    }
    __syncwarp();   // every lane is done reading the K slot
    if (next_k) tile_copy_async(kslot, next_k, lane, kbar);
    return attend_finish(st, s, vslot, vbar, phase, next_v, lane, rows, mine, logit_scale_log2);
}

// Second half of a block: s[nt][x] = q . k of head r % 4 and token 8 nt + 2j + x (rows r and r + 4 hold the same
// values) -> online softmax (log2 domain) -> O += P V.  Issues the copy of the next V tile when the slot is free.
__device__ __forceinline__ bool attend_finish(AttendState& st, float (&s)[8][2], uint32_t vslot, uint32_t vbar,
                                              uint32_t& phase, const uint4* next_v, int lane, int rows, bool mine,
                                              float logit_scale_log2) {
    const int r = lane >> 2, j = lane & 3;
    float mx = -INFINITY;
#pragma unroll
    for (int nt = 0; nt < 8; ++nt)
#pragma unroll
        for (int x = 0; x < 2; ++x) {
            const int tok = 8 * nt + 2 * j + x;
            float t = s[nt][x] * logit_scale_log2;
            t = (mine && tok < rows) ? t : -INFINITY;
            s[nt][x] = t;
            mx = fmaxf(mx, t);
        }
    mx = fmaxf(mx, __shfl_xor_sync(kFull, mx, 1));
    mx = fmaxf(mx, __shfl_xor_sync(kFull, mx, 2));
    const float m_new = fmaxf(st.m, mx);
    const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
    const float alpha = exp2f(st.m - m_use);
    st.m = m_new;
    float psum = 0.f;
    uint32_t pa[8];  // A fragments of P: pa[2kt] (tokens 16kt+2j..), pa[2kt+1] (tokens 16kt+8+2j..)
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
        float p0 = exp2f(s[nt][0] - m_use), p1 = exp2f(s[nt][1] - m_use);
        psum += p0 + p1;
        float h0 = bf16_round(p0), h1 = bf16_round(p1);
        pa[nt] = (r < 4) ? pack_bf16(h0, h1) : pack_bf16(p0 - h0, p1 - h1);
    }
    st.l = st.l * alpha + psum;
#pragma unroll
    for (int nt = 0; nt < 16; ++nt) { st.acc[nt][0] *= alpha; st.acc[nt][1] *= alpha; }
    // O += P V
    if (!mbar_wait(vbar, phase & 1u)) return false;
    if (rows < kBlk) {   // partial tail block: rows past the sequence end must not meet P = 0 as stale NaN / Inf
        for (int c = lane; c < (kBlk - rows) * 16; c += 32)
            asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};\n" ::"r"(vslot + rows * 256 + c * 16), "r"(0u) : "memory");
        __syncwarp();
    }
#pragma unroll
    for (int kt = 0; kt < 4; ++kt) {
        const int t0 = 16 * kt + 2 * j;
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
            uint4 v[4];
#pragma unroll
            for (int tt = 0; tt < 4; ++tt) {
                const int tok = t0 + (tt & 1) + ((tt >> 1) << 3);
                const uint32_t swz_v = (uint32_t)(j << 1) ^ ((uint32_t)(tt & 1) << 2);   // = swz(tok)
                v[tt] = lds128(vslot + tok * 256 + (((8 * hf + r) ^ swz_v) << 4));
            }
            const uint32_t* x0 = reinterpret_cast<const uint32_t*>(&v[0]);
            const uint32_t* x1 = reinterpret_cast<const uint32_t*>(&v[1]);
            const uint32_t* x2 = reinterpret_cast<const uint32_t*>(&v[2]);
            const uint32_t* x3 = reinterpret_cast<const uint32_t*>(&v[3]);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t b0e = __byte_perm(x0[c], x1[c], 0x5410), b1e = __byte_perm(x2[c], x3[c], 0x5410);
                uint32_t b0o = __byte_perm(x0[c], x1[c], 0x7632), b1o = __byte_perm(x2[c], x3[c], 0x7632);
                const int nt = 8 * hf + 2 * c;
                mma_bf16_top(st.acc[nt][0], st.acc[nt][1], pa[2 * kt], pa[2 * kt + 1], b0e, b1e);
                mma_bf16_top(st.acc[nt + 1][0], st.acc[nt + 1][1], pa[2 * kt], pa[2 * kt + 1], b0o, b1o);
            }
        }
    }
    __syncwarp();   // every lane is done reading the V slot
    if (next_v) tile_copy_async(vslot, next_v, lane, vbar);
    phase ^= 1u;
    return true;
}

// ---- attend on the 2 + 8 bit key format (Sec. 3.3: s_final = (q . k_quant + q . k_res) / sqrt(d)) -------------
//
// q . k_quant is not computed again: the scan warp that judged the block wrote its per-token approximate logits
// (all four heads, 64 tokens) to a score tile in global memory, which stays in L2, and the attend warp copies that
// tile along with the residuals ("the computer reuses the selector's estimation results", Sec. 3).  The K slot of a
// kept block holds, instead of the 16 KB bf16 tile: the 8 KB int8 residual tile (token rows of 128 bytes, the two
// 64-byte halves of odd rows swapped so that a quarter-warp's reads cover all banks), the 1152-byte score tile
// (head h, token t at float h * 72 + t: the padding spreads the four heads over the banks) and the 256 bytes of
// scales.
//
// q . k_res: int8 MMA, K = 32.  A lane's B fragments are its two 16-byte reads of token lane/4 (channels 16j..16j+15
// and 64+16j..64+16j+15); the A operand is v_c = q_c * s_c written with two signed 8-bit digits,
// v_c ~ (vmax / 127) * (d0 + d1 / 254): row r < 4 = digit d0 of head r, row r + 4 = digit d1.
constexpr int kScoreStride = 72;                          // floats per head in a score tile
constexpr int kScoreTileFloats = 4 * kScoreStride;        // 1152 bytes
constexpr uint32_t kResOffScores = 8192, kResOffScales = kResOffScores + kScoreTileFloats * 4;

__device__ __forceinline__ void res_copy_async(uint32_t slot, const DecodeParams& p, uint32_t tile, const float* scores,
                                               int lane, uint32_t bar) {
    const uint4* res = reinterpret_cast<const uint4*>(p.k_res + (size_t)tile * (kBlk * kD));
#pragma unroll
    for (int x = 0; x < 16; ++x) {
        const uint32_t idx = x * 32 + lane, t = idx >> 3, c = idx & 7;
        cp_async16(slot + t * 128 + ((c ^ ((t & 1u) << 2)) << 4), res + idx);
    }
    const uint4* sc = reinterpret_cast<const uint4*>(scores);
    cp_async16(slot + kResOffScores + lane * 16, sc + lane);
    cp_async16(slot + kResOffScores + (32 + lane) * 16, sc + 32 + lane);
    if (lane < kScoreTileFloats / 4 - 64) cp_async16(slot + kResOffScores + (64 + lane) * 16, sc + 64 + lane);
    if (lane >= 16)
        cp_async16(slot + kResOffScales + (lane - 16) * 16,
                   reinterpret_cast<const uint4*>(p.k_scales + (size_t)tile * kD) + (lane - 16));
    cp_async_arrive(bar);
}
static_assert(kScoreTileFloats / 4 - 64 <= 16, "score tile: at most 80 chunks");

// Per batch: qb = bf16 q of head r % 4 for the 16 residual channels whose digits this lane works out
// (16j..16j+15 in rows r < 4, 64+16j..64+16j+15 in rows r + 4).
__device__ __forceinline__ void attend_setup_res(AttendState& st, uint32_t (&qb)[8], const DecodeParams& p, int b, int g,
                                                 int lane) {
    const int r = lane >> 2, j = lane & 3, head = r & 3;
    const __nv_bfloat16* qh = p.q + ((size_t)b * p.Hq + (size_t)g * p.G + head) * kD + 64 * (r >> 2) + 16 * j;
#pragma unroll
    for (int x = 0; x < 2; ++x) {
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (head < p.G) v = *reinterpret_cast<const uint4*>(qh + 8 * x);
        qb[4 * x + 0] = v.x; qb[4 * x + 1] = v.y; qb[4 * x + 2] = v.z; qb[4 * x + 3] = v.w;
    }
    attend_reset(st);
}

// v = q * s of the two channels held in one bf16 pair / fp16 pair
__device__ __forceinline__ float2 res_qs(uint32_t q2, uint32_t s2) {
    const float2 sf = __half22float2(*reinterpret_cast<const __half2*>(&s2));
    return make_float2(__uint_as_float(q2 << 16) * sf.x, __uint_as_float(q2 & 0xffff0000u) * sf.y);
}

__device__ __forceinline__ bool attend_block_res(AttendState& st, const uint32_t (&qb)[8], const DecodeParams& p,
                                                 uint32_t kslot, uint32_t vslot, uint32_t kbar, uint32_t vbar,
                                                 uint32_t& phase, int next_tile, const float* next_scores,
                                                 const uint4* next_v, int lane, int rows, unsigned keep4) {
    const int r = lane >> 2, j = lane & 3;
    const bool mine = (keep4 >> (r & 3)) & 1u;
    const int piece = r >> 2;
    if (!mbar_wait(kbar, phase & 1u)) return false;
    float s[8][2];
    {
        // The lanes of rows r and r + 4 need the digits of the same 32 channels of the same head (one the first, the
        // other the second digit): each works out both digits of 16 of them and they swap.  This lane's half:
        // channels 16j..16j+15 (piece 0) or 64+16j..64+16j+15 (piece 1) = registers 4 piece .. 4 piece + 3.
        const uint4 sa = lds128(kslot + kResOffScales + (8 * piece + 2 * j) * 16);
        const uint4 sb = lds128(kslot + kResOffScales + (8 * piece + 2 * j + 1) * 16);
        const uint32_t s2[8] = {sa.x, sa.y, sa.z, sa.w, sb.x, sb.y, sb.z, sb.w};
        float2 v[8];
        float vmax = 0.f;
#pragma unroll
        for (int y = 0; y < 8; ++y) {
            v[y] = res_qs(qb[y], s2[y]);
            vmax = fmaxf(vmax, fmaxf(fabsf(v[y].x), fabsf(v[y].y)));
        }
        vmax = fmaxf(vmax, __shfl_xor_sync(kFull, vmax, 1));
        vmax = fmaxf(vmax, __shfl_xor_sync(kFull, vmax, 2));
        vmax = fmaxf(vmax, __shfl_xor_sync(kFull, vmax, 16));
        const float inv = vmax > 0.f ? 127.f / vmax : 0.f, step = vmax * (1.f / 127.f);
        const float inv1 = inv * 254.f;
        constexpr float kMagic = 12582912.f;   // 1.5 * 2^23: adding it leaves rint(x) in the low mantissa bits
        uint32_t adig[8];   // register rho: channels 4 rho .. 4 rho + 3 of the 32, this row's digit in every byte
#pragma unroll
        for (int x = 0; x < 4; ++x) {
            uint32_t b0[4], b1[4];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const float2 vv = v[2 * x + h];
                const float t0x = fmaf(vv.x, inv, kMagic), t0y = fmaf(vv.y, inv, kMagic);
                b0[2 * h] = __float_as_uint(t0x);
                b0[2 * h + 1] = __float_as_uint(t0y);
                b1[2 * h] = __float_as_uint(fmaf(fmaf(-(t0x - kMagic), step, vv.x), inv1, kMagic));
                b1[2 * h + 1] = __float_as_uint(fmaf(fmaf(-(t0y - kMagic), step, vv.y), inv1, kMagic));
            }
            const uint32_t d0 = __byte_perm(__byte_perm(b0[0], b0[1], 0x0040), __byte_perm(b0[2], b0[3], 0x0040), 0x5410);
            const uint32_t d1 = __byte_perm(__byte_perm(b1[0], b1[1], 0x0040), __byte_perm(b1[2], b1[3], 0x0040), 0x5410);
            // keep this row's digit of the own half, hand the other digit to the partner and take its half
            const uint32_t got = __shfl_xor_sync(kFull, piece ? d0 : d1, 16);
            const uint32_t own = piece ? d1 : d0;
            adig[x] = piece ? got : own;
            adig[4 + x] = piece ? own : got;
        }
        // digits -> logits: v ~ step * (d0 + d1 / 254); a residual step is s / 254 (s is inside v)
        const float unit = p.sm_scale * step * (1.f / 254.f) * (piece ? 1.f / 254.f : 1.f);
        const uint32_t flip = (uint32_t)(r & 1) << 2;   // token 8 nt + r: odd rows have their halves swapped
        const uint32_t score_row = kslot + kResOffScores + ((r & 3) * kScoreStride + 2 * j) * 4;
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            const uint32_t row = kslot + (8 * nt + r) * 128;
            const uint4 k0 = lds128(row + ((j ^ flip) << 4)), k1 = lds128(row + (((j + 4) ^ flip) << 4));
            int d0 = 0, d1 = 0;
            mma_s8_top(d0, d1, adig[0], adig[1], k0.x, k0.y);
            mma_s8_top(d0, d1, adig[2], adig[3], k0.z, k0.w);
            mma_s8_top(d0, d1, adig[4], adig[5], k1.x, k1.y);
            mma_s8_top(d0, d1, adig[6], adig[7], k1.z, k1.w);
            // the scan's approximate logit (the q . k_quant term) is added once, in the rows of the first digit
            float a0, a1;
            asm volatile("ld.shared.v2.f32 {%0,%1}, [%2];\n" : "=f"(a0), "=f"(a1) : "r"(score_row + nt * 32));
            s[nt][0] = fmaf((float)d0, unit, piece ? 0.f : a0);
            s[nt][1] = fmaf((float)d1, unit, piece ? 0.f : a1);
        }
    }
    __syncwarp();   // every lane is done reading the K slot
    if (next_tile >= 0) res_copy_async(kslot, p, (uint32_t)next_tile, next_scores, lane, kbar);
    // rows r and r + 4 hold the two digits' shares of the same head: both get the sum
#pragma unroll
    for (int nt = 0; nt < 8; ++nt) {
        s[nt][0] += __shfl_xor_sync(kFull, s[nt][0], 16);
        s[nt][1] += __shfl_xor_sync(kFull, s[nt][1], 16);
    }
    return attend_finish(st, s, vslot, vbar, phase, next_v, lane, rows, mine, kLog2e);
}

// output channel of O fragment (n-tile nt, column n)
__device__ __forceinline__ int attend_channel(int nt, int n) { return 64 * (nt >> 3) + 8 * n + (nt & 7); }

}  // namespace ffd
