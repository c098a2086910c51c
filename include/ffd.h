/*
 * ffd.h - C ABI of the B200 (sm_100a) FFD sparse decode-attention library.
 *
 * The library implements one decode step of "Faster Than Flash" (FFD) for one attention layer:
 * keys are kept twice, as 16-bit K and as a 2-bit mid-rise "thumbnail" with per-channel scales; a step
 * scans the thumbnails of every 64-token block, skips blocks whose best approximate score lies more than
 * delta below a pseudo-max taken from the sink and local blocks, and runs exact softmax attention over the
 * kept blocks only.
 *
 * Conventions for every entry point
 *   - All data pointers are DEVICE pointers, 16-byte aligned, owned by the caller; `cfg` and output
 *     size pointers are HOST pointers.  The library allocates no device memory.  It keeps no state between calls
 *     apart from two things that are documented where they are declared: the event pair of ffd_profile_events and the
 *     per-device address of the scratch array of ffd_decode_static.  Everything else a call needs from an earlier
 *     one (zeroed work counters) lives in the caller's workspace.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls only enqueue work;
 *     nothing synchronizes except ffd_read_device_status.
 *   - Host-detectable problems return a non-zero ffd_status and launch nothing.
 *   - Layouts (row-major, innermost last), D = head_dim = 128, BLK = block_tokens = 64:
 *       q        bf16  [batch, num_q_heads, D]
 *       k_cache  bf16  [num_pages, num_kv_heads, BLK, D]     (v_cache the same)
 *       k_quant  u8    [num_pages, num_kv_heads, 1024 * quant_bits]  packed codes (2048 bytes per tile for the
 *                                                            2-bit thumbnails), physical order below
 *       k_scales fp16  [num_pages, num_kv_heads, D]          one scale per (page, KV head, channel)
 *       block_table int32 [batch, max_blocks_per_seq]        logical block -> physical page;
 *                                                            NULL = page b*max_blocks_per_seq + blk
 *       seq_lens int32 [batch]                               tokens in each sequence (0 allowed)
 *     Token t of sequence b lives in logical block t/64, row t%64.  Query head h uses KV head
 *     h / (num_q_heads / num_kv_heads).  Group sizes G = num_q_heads / num_kv_heads: 1, 2, 3, 4, and also 6 and 8 in
 *     ffd_workspace_bytes, ffd_workspace_init, ffd_quantize_keys, ffd_unpack_codes, ffd_decode, ffd_decode_dense and
 *     ffd_decode_select.  A KV head with 6 or 8 query heads is served as two groups of 3 or 4 heads that read the same
 *     tiles, so its codes and kept K/V tiles are read twice (same results as a kernel with wider fragments would give,
 *     twice the traffic); the other entry points return FFD_ERR_UNSUPPORTED for G > 4, every entry point for G = 5, 7
 *     and G > 8.
 *   - Physical order of k_quant: a (page, head) tile is 4 groups of 16 tokens, 512 bytes each.  Inside a
 *     group, 32 lanes own 16 bytes each: lane = 4*r + j holds 32-bit words W0..W3 for tokens r (W0, W2)
 *     and r+8 (W1, W3) of the group.  Bits [2i+1:2i] of the low / high half of W0 (W1) hold the codes of
 *     channels 32j+4i and 32j+4i+1; those of W2 (W3) hold channels 32j+4i+2 and 32j+4i+3 (i = 0..7).
 *     A code c in 0..3 stands for level c - 1.5.  ffd_unpack_codes returns the canonical form.
 *   - Deeper thumbnails, quant_bits = 4 or 8 (the quantization-depth study of the appendix "Bandwidth Proportionality
 *     of Quantization Depth").  The paper states no quantizer for them; the library continues the 2-bit construction:
 *     2^b levels +-(k + 1/2) * s, k = 0 .. 2^(b-1) - 1, s = fp16_rne(min(fp32(absmax) / (2^(b-1) - 1/2), 65504)) (the
 *     outermost level at the channel's absolute maximum, as 1.5 s is for 2 bits), nearest level with ties outward, +-0
 *     to +1/2, an all-zero channel coded with the outermost positive level; a code c in 0 .. 2^b - 1 stands for level
 *     c - (2^b - 1) / 2.  Physical order of a (page, head) tile: 4 groups of 16 tokens; inside a group lane = 4*r + j
 *     owns 2*b 32-bit words.  Word n of the lane is at byte offset ((((mt*V + n/4)*32 + lane)*4 + n%4)*4 of the tile
 *     (mt = group, V = b/2).  4 bits: word i (i = 0..7) holds, in nibble x of its low / high half, the codes of token
 *     16*mt + r + 8*(x&1), channels 32j + 4i + 2*(x>>1) and that channel + 1.  8 bits: words 2i and 2i+1; byte n of the
 *     low / high half of word 2i + h holds token 16*mt + r + 8*n, channels 32j + 4i + 2h and + 1.  Supported by
 *     ffd_quantize_keys, ffd_unpack_codes, ffd_workspace_bytes, ffd_workspace_init, ffd_decode, ffd_decode_dense and
 *     ffd_read_device_status; the entry points of the 2 + 8 bit key format, of the device-side append and
 *     ffd_decode_static return FFD_ERR_UNSUPPORTED for them.  The scan forms q * s in fp16 after scaling each head's
 *     query to below 2 in magnitude: blocks whose scales exceed about 30000 overflow it, are kept and reported with
 *     FFD_DEV_RANGE (the 2-bit scan falls back to binary32 there instead).
 */
#ifndef FFD_H_
#define FFD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    FFD_OK = 0,
    FFD_ERR_NULL = 1,          /* a required pointer is NULL */
    FFD_ERR_SHAPE = 2,         /* batch / heads / block counts out of range */
    FFD_ERR_UNSUPPORTED = 3,   /* head_dim != 128, block_tokens != 64, quant_bits not 2, 4 or 8 (or not 2 where the entry
                                  point needs the 2-bit thumbnails), group size not 1..4 (6 and 8 where the
                                  conventions above say so) ... */
    FFD_ERR_ALIGN = 4,         /* a device pointer is not 16-byte aligned */
    FFD_ERR_WORKSPACE = 5,     /* workspace smaller than ffd_workspace_bytes reports */
    FFD_ERR_DELTA = 6,         /* delta is NaN or negative */
    FFD_ERR_CUDA = 7,          /* a CUDA runtime call failed (launch error, wrong device ...) */
    FFD_ERR_DEVICE_STATUS = 8, /* a kernel recorded a problem in the workspace status word */
    FFD_ERR_STATIC_LIMIT = 9   /* ffd_decode_static: the geometry needs more scratch than the built-in array holds */
} ffd_status;

/* bits of the device status word (ffd_read_device_status) */
#define FFD_DEV_BAD_PAGE 1u     /* a block_table entry was outside [0, num_pages); that block was skipped */
#define FFD_DEV_BAD_SEQ_LEN 2u  /* a seq_len was negative or above max_blocks_per_seq*64; clamped */
#define FFD_DEV_TIMEOUT 4u      /* a bounded wait for an asynchronous copy ran out; that split's result is incomplete */
#define FFD_DEV_RANGE 8u        /* an approximate score left the binary32 range (non-finite); that block was kept */
#define FFD_DEV_BAD_WORKSPACE 16u /* the workspace header was never initialised (ffd_workspace_init), or an interrupted
                                     call left its work counters behind: no work was handed out, `out` is undefined */

typedef struct {
    int32_t num_q_heads;
    int32_t num_kv_heads;
    int32_t head_dim;        /* 128 */
    int32_t block_tokens;    /* 64 */
    int32_t quant_bits;      /* 2 (the paper's thumbnails), 4 or 8 (deeper thumbnails, see above) */
    int32_t n_sink_blocks;   /* size of the sink set S_global in blocks (>= 0) */
    int32_t n_local_blocks;  /* size of the local set S_local in blocks, counted from the last block (>= 0);
                                n_sink_blocks + n_local_blocks must be >= 1 */
    float sm_scale;          /* 0 => 1/sqrt(head_dim) */
    int32_t out_dtype;       /* 0: bf16 output, 1: fp32 output */
} ffd_config;

const char* ffd_status_string(ffd_status status);

/* Bytes of device workspace ffd_decode / ffd_decode_dense need for this geometry.  A host computation; the split
 * geometry follows the SM count of the current CUDA device (148, a B200's, when no device can be asked), so ask
 * with the device current on which the workspace will be used. */
ffd_status ffd_workspace_bytes(const ffd_config* cfg, int32_t batch, int32_t max_blocks_per_seq, size_t* bytes);

/* The same for ffd_decode_residual: the workspace of ffd_decode for this geometry followed by the tiles in which the
 * scan leaves the approximate scores of kept blocks for the refinement (about 57 MB, independent of the geometry).
 * Such a workspace serves every other call too. */
ffd_status ffd_workspace_bytes_residual(const ffd_config* cfg, int32_t batch, int32_t max_blocks_per_seq,
                                        size_t* bytes);

/* Zeroes the header of a freshly allocated workspace (status word, work counters) and marks it as initialised.  Call
 * once before the first decode with that workspace.  The status word is sticky across calls until
 * ffd_read_device_status clears it; the work counters are put back to zero by the last kernel of every completed
 * ffd_decode, for the next call.  If a decode call was interrupted (a CUDA error), call this again before reusing the
 * workspace.  A decode on a workspace that was never initialised, or whose counters an interrupted call left behind,
 * is detected on the device: it hands out no work, stores nothing out of range and reports FFD_DEV_BAD_WORKSPACE. */
ffd_status ffd_workspace_init(void* workspace, size_t workspace_bytes, void* stream);

/*
 * Cache append: quantize keys to 2-bit thumbnails (App. A.1, "Symmetric Mid-rise Uniform Quantization").
 * For every sequence b, every logical block that holds a token in [first_token[b], seq_lens[b]) is
 * (re)quantized over its valid rows r < min(64, seq_lens[b] - 64*blk): per channel
 *   s = fp16_rne(min(fp32(max_r |K[r,c]|) / 1.5f, 65504)),  code = x<0 ? (|x|>=s ? 0 : 1) : (|x|>=s ? 3 : 2)
 * (the nearest level of {-1.5,-0.5,+0.5,+1.5}*s; ties go outward, +-0 to +0.5).  Codes of rows past the
 * sequence end are unspecified.  first_token NULL means 0 (quantize everything).  K must be finite (no NaN: the
 * whole-cache path and the first_token path would code a NaN differently; +-inf is handled like a large value).
 * Writes k_quant and k_scales of the touched (page, head) tiles only.  Blocks whose block_table entry is
 * outside [0, num_pages) are skipped; a seq_len outside [0, max_blocks_per_seq*64] is clamped.
 */
ffd_status ffd_quantize_keys(const ffd_config* cfg, const void* k_cache, void* k_quant, void* k_scales,
                             const int32_t* block_table, const int32_t* seq_lens, const int32_t* first_token,
                             int32_t batch, int32_t max_blocks_per_seq, int32_t num_pages, void* stream);

/*
 * 8-bit residual of the keys (Sec. 3.1: the key cache is split into 2-bit thumbnails k_quant and 8-bit residuals
 * k_res; Alg. 1 "Dequant").  The paper prints no residual quantizer; this one puts the remainder of every valid
 * element on a symmetric 8-bit grid over the cell of its 2-bit level, whose half-width is s/2 (s = the channel's
 * scale in k_scales):
 *   r = x - (code - 1.5) * s,   k_res = clamp(rint(r * (254 / s)), -127, 127),   0 when s = 0
 * with every operation one IEEE binary32 operation (round to nearest even).  The rebuilt key
 * (code - 1.5) * s + k_res * s / 254 is within s/508 of x.  Rows past the sequence end get 0.
 *   k_res  int8 [num_pages, num_kv_heads, 64, 128] (device, row-major, same indexing as k_cache)
 * Call after ffd_quantize_keys on the same stream with the same block_table / seq_lens / first_token: it reads
 * k_cache and k_scales and (re)writes k_res of the blocks that hold a token in [first_token[b], seq_lens[b]).
 * Other arguments, skipped pages, clamping and host errors as for ffd_quantize_keys.
 */
ffd_status ffd_quantize_residual(const ffd_config* cfg, const void* k_cache, const void* k_scales, void* k_res,
                                 const int32_t* block_table, const int32_t* seq_lens, const int32_t* first_token,
                                 int32_t batch, int32_t max_blocks_per_seq, int32_t num_pages, void* stream);

/*
 * ffd_quantize_keys and ffd_quantize_residual in one call.  With first_token (a decode step: only the block the
 * newest token fell into is redone) both are written by a single kernel launch; without it the two whole-cache
 * kernels run one after the other.  Results equal those of the two separate calls.
 */
ffd_status ffd_quantize_keys_residual(const ffd_config* cfg, const void* k_cache, void* k_quant, void* k_scales,
                                      void* k_res, const int32_t* block_table, const int32_t* seq_lens,
                                      const int32_t* first_token, int32_t batch, int32_t max_blocks_per_seq,
                                      int32_t num_pages, void* stream);

/*
 * Cache append for one decode step, all indices on the device (Sec. 3.3: a cache that a captured graph can replay
 * needs tensor indices instead of host-side lengths; App. A.1 for the quantizer).  For every sequence b with
 * pos = seq_lens[b] < max_blocks_per_seq*64: the rows k_new[b, g, :] and v_new[b, g, :] (bf16 [B, Hkv, 128], device)
 * are written to token position pos of k_cache / v_cache (block pos/64 through block_table, row pos%64), that
 * block's thumbnails (k_quant, k_scales) are re-quantized over its rows 0 .. pos%64 exactly as ffd_quantize_keys
 * would, and seq_lens[b] becomes pos + 1.  A sequence with no room left is left untouched and reported in the status
 * word (FFD_DEV_BAD_SEQ_LEN); if the block_table entry for the block is outside [0, num_pages) the rows are not
 * written and FFD_DEV_BAD_PAGE is reported, but the length still advances (a decode skips such a block anyway).
 * workspace: device memory of at least 256 bytes whose first word is the status word (a decode workspace will do).
 * Asynchronous on `stream`; two kernel launches; allocates nothing; may be captured in a CUDA graph together with
 * the decode call that follows it.  Host errors as for ffd_quantize_keys (FFD_ERR_WORKSPACE if workspace_bytes < 256).
 */
ffd_status ffd_append_kv(const ffd_config* cfg, const void* k_new, const void* v_new, void* k_cache, void* v_cache,
                         void* k_quant, void* k_scales, const int32_t* block_table, int32_t* seq_lens, int32_t batch,
                         int32_t max_blocks_per_seq, int32_t num_pages, void* workspace, size_t workspace_bytes,
                         void* stream);

/*
 * ffd_append_kv for the 2 + 8 bit key format: the residuals (k_res) of the block the new token falls into are redone
 * together with its thumbnails, in the same two launches.  Everything else as for ffd_append_kv.
 */
ffd_status ffd_append_kv_residual(const ffd_config* cfg, const void* k_new, const void* v_new, void* k_cache,
                                  void* v_cache, void* k_quant, void* k_scales, void* k_res, const int32_t* block_table,
                                  int32_t* seq_lens, int32_t batch, int32_t max_blocks_per_seq, int32_t num_pages,
                                  void* workspace, size_t workspace_bytes, void* stream);

/*
 * One sparse decode step (Alg. 1; Sec. 3.2 Eq. 1 and the pseudo-max equation; Sec. 3.3 kernel steps).
 * Per query head h of sequence b, with sm = sm_scale and khat = (code - 1.5) * scale:
 *   approx[t]  = sm * sum_c q[c] * khat[t,c]                      every valid token t
 *   bm[blk]    = max of approx over the block's valid tokens
 *   m_tilde    = max of bm over blocks blk < n_sink_blocks or blk >= nb - n_local_blocks
 *   keep[blk]  = bm[blk] >= m_tilde - delta                        (delta = +inf keeps every block)
 *   out        = softmax over tokens of kept blocks of (sm * q . K[t]) applied to V;  lse = log-sum-exp
 * K and V of a block are read if any query head of the KV group keeps it; a head gives zero weight to
 * blocks it did not keep.  seq_len 0 gives out = 0 and lse = -inf.
 *   out       [batch, num_q_heads, D], bf16 or fp32 per cfg->out_dtype; bf16 is the rounding of the fp32 result
 *   lse       nullable fp32 [batch, num_q_heads]
 *   kept_mask nullable u8 [batch, num_q_heads, max_blocks_per_seq]: 0/1 for blk < nb, others untouched
 *   block_max nullable fp32 [batch, num_q_heads, max_blocks_per_seq]: bm (same validity)
 * delta must be >= 0 or +inf.  Arithmetic: approximate scores are binary32-accurate (tensor-core products of
 * exact fp16 operands, binary32 accumulation: error of a few 2^-24 of sm * sum_c |q[c]| * scale[c], the precise
 * re-scan of blocks near the threshold included); exact scores bf16 x bf16 -> fp32; P.V with P split in two bf16
 * pieces.  Input range: q, K and V must be finite.  Every magnitude of q is handled (each head's query is scaled by
 * an exact power of two before it becomes an fp16 operand, undone afterwards); blocks with a scale above ~2000 (keys
 * beyond +-3000) leave the tensor-core path and are scored in binary32 on the ordinary lanes, same result, slower.
 * If an approximate score leaves the binary32 range altogether the block is kept and FFD_DEV_RANGE is reported.
 * Device-detected problems (bad page index, seq_len beyond max_blocks_per_seq*64) skip / clamp the
 * offending work and set bits in the workspace status word; nothing traps.
 */
ffd_status ffd_decode(const ffd_config* cfg, const void* q, const void* k_cache, const void* v_cache,
                      const void* k_quant, const void* k_scales, const int32_t* block_table,
                      const int32_t* seq_lens, int32_t batch, int32_t max_blocks_per_seq, int32_t num_pages,
                      float delta, void* out, float* lse, uint8_t* kept_mask, float* block_max, void* workspace,
                      size_t workspace_bytes, void* stream);

/*
 * The decode step under one of the comparison selection rules (Fig. 1; Sec. 4.4 "Selection-Rule Overhead"; Sec. 5.2),
 * for measuring what each rule costs and keeps next to the paper's own.  Same arguments, outputs, errors and workspace as
 * ffd_decode, at every quantization depth; always runs as three kernels (scan of all blocks into the workspace, the rule,
 * attention over the kept blocks), also where ffd_decode would fuse them.  rule:
 *   FFD_RULE_PSEUDO_MAX   keep a block iff its maximum approximate score >= m_tilde - delta (Alg. 1, Eq. 1; what
 *                         ffd_decode computes)
 *   FFD_RULE_GLOBAL_MAX   ... >= (maximum over all blocks of the head) - delta: needs the whole scan before any decision
 *   FFD_RULE_RUNNING_MAX  ... >= max(m_tilde, maxima of blocks 0 .. blk) - delta: the reference a streaming scan in logical
 *                         block order has when it meets block blk; a function of the inputs only, whatever the split
 *                         geometry of the kernels
 *   FFD_RULE_TOP_K        the top_k blocks of each head by maximum approximate score (>= 1; blocks equal to the k-th value
 *                         are all kept; top_k >= the head's block count keeps everything); delta is not used
 * The kept sets are nested: global max within running max within pseudo-max.  `mtilde` in the workspace, kept_mask and
 * block_max are written as by ffd_decode (block_max is NaN for a block whose page index is bad).
 */
#define FFD_RULE_PSEUDO_MAX 0
#define FFD_RULE_GLOBAL_MAX 1
#define FFD_RULE_RUNNING_MAX 2
#define FFD_RULE_TOP_K 3
ffd_status ffd_decode_select(const ffd_config* cfg, int32_t rule, int32_t top_k, const void* q, const void* k_cache,
                             const void* v_cache, const void* k_quant, const void* k_scales, const int32_t* block_table,
                             const int32_t* seq_lens, int32_t batch, int32_t max_blocks_per_seq, int32_t num_pages,
                             float delta, void* out, float* lse, uint8_t* kept_mask, float* block_max, void* workspace,
                             size_t workspace_bytes, void* stream);

/*
 * The same step on the 2 + 8 bit key format (Sec. 3.3, "Fine-grained refinement": a block that passes the filter
 * loads its 8-bit residual keys and its values; s_final = (q . k_quant + q . k_res) / sqrt(d), both dot products
 * accumulated without a full-precision key).  Selection is exactly ffd_decode's; the refined logit of a kept token is
 *   sm * sum_c q[c] * ((code - 1.5) * s[c] + k_res[t,c] * s[c] / 254)
 * so a kept block costs 8 KB of k_res + 16 KB of V instead of 32 KB, and the 16-bit keys are not read at all.  The
 * q . k_quant term is the scan's own per-token result, handed from the scanning to the refining warps through
 * score tiles in the workspace (1.1 KB per kept block, L2-resident), as Sec. 3 describes ("the computer reuses the
 * selector's estimation results").  k_res as written by ffd_quantize_residual; workspace_bytes at least
 * ffd_workspace_bytes_residual (FFD_ERR_WORKSPACE otherwise; FFD_ERR_UNSUPPORTED on a GPU with more than 192 SMs);
 * every other argument, the outputs and the error behaviour as for ffd_decode.  Arithmetic: q . k_quant as in the
 * scan (exact fp16 tensor-core products, fp32 accumulation); q . k_res with int8 tensor-core products of k_res and
 * q[c] * s[c] split into two 8-bit digits (relative error below 2^-15 of the largest |q[c] * s[c]| per channel).
 */
ffd_status ffd_decode_residual(const ffd_config* cfg, const void* q, const void* k_res, const void* v_cache,
                               const void* k_quant, const void* k_scales, const int32_t* block_table,
                               const int32_t* seq_lens, int32_t batch, int32_t max_blocks_per_seq, int32_t num_pages,
                               float delta, void* out, float* lse, uint8_t* kept_mask, float* block_max,
                               void* workspace, size_t workspace_bytes, void* stream);

/*
 * One serving step in a single call: ffd_append_kv followed by ffd_decode on the lengthened sequences, with the
 * append folded into the first kernel of the decode (three launches instead of five; Sec. 3.3).  Arguments as for
 * those two calls; k_cache, v_cache, k_quant, k_scales are written (the new rows, the re-quantized tail block) and
 * seq_lens[b] becomes seq_lens[b] + 1 for every sequence that had room.  While the call runs, its kernels take the
 * new lengths from the workspace; the caller's seq_lens array is updated by the last kernel.  A sequence without
 * room is decoded at its old length and reported (FFD_DEV_BAD_SEQ_LEN).  Results equal those of the two separate
 * calls.  Asynchronous, allocation-free, capturable in a CUDA graph.
 */
ffd_status ffd_append_decode(const ffd_config* cfg, const void* k_new, const void* v_new, const void* q, void* k_cache,
                             void* v_cache, void* k_quant, void* k_scales, const int32_t* block_table,
                             int32_t* seq_lens, int32_t batch, int32_t max_blocks_per_seq, int32_t num_pages,
                             float delta, void* out, float* lse, uint8_t* kept_mask, float* block_max, void* workspace,
                             size_t workspace_bytes, void* stream);

/*
 * Dense decode attention over every valid token (the exact baseline the paper compares against in
 * Sec. 4.2): out = softmax(sm * q K^T) V, split over the sequence and merged.  Same layouts as ffd_decode.
 */
ffd_status ffd_decode_dense(const ffd_config* cfg, const void* q, const void* k_cache, const void* v_cache,
                            const int32_t* block_table, const int32_t* seq_lens, int32_t batch,
                            int32_t max_blocks_per_seq, int32_t num_pages, void* out, float* lse, void* workspace,
                            size_t workspace_bytes, void* stream);

/*
 * Canonical view of the packed thumbnails (App. A.1 codebook index): codes u8 [num_pages, num_kv_heads, 64, 128]
 * with values 0..3, level = code - 1.5.  Used to compare codes bit for bit with another implementation.
 */
ffd_status ffd_unpack_codes(const ffd_config* cfg, const void* k_quant, uint8_t* codes, int32_t num_pages,
                            void* stream);

/* Waits for `stream`, copies the workspace status word to *status_bits (HOST) and clears it on the device.
 * Returns FFD_ERR_DEVICE_STATUS if any bit was set. */
ffd_status ffd_read_device_status(void* workspace, void* stream, uint32_t* status_bits);

/*
 * ffd_decode without a caller-supplied workspace and without any allocation.  (The paper has no counterpart to
 * this entry point; it exists for integration reasons only.)
 *
 * Who needs it: callers that are not in a position to obtain device memory at the time they want to decode - a
 * serving loop whose device memory was handed out completely at start-up and whose request path must not call
 * cudaMalloc, or a plug-in whose host application gives it streams and tensors but no allocator.  ffd_decode asks
 * such a caller for a workspace it cannot produce; this variant brings its own.
 *
 * The scratch is one array of FFD_STATIC_SCRATCH_BYTES bytes that is part of the library image: every GPU that
 * loads the library sets that much memory aside until the process exits, whether or not this function is ever
 * called.  The function computes exactly what ffd_decode computes (same kernels, same split geometry; results are
 * bit-identical), with the same arguments minus kept_mask / block_max / workspace.  It calls no cudaMalloc, cudaFree
 * or other allocating routine.
 *
 * Limits and rules
 *   - Geometry: ffd_workspace_bytes(cfg, batch, max_blocks_per_seq) must not exceed FFD_STATIC_SCRATCH_BYTES,
 *     otherwise FFD_ERR_STATIC_LIMIT is returned and nothing is launched.  With 32 query / 8 KV heads on a 148-SM
 *     GPU the 8 MiB hold batch 1 up to about 113 K tokens of context, batch 4 up to about 27 K, batch 16 up to about
 *     6 K (ask ffd_workspace_bytes for the exact figure of a geometry).
 *   - First use on a device: the first call made while a given device is current looks up the device address of
 *     the array (cudaGetSymbolAddress) and remembers it.  Make that first call during start-up, outside of any
 *     stream capture.
 *   - One array for everybody: all calls on a device share the scratch, and it keeps whatever the previous call
 *     left in it.  The function rewrites the parts that must start at zero itself (a small kernel at the start of
 *     every call clears the status word and the work counters), but two calls whose kernels overlap on the GPU
 *     (different streams, or different host threads) overwrite each other's partial results.  Issue calls that can overlap through ffd_decode with
 *     separate workspaces instead.
 *   - Device-detected problems (bad page index, seq_len out of range) are skipped exactly as in ffd_decode, but the
 *     status word lives in the private scratch and cannot be read back: validate such inputs on the caller's side.
 */
#define FFD_STATIC_SCRATCH_BYTES (8u << 20)
ffd_status ffd_decode_static(const ffd_config* cfg, const void* q, const void* k_cache, const void* v_cache,
                             const void* k_quant, const void* k_scales, const int32_t* block_table,
                             const int32_t* seq_lens, int32_t batch, int32_t max_blocks_per_seq, int32_t num_pages,
                             float delta, void* out, float* lse, void* stream);

/*
 * Measurement hook (process-wide, not thread-safe): while both events are
 * non-NULL, ffd_decode and ffd_decode_dense record `start` right before and `stop` right after their fused
 * scan-select-attend kernel on the call's stream, so a benchmark can time that kernel alone.  Both are
 * cudaEvent_t passed as void*; pass NULL, NULL to switch the hook off.  No counterpart in the paper.
 */
ffd_status ffd_profile_events(void* start_event, void* stop_event);

#ifdef __cplusplus
}
#endif
#endif /* FFD_H_ */
