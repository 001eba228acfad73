/*
 * moqae.h - C ABI of the B200 (sm_100a) MoQAE inference hot path.
 *
 * The library implements, as CUDA kernels, the three inference-time steps of MoQAE
 * (Section 3.1 of the paper: input chunks -> per-block quantisation strategy -> quantised
 * KV -> attention):
 *   moqae_route        chunk-wise router, Section 3.2 Eq. 1 and Eq. 2, with routing freezing
 *                      and routing sharing of Section 3.4
 *   moqae_quantize_kv  quantise + bit-pack each chunk at its routed width into per-width pools
 *   moqae_decode_attn  decode attention over the mixed-precision cache, dequantising inside
 *                      the kernel (Limitations section: keys are dequantised before the
 *                      product with the query)
 *
 * General rules
 *   - Every function returns an int: MOQAE_OK (0) or a negative MOQAE_ERR_* code.  Argument
 *     errors are found on the host before anything is launched.
 *   - Unless a parameter says "host", every pointer is a DEVICE pointer owned by the caller.
 *     The library allocates no device memory and keeps no per-call state; work is enqueued on
 *     the caller's stream (a cudaStream_t passed as void*) and the call returns without
 *     synchronising.  Calls on the same cache must be ordered by the caller (same stream or
 *     events).
 *   - Device pointers must be 16-byte aligned.
 *   - No C++ types or exceptions cross this boundary.
 *
 * Fixed by this build: head_dim = 128, quantisation group = 32, experts = 4 with bit widths
 * {2, 4, 8, 16} at expert indices {0, 1, 2, 3}, chunk a multiple of 32 or one of the short
 * sizes 8 and 16, 32 <= d_in and d_in a multiple of 32, n_q_heads / n_kv_heads in {1, .., 8}.
 * Error state: the code of the last failed CUDA runtime call is kept per host thread
 * (moqae_last_cuda_error); nothing else outlives a call.
 *
 * Storage format of the cache (what moqae_quantize_kv writes and moqae_decode_attn reads)
 *   tile   = 32 consecutive tokens of one chunk and one kv head.
 *   quantised tile, b in {2, 4, 8} bits, 1024 + 1024*b bytes:
 *       [   0,  256)  key scale    fp16 x 128   (one per channel, over the tile's 32 tokens)
 *       [ 256,  512)  key zero     fp16 x 128
 *       [ 512,  768)  value scale  fp16 x 128   (4 channel groups of 32 x 32 tokens)
 *       [ 768, 1024)  value zero   fp16 x 128
 *       [1024, 1024+512b)         key payload
 *       [1024+512b, 1024+1024b)   value payload
 *     Inside each part the order is the one in which the 32 lanes of the decode kernel consume
 *     it (lane = 4*g + t4), so that every lane reads whole 16-byte units:
 *     Key payload.  Token t = 16*blk + 8*hh + g, channel c = 32*q + cc.  The 32 codes of one
 *       (t, q) form a piece of 4b bytes, code cc at bits [b*cc, b*cc + b) of the piece read as a
 *       little-endian bit string.  Pieces sit in 16-byte units; unit index
 *         b = 2:  32*blk + 4*g + q,                   hh selects bytes [8hh, 8hh + 8) of the unit
 *         b = 4:  32*(2*blk + hh) + 4*g + q
 *         b = 8:  32*(2*(2*blk + hh) + j) + 4*g + q,  j = which 16 bytes of the piece.
 *     Value payload.  Token t = 16*blk + 8*half + 2*t4 + e, channel c = 32*cg + 4*g + r4.
 *       Lane 4*g + t4 owns, per blk, the 16 channel rows R = 4*cg + r4; row R sits in the lane's
 *       little-endian 32-bit word w = R*b/8 at slot R mod (8/b), its code at bit
 *       b*slot + 8*half + 16*e.  Word w is at byte ((blk*(b/2) + w/4)*32 + lane)*16 + (w mod 4)*4.
 *     Key scale / zero.  With n = 32/b codes per payload word, channel c = 32*q + cc is code
 *       i = cc mod n of word j = cc / n; let i mod (n/2) = s*(n/4) + m and r = j*(n/2) + s*(n/4) + m;
 *       halfword index = ((r/4)*4 + q)*8 + p*2 + (i >= n/2), with p = r mod 4 for the scales and
 *       p = (0, 2, 1, 3)[r mod 4] for the zeros.
 *     Value scale of (cg, t): halfword (((blk*2 + cg/2)*4 + t4)*4 + (cg mod 2)*2 + half)*2 + e.
 *     Value zero  of (cg, t): halfword (((blk*4 + cg)*4 + t4)*2 + half)*2 + e.
 *     Dequantised value = code * scale + zero.
 *   16-bit tile, 16384 bytes: 32 key rows then 32 value rows of 256 bytes in the input dtype;
 *     16-byte unit U of row t is stored at (U & 8) | ((U xor t) & 7).
 *   slot   = the chunk/32 tiles of one chunk and one kv head, in token order.  A chunk of 8 or 16
 *     tokens is ONE tile: its tokens sit at token positions 0 .. chunk-1, the other positions are
 *     padding (codes 0, value scale and zero 0, raw rows 0) that no kernel attends to, and its key
 *     scale / zero of a channel are taken over the chunk's own tokens.  moqae_prefill_attn and
 *     moqae_project_quantize_kv refuse such configurations (MOQAE_ERR_UNSUPPORTED).
 *   pool[w] = [n_layers][batch][n_kv_heads][capacity[w]] slots of width w.
 *   map/slot/count/votes tables are per routing-sharing group: [n_groups][rows][max_chunks]
 *     (count: [n_groups][rows][4], votes: [n_groups][rows][max_chunks][4]),
 *     n_groups = ceil(n_layers / rs_group), max_chunks = max_tokens / chunk, rows = batch, or
 *     batch * n_kv_heads with per-head routing (cfg->per_head_routing).
 *   tail_k / tail_v = [n_layers][batch][n_kv_heads][tail_capacity][128] rows in the input
 *     dtype (tokens that do not fill a chunk stay 16-bit, Section 3.2); tail_len =
 *     int32 [n_layers][batch].
 */
#ifndef MOQAE_H
#define MOQAE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define MOQAE_OK 0
#define MOQAE_ERR_INVALID_ARG (-1)
#define MOQAE_ERR_UNSUPPORTED (-2)
#define MOQAE_ERR_MISALIGNED (-3)
#define MOQAE_ERR_POOL_FULL (-4)
#define MOQAE_ERR_WORKSPACE_TOO_SMALL (-5)
#define MOQAE_ERR_CUDA (-6)
#define MOQAE_ERR_TIMEOUT (-7)
#define MOQAE_ERR_CORRUPT_TABLE (-8)

#define MOQAE_DTYPE_FP16 0
#define MOQAE_DTYPE_BF16 1

#define MOQAE_N_EXPERTS 4
#define MOQAE_N_CACHE_BUFFERS 12

/* Problem description shared by every call (plain data, passed by pointer, host memory). */
typedef struct moqae_config {
  int32_t n_layers;
  int32_t n_q_heads;
  int32_t n_kv_heads;
  int32_t head_dim;        /* 128 */
  int32_t chunk;           /* tokens per chunk, multiple of 32 */
  int32_t group;           /* 32 */
  int32_t dtype;           /* MOQAE_DTYPE_* of hidden states, K, V, q, W1, W2 */
  int32_t n_experts;       /* 4 */
  int32_t expert_bits[4];  /* {2, 4, 8, 16} */
  int32_t rs_group;        /* routing sharing: consecutive layers per group (>= 1) */
  int32_t rf_first_chunk;  /* routing freezing: 1 = chunk 0 is fixed to the 16-bit expert */
  int32_t d_in;            /* router input width */
  int32_t max_tokens;      /* largest context the tables are sized for */
  int32_t tail_capacity;   /* rows per (layer, batch, kv head) in the 16-bit tail */
  int32_t batch;
  int32_t per_head_routing; /* 0: one map per (group, sequence), shared by all kv heads (router input =
                               the block's hidden state).  1: one map per (group, sequence, kv head),
                               routed on that head's own 128-wide rows (Section 3.2: D = the
                               embedding dimension within each attention head): d_in must be 128,
                               hidden is [batch][T][n_kv_heads][128], and map / slot / count /
                               votes have batch * n_kv_heads rows per group, row b * n_kv_heads + h */
} moqae_config;

/* View of a cache: device pointers supplied by the caller (see moqae_cache_bytes for sizes). */
typedef struct moqae_cache {
  void* pool[4];
  int64_t capacity[4];     /* slots per (layer, batch, kv head) in pool[w] */
  uint8_t* map;            /* expert index per chunk */
  int32_t* slot;           /* slot of each chunk inside its width's pool */
  int32_t* count;          /* chunks per width */
  int32_t* votes;          /* Eq. 2 histograms */
  void* tail_k;
  void* tail_v;
  int32_t* tail_len;
  int32_t* status;         /* int32[4]: sticky device-side error code and two detail words */
} moqae_cache;

/* Library version, major*10000 + minor*100 + patch. */
int moqae_version(void);

/* Last CUDA runtime error code seen by a call that returned MOQAE_ERR_CUDA (0 if none). */
int moqae_last_cuda_error(void);

/* Static string for an error code (host pointer, never NULL). */
const char* moqae_error_string(int code);

/*
 * Sizes in bytes of the twelve cache buffers for `cfg` and per-width capacities (host
 * arrays): out_bytes[0..3] pools, [4] map, [5] slot, [6] count, [7] votes, [8] tail_k,
 * [9] tail_v, [10] tail_len, [11] status.  Pure host arithmetic.
 */
int moqae_cache_bytes(const moqae_config* cfg, const int64_t capacity[4],
                      int64_t out_bytes[MOQAE_N_CACHE_BUFFERS]);

/*
 * Fill `out` from twelve device pointers in the order of moqae_cache_bytes; checks
 * alignment.  Allocates nothing.  The caller must have zeroed count, tail_len and status.
 */
int moqae_cache_bind(const moqae_config* cfg, const int64_t capacity[4],
                     void* const buffers[MOQAE_N_CACHE_BUFFERS], moqae_cache* out);

/*
 * Router of one routing-sharing group (Section 3.2, Eq. 1 and Eq. 2; Section 3.4).
 *   hidden  [batch][T][d_in] input-dtype rows of the group's FIRST layer; with per-head routing
 *           [batch][T][n_kv_heads][128] (token-major), head h of sequence b being routed on its own
 *           rows into table row b * n_kv_heads + h.
 *   W1, W2  [d_in][4] input dtype; W3 [4][4] float32 row-major; bias [4] float32.
 *           W2 = W3 = NULL selects the linear router P = C W1 + bias; all non-NULL selects
 *           Eq. 1, P = SiLU((C W1) * (C W2)) W3 + bias.  bias may be NULL (zero).
 *   Each token takes its arg-max expert, each chunk the expert most tokens chose (ties: the
 *   lower index, i.e. the narrower width).  With cfg->rf_first_chunk chunk 0 is not routed and
 *   is the 16-bit expert.  The T mod chunk trailing tokens are not routed.
 *   Writes map, slot, count and votes of group `layer_group`; if votes_out is not NULL it
 *   also receives the group's [batch][T/chunk][4] int32 histograms (compact).
 *   Products are exact, sums are float32 in an unspecified order.
 */
int moqae_route(const moqae_config* cfg, const void* hidden, int32_t T, const void* W1,
                const void* W2, const float* W3, const float* bias, int32_t layer_group,
                const moqae_cache* cache, int32_t* votes_out, void* stream);

/*
 * Quantise and pack the keys and values of one layer (prefill).
 *   K, V [batch][T][n_kv_heads][128] input dtype.
 *   forced_map: NULL = use the map routed for the layer's group; otherwise uint8
 *   [rows][T/chunk] expert indices (rows as in the tables above) that REPLACE the group's map
 *   (slot and count are recomputed) before quantising.
 *   Chunk c of sequence b goes to pool[map] slot `slot[b][c]` of every kv head; trailing
 *   T mod chunk tokens are copied to the tail and tail_len[layer][b] is set.
 *   A chunk whose slot index is >= capacity is skipped and status[0] becomes
 *   MOQAE_ERR_POOL_FULL (read it with moqae_poll_status).
 *   Quantiser: group-wise asymmetric min-max, group 32 (keys per channel over the tile's
 *   tokens, values per token over 32 channels); zero = largest fp16 <= min,
 *   (-0 stored as +0), scale = smallest fp16 >= (max - zero)/(2^b - 1),
 *   code = rint((x - zero) * (1/scale)): subtraction, division and reciprocal are single
 *   binary32 operations, the product is rounded once, to the nearest integer (halves to even).
 *   Inputs must be finite with |x| < 32752.
 */
int moqae_quantize_kv(const moqae_config* cfg, const void* K, const void* V, int32_t T,
                      int32_t layer, const uint8_t* forced_map, const moqae_cache* cache,
                      void* stream);

/*
 * The K and V projections of one layer fused with moqae_quantize_kv (Section 3.1: the chunks are
 * quantised with the configuration the router has just determined, then the block goes on with
 * its computation): K = hidden Wk^T and V = hidden Wv^T are computed on the tensor cores, rounded
 * to the input dtype exactly as a separate projection would have stored them, and quantised and
 * packed from the accumulators; the 16-bit K/V rows never exist in device memory.
 *   hidden [batch][T][d_in] input dtype (the block's hidden states, the router's input);
 *   Wk, Wv [n_kv_heads * 128][d_in] input dtype, row-major (one row per output channel);
 *   products accumulate in float32 in an unspecified order; d_in must be a multiple of 64.
 *   forced_map, chunk placement, the tail and POOL_FULL reporting are those of
 *   moqae_quantize_kv applied to the rounded K and V.
 *   k_rounded, v_rounded: both NULL, or [batch][T][n_kv_heads][128] input-dtype buffers that
 *   receive the rounded rows as well (for checking; costs the traffic the fusion saves).
 */
int moqae_project_quantize_kv(const moqae_config* cfg, const void* hidden, const void* Wk,
                              const void* Wv, int32_t T, int32_t layer, const uint8_t* forced_map,
                              const moqae_cache* cache, void* k_rounded, void* v_rounded,
                              void* stream);

/*
 * Append one decoded token per sequence to the 16-bit tail of `layer` (tokens that do not
 * fill a chunk stay 16-bit, Section 3.2).  k_new, v_new [batch][n_kv_heads][128].  A full
 * tail sets status[0] = MOQAE_ERR_POOL_FULL and drops the token.
 */
int moqae_append_kv(const moqae_config* cfg, const void* k_new, const void* v_new,
                    int32_t layer, const moqae_cache* cache, void* stream);

/*
 * Turn the full 16-bit tails of one routing-sharing group into one more routed, quantised
 * chunk during generation.  Section 3.2 keeps the tokens that do not fill a chunk in 16 bits;
 * once `chunk` tokens have been appended they are a complete chunk and go through the same
 * router (Eq. 1, Eq. 2) and quantiser as a prefill chunk.  (The paper does not say when this
 * happens during decoding; this call is the reading "as soon as the chunk is complete".)
 *   hidden_tail [batch][chunk][d_in] input dtype: the hidden states (router inputs of the group's
 *   first layer) of the tail's tokens, buffered by the caller as the tokens were generated.
 *   W1, W2, W3, bias as in moqae_route.
 *   A sequence takes part only if tail_len of the group's first layer equals `chunk` exactly;
 *   the others are left untouched.  For a participating sequence the new chunk gets index
 *   n = chunks so far, map[n] = winner of the vote (16-bit if n = 0 and rf_first_chunk),
 *   slot[n] / count are updated, the tails of ALL layers of the group are packed into that slot
 *   of their pools, and their tail_len becomes 0.  Needs tail_capacity >= chunk.  A full table or
 *   pool sets status[0] = MOQAE_ERR_POOL_FULL and leaves the sequence untouched.
 */
int moqae_flush_tail(const moqae_config* cfg, const void* hidden_tail, const void* W1, const void* W2,
                     const float* W3, const float* bias, int32_t layer_group, const moqae_cache* cache,
                     void* stream);

/*
 * Bytes of scratch moqae_decode_attn needs for `cfg` on the current device (host out).
 * Layout: float [batch][n_q_heads][n_splits][130] split partials, then int32
 * [batch][n_kv_heads] arrival counters.
 */
int moqae_decode_attn_workspace(const moqae_config* cfg, int64_t* out_bytes);

/*
 * One decode step of attention for one layer: for every query head h,
 *   out[b][h] = softmax(scale * K̂ q[b][h]) V̂   over all cached tokens of kv head
 *   h / (n_q_heads / n_kv_heads), K̂ and V̂ being the dequantised cache rows plus the tail.
 *   q [batch][n_q_heads][128] input dtype; out [batch][n_q_heads][128] float32;
 *   scale <= 0 selects 1/sqrt(128).  An empty cache gives zeros.
 *   workspace: at least moqae_decode_attn_workspace bytes, 16-byte aligned.  ZERO IT ONCE after
 *   allocating it (cudaMemsetAsync on the same stream is enough): the arrival counters at its end
 *   must be zero when a call starts, and every completed call leaves them zero, so no call
 *   clears them and consecutive calls may reuse the buffer as it is.  The partials in front of
 *   them are plain scratch.  Zero the buffer again after a call that ended in
 *   MOQAE_ERR_TIMEOUT and before using it with a different configuration.
 *   Domain: q finite with |q| < 2^40; cache contents as moqae_quantize_kv writes them.  Inside
 *   that domain no intermediate leaves the fp16 range: each query row is normalised by a power
 *   of two before it meets the key scales, and the softmax weights are kept <= 2 before they
 *   meet the value scales.
 */
int moqae_decode_attn(const moqae_config* cfg, const void* q, int32_t layer,
                      const moqae_cache* cache, float* out, float scale, void* workspace,
                      int64_t workspace_bytes, void* stream);

/*
 * moqae_decode_attn with flags (flags = 0 is moqae_decode_attn).
 *   MOQAE_DECODE_OVERLAP_PREVIOUS: the launch is made with programmatic stream serialisation, so
 *   its CTAs may start while the kernel enqueued on `stream` directly before it is still
 *   finishing (they take the SM slots that kernel frees), which hides launch latency, the start-up
 *   of the copy pipelines and the uneven finish of the previous kernel's CTAs.  q, the cache
 *   tables, pools and tail are then READ before that previous kernel is known to be complete; out
 *   and workspace are touched only after it is.  The caller therefore promises that the kernel
 *   directly before this call on the stream does not write anything this call reads - true for a
 *   run of decode calls over different layers (Limitations section: the attention over the
 *   quantised cache is the cost that grows with the context), false directly after
 *   moqae_append_kv, moqae_quantize_kv or moqae_flush_tail of the same cache.  Any other bit in
 *   flags: MOQAE_ERR_INVALID_ARG.
 */
#define MOQAE_DECODE_OVERLAP_PREVIOUS 1
int moqae_decode_attn_ex(const moqae_config* cfg, const void* q, int32_t layer,
                         const moqae_cache* cache, float* out, float scale, void* workspace,
                         int64_t workspace_bytes, int32_t flags, void* stream);

/*
 * One generation step of a layer without touching the cache: moqae_decode_attn_ex that also
 * attends to the CURRENT token's own key / value rows k_new, v_new [batch][n_kv_heads][128]
 * (input dtype), taken as the 16-bit row that would follow the tail (Section 3.2: tokens that do
 * not fill a chunk stay 16-bit).  The result equals moqae_append_kv followed by
 * moqae_decode_attn, but nothing is written to the cache, so the call reads nothing a previous
 * decode call writes and a whole step (layer after layer) can be chained with
 * MOQAE_DECODE_OVERLAP_PREVIOUS; the rows are appended afterwards with moqae_append_kv, at any
 * time before the layer's next step.  k_new = v_new = NULL gives moqae_decode_attn_ex.
 */
int moqae_decode_attn_step(const moqae_config* cfg, const void* q, const void* k_new,
                           const void* v_new, int32_t layer, const moqae_cache* cache, float* out,
                           float scale, void* workspace, int64_t workspace_bytes, int32_t flags,
                           void* stream);

/*
 * Causal attention of the prompt over its own quantised cache (Section 3.1: a block quantises
 * its chunks, then carries out its attention; Limitations section: keys are dequantised to
 * 16-bit floats before the product with the query).  For every position t < T and query head h
 *   out[b][t][h] = softmax(scale * K̂[0..t] q[b][t][h]) V̂[0..t]
 * over kv head h / (n_q_heads / n_kv_heads), K̂ and V̂ being the cache rows in token order
 * (chunk c from pool map[c], slot slot[c]; then the 16-bit tail), each rounded to fp16 after
 * dequantisation; probabilities are rounded to fp16 too, products accumulate in float32.
 *   q   [batch][T][n_q_heads][128] input dtype;  out [batch][T][n_q_heads][128] float32.
 *   T must be the number of tokens the cache of `layer` holds for every sequence
 *   (chunks * chunk + tail_len), i.e. call it after moqae_quantize_kv of the same prompt.
 *   scale <= 0 selects 1/sqrt(128).
 *   workspace: NULL, or caller-owned device scratch of at least moqae_prefill_attn_workspace()
 *   bytes (2 * batch * n_kv_heads * round_up(T, 128) * 256), 16-byte aligned.  With a workspace the
 *   layer's cache is expanded once into fp16 rows there and every CTA fetches its blocks from it
 *   (faster: without it each CTA expands the packed tiles it walks over again, but no extra
 *   memory is needed).  Both ways compute the same quantity; the workspace holds nothing the
 *   caller needs afterwards.  Errors: MOQAE_ERR_WORKSPACE_TOO_SMALL, MOQAE_ERR_MISALIGNED,
 *   MOQAE_ERR_INVALID_ARG (T outside [0, max_tokens], bad layer, missing pointers).
 */
int moqae_prefill_attn_workspace(const moqae_config* cfg, int32_t T, int64_t* bytes);
int moqae_prefill_attn(const moqae_config* cfg, const void* q, int32_t T, int32_t layer,
                       const moqae_cache* cache, float* out, float scale, void* workspace,
                       int64_t workspace_bytes, void* stream);

/*
 * (No counterpart in the paper: this entry point exists for deployment reasons only.)
 * moqae_decode_attn for callers that cannot allocate device memory - for example a plug-in
 * inside a server whose device memory is entirely owned by the host application, a control
 * loop that bans allocator calls once it is running, or a binding that can forward pointers
 * but has no allocator.  Such callers cannot provide the `workspace` of moqae_decode_attn,
 * so the split partials go to a fixed array inside the library image instead:
 * moqae_decode_attn_static_max_bytes() bytes (4 MiB), present on every device that loads the
 * library until the process ends.
 *   - Arguments, results and error codes are those of moqae_decode_attn without the two
 *     workspace arguments.  A configuration whose moqae_decode_attn_workspace size exceeds
 *     the fixed array is refused with MOQAE_ERR_WORKSPACE_TOO_SMALL before anything runs.
 *   - Nothing is allocated or freed, by this library or through any other one.
 *   - The first call on each device looks up the array's device address (that device must be
 *     current, as for every call); make that first call outside any stream capture.
 *   - All calls on one device share the one array, and it keeps whatever the previous call
 *     left there.  The only part that must start at zero, the arrival counters, is cleared by
 *     every call (a memset node on the caller's stream in front of the kernel); the partials are
 *     overwritten before they are read.  Two calls that overlap on the GPU (different streams,
 *     no ordering) race on the array: order them.
 */
int64_t moqae_decode_attn_static_max_bytes(void);
int moqae_decode_attn_static(const moqae_config* cfg, const void* q, int32_t layer,
                             const moqae_cache* cache, float* out, float scale, void* stream);

/*
 * Debugging aid: check the chunk index tables of one routing-sharing group against the rules
 * the kernels rely on (the slot rule of the storage format above: chunks of one width occupy
 * slots 0, 1, 2, .. of that width's pool in chunk order).  For every table row and its first
 * n_chunks chunks: map[c] is an expert index 0..3; slot[c] equals the number of earlier chunks
 * of the row with the same width; slot[c] < capacity[width]; count[w] equals the number of chunks
 * of width w.  The kernels never follow a slot beyond its pool (they report MOQAE_ERR_POOL_FULL
 * or clamp), but a table that breaks these rules means chunks overwrite each other or are skipped.
 *   moqae_validate_tables_host: map / slot / count are HOST arrays of one group laid out as the
 *   device tables ([rows][max_chunks], count [rows][4]); pure host arithmetic.
 *   moqae_validate_tables: copies the group's tables from the device (waits for `stream`) and
 *   runs the same check; T is the context the tables describe (n_chunks = T / chunk).
 * Returns MOQAE_OK or MOQAE_ERR_CORRUPT_TABLE; *bad_row / *bad_chunk (host, may be NULL) receive
 * the first offending position.
 */
int moqae_validate_tables_host(const uint8_t* map, const int32_t* slot, const int32_t* count,
                               int32_t rows, int32_t max_chunks, int32_t n_chunks,
                               const int64_t capacity[4], int32_t* bad_row, int32_t* bad_chunk);
int moqae_validate_tables(const moqae_config* cfg, const moqae_cache* cache, int32_t T,
                          int32_t layer_group, void* stream, int32_t* bad_row, int32_t* bad_chunk);

/*
 * Synchronous read of the cache's device status word: *out_status (host) receives MOQAE_OK
 * or the first device-side error recorded since the buffer was zeroed.  Waits for `stream`.
 */
int moqae_poll_status(const moqae_cache* cache, void* stream, int32_t* out_status);

#ifdef __cplusplus
}
#endif
#endif /* MOQAE_H */
