/*
 * libspecstream - streamed-KV verification attention for speculative decoding (C ABI).
 *
 * One verification round of one layer: the T_q candidate queries of every request
 * (pending committed token + drafts), times the GQA group, attend to the request's
 * committed KV history as it arrives chunk by chunk, plus the on-GPU candidate KV
 * under a chain or tree mask.  Each chunk is read from HBM once and serves every
 * query of the round; it yields per-row partial states (m, l, a) that are merged by
 * online softmax, so the result equals full attention over [history ; candidates].
 * A bit-exact commit-gather appends the accepted candidates' KV to the committed
 * buffer.  (Paper Section 4.2: Eq. 12 defines the result, Eq. 13 the per-chunk
 * state, Eq. 14 the merge, Eq. 17 the equivalence; Section 4.1 the commit rule.)
 *
 * Conventions
 *  - All tensor pointers are DEVICE pointers unless a comment says HOST.  Element type
 *    of Q/K/V/O is bf16 (16-bit words); LSE is fp32.
 *  - ss_tensor strides are in ELEMENTS; the innermost (head-dim) axis is contiguous,
 *    base pointers and all strides are multiples of 8 elements (16 bytes).
 *  - Ownership: the caller owns every tensor and the workspace.  The library allocates
 *    no device memory on these calls and keeps no caller pointer after finalize,
 *    except Q between begin and finalize.
 *  - Asynchrony: every call validates its arguments on the host, enqueues work on the
 *    given CUDA stream and returns; results are valid once the stream reaches that
 *    point.  All calls of one round must use the same stream.
 *    Nothing synchronises or allocates, so a whole round can be recorded into a CUDA graph
 *    by stream capture and replayed (the call-order state machine runs at capture time).
 *  - Call order per round: begin -> {chunk | local}* -> finalize.  Chunks may come in
 *    any order and any number (including zero); local at most once.  Anything else
 *    returns SS_ERR_STATE.  ss_verify_abort drops an open round.
 *  - Errors: host-detectable problems return a code and enqueue nothing.  Problems only
 *    the device can see (valid_len outside [0, L_c], accept index outside [0, T_loc),
 *    destination overflow, a bounded wait that expired) set a status word in the
 *    workspace, skip the offending item, never trap; read it with ss_poll_status.
 *  - Threads: a context holds the state of one round at a time and is not thread-safe; calls
 *    on one context from several host threads must be serialised by the caller.  Different
 *    contexts (each with its own workspace) are independent and may be used concurrently.
 *  - Determinism: same inputs, same call sequence, same config -> bitwise-same output.
 *  - A query row with no visible key yields O = 0 and LSE = -inf.
 */
#ifndef SPECSTREAM_H_
#define SPECSTREAM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ss_ctx ss_ctx; /* opaque */

typedef enum {
  SS_OK = 0,
  SS_ERR_ARG = 1,         /* null pointer, non-positive size */
  SS_ERR_SHAPE = 2,       /* exceeds the limits given at ss_create, H_q % H_kv, d not in {64,128} */
  SS_ERR_ALIGN = 3,       /* base or stride not a multiple of 16 bytes */
  SS_ERR_STATE = 4,       /* call order violated */
  SS_ERR_CAPACITY = 5,    /* workspace too small */
  SS_ERR_UNSUPPORTED = 6, /* device is not sm_100 */
  SS_ERR_CUDA = 7,        /* a CUDA runtime/driver call failed; see ss_last_cuda_error */
  SS_ERR_DEVICE_FLAG = 8, /* the device status word is non-zero (see SS_DEV_*) */
  SS_ERR_TIMEOUT = 9      /* a host wait ran past its deadline */
} ss_status;

/* bits of the device status word */
#define SS_DEV_BAD_VALID_LEN 1u /* valid_len[b] outside [0, L_c]: clamped             */
#define SS_DEV_BAD_ACCEPT 2u    /* accept_cnt/accept_idx out of range: row skipped     */
#define SS_DEV_DST_OVERFLOW 4u  /* dst_off + k outside [0, cap): row skipped           */
#define SS_DEV_WAIT_EXPIRED 8u  /* a bounded in-kernel wait gave up: round is invalid  */
#define SS_DEV_BAD_PAGE 16u     /* page id outside the pool: its tokens read as zeros  */

typedef struct {
  int32_t max_B;      /* requests per call                                          */
  int32_t H_q, H_kv;  /* query heads, kv heads (H_q % H_kv == 0)                     */
  int32_t d;          /* head dim, 64 or 128 (both on the tensor-core kernels)       */
  int32_t max_Tq;     /* candidate queries per request                               */
  int32_t max_Tloc;   /* local candidate KV tokens per request (<= 1024)             */
  int32_t max_Lc;     /* tokens per history chunk call                               */
  int32_t max_chunks; /* chunk calls held as separate partial sets before the library
                         folds them (any number of calls stays legal); 0 = default 64;
                         1 is taken as 2 (a fold needs a free set to go on with)      */
  int32_t device;     /* CUDA device ordinal                                         */
  uint32_t flags;     /* SS_FLAG_*                                                   */
} ss_config;

/* Force the CUDA-core chunk kernel even where the tensor-core kernel applies. */
#define SS_FLAG_FORCE_SIMT 1u
/* Let successive chunk kernels of a round overlap on the GPU (programmatic dependent
 * launch).  The caller promises that Q and the K/V of a chunk call are complete in
 * memory before the PREVIOUS ss_ call of the round was enqueued on the stream, or were
 * produced by a copy / an event the stream waited on - not by a kernel enqueued on the
 * same stream between two ss_ calls.  With the flag a round's FIRST chunk kernel (and the
 * single launch of a small ss_verify_round) is also launched that way, but waits for the
 * completion of whatever precedes it on the stream before it reads or writes anything:
 * only its launch and set-up overlap the previous round's finalize, and the promise above
 * is not needed for it. */
#define SS_FLAG_OVERLAP_CHUNKS 2u
/* Use the tensor-core chunk kernel that puts the query rows on the MMA's M axis instead of
 * the default one that puts the keys there.  For cross-checks. */
#define SS_FLAG_ROWS_ON_M 4u
/* Use the keys-on-M kernel for any number of rows per kv-head (default: up to 32). */
#define SS_FLAG_KEYS_ON_M 8u
/* ss_stream_round also times its phases with device events (read with ss_get_stats):
 * an event pair around every chunk call and one around the local / finalize / commit tail. */
#define SS_FLAG_STREAM_TIMING 16u
/* Tuning overrides read from the environment by ss_create (for experiments; unset = automatic):
 *   SS_CHUNK_KERNEL=rows|keys  as SS_FLAG_ROWS_ON_M / SS_FLAG_KEYS_ON_M
 *   SS_SPLITS=n                token splits of every chunk call (default: sized so that a
 *                              call launches about one CTA per SM)
 *   SS_TARGET_CTAS=n           the CTA count the automatic split choice aims at
 *   SS_ROUND_CLUSTER=never     the single-launch small round merges its token splits through
 *                              scratch memory and a ticket instead of a thread-block cluster
 * and, read at every ss_verify_chunks call:
 *   SS_HISTORY_LAUNCH=never|always  never / wherever possible take a list of chunks in one launch
 *   SS_HISTORY_WALK=never|always    ragged batches never take / batches of any known lengths take
 *                                   the one launch with shares across requests */

typedef struct {
  const void* ptr;                      /* device pointer, bf16                      */
  int64_t stride_b, stride_h, stride_t; /* elements; innermost dim contiguous        */
} ss_tensor;

typedef enum { SS_MASK_CHAIN = 0, SS_MASK_TREE_BITS = 1 } ss_mask_kind;

/* Bytes of device workspace a context with this config needs (0 on invalid config). */
size_t ss_workspace_bytes(const ss_config* cfg);

/* Create a context over a caller-allocated device workspace (256-byte aligned, at least
 * ss_workspace_bytes).  Synchronous; clears the device status word on `stream` 0. */
ss_status ss_create(ss_ctx** out, const ss_config* cfg, void* workspace, size_t workspace_bytes);
ss_status ss_destroy(ss_ctx* ctx);

/* a1. Start a round: bind Q [B, H_q, T_q, d] and reset every row's state to the
 * identity (m, l, a) = (-inf, 0, 0) (Section 4.2, accumulator initialisation).
 * `scale` multiplies the scores (1/sqrt(d) in the paper), is applied in fp32 and must be
 * positive and finite (SS_ERR_ARG otherwise). */
ss_status ss_verify_begin(ss_ctx* ctx, ss_tensor Q, int32_t B, int32_t T_q, float scale,
                          void* stream);

/* a2+a3. One history chunk for the whole batch: K, V [B, H_kv, L_c, d]; valid_len
 * (device, [B], may be NULL = all L_c) gives the number of leading valid tokens of each
 * request's chunk; tokens past it are invisible and may hold anything, NaN included.
 * Computes the chunk-local state of Eq. 13 for every query row (all T_q*H_q/H_kv rows of
 * a kv-head share one pass over its K/V) and records it for the Eq. 14 merge.  History
 * is visible to every query of the round.  An on-GPU Active Tail is passed the same way. */
ss_status ss_verify_chunk(ss_ctx* ctx, ss_tensor K, ss_tensor V, int32_t L_c,
                          const int32_t* valid_len, void* stream);

/* Same as ss_verify_chunk, with a HOST copy of valid_len ([B], may be NULL) as a scheduling
 * hint: the token splits are sized for the requests that are still active, which keeps the GPU
 * full when most of a ragged batch has run out of history, and (batches of up to 256 requests)
 * requests whose hinted length is 0 get no thread blocks at all in this call.  The device
 * array stays authoritative for the lengths that are used; a wrong hint can cost speed or, if
 * it understates a length, drop tokens (those past the hinted maximum of the batch; all of a
 * request hinted as 0) - pass the same values. */
ss_status ss_verify_chunk_hinted(ss_ctx* ctx, ss_tensor K, ss_tensor V, int32_t L_c,
                                 const int32_t* valid_len, const int32_t* valid_len_host,
                                 void* stream);

/* A chunk whose tokens live in pages of a pool (requests keep independent KV indices): K_pool,
 * V_pool are [n_pages, H_kv, page_size, d] (ss_tensor: stride_b = page stride; any strides
 * that are multiples of 8 elements, so a pool stored [n_pages, page_size, H_kv, d] is passed
 * with stride_t = H_kv * d and stride_h = d); the chunk of
 * request b is the concatenation of pages page_table[b][0 .. pages_per_req) (device int32
 * [B, pages_per_req]), i.e. L_c = pages_per_req * page_size tokens of which valid_len[b] are
 * valid (NULL = all).  Same result as ss_verify_chunk on the gathered chunk.  The tensor-core
 * kernels take pages of 8, 16, 32, 64 tokens (gathered page by page into their tiles) and any
 * multiple of 64 (rows on M) or 128 (keys on M); other page sizes take the CUDA-core kernel,
 * which is an order of magnitude slower.  Only the pages that hold valid tokens are looked up:
 * table entries past ceil(valid_len[b] / page_size) may hold anything.  valid_len_host (HOST,
 * may be NULL) is the scheduling hint of ss_verify_chunk_hinted.  A looked-up page id outside
 * [0, n_pages) raises SS_DEV_BAD_PAGE and its tokens read as zeros. */
ss_status ss_verify_chunk_paged(ss_ctx* ctx, ss_tensor K_pool, ss_tensor V_pool, int32_t n_pages,
                                int32_t page_size, const int32_t* page_table, int32_t pages_per_req,
                                const int32_t* valid_len, const int32_t* valid_len_host, void* stream);

/* a2, several chunks with one call (Section 4.2: the chunks of a request are reduced into one
 * running state; Eq. 13-14).  chunks is a HOST array of n_chunks (>= 0) descriptors, read before
 * the call returns; the result is that of one ss_verify_chunk_hinted per descriptor, in order.
 * Where one tensor-core kernel would take every chunk and one CTA per (request, kv-head, row
 * tile) fits the GPU at once, the whole list takes ONE launch: a CTA walks an equal share of its
 * request's tiles across the chunk boundaries with one accumulator, so the list leaves a few
 * partial states per row instead of one per chunk, and set-up and write-out are paid once per
 * request instead of once per chunk.  This is done (2 to 32 contiguous chunks) when the host
 * knows the requests' histories to be equally long - no valid_len at all, or valid_len_host for
 * every chunk with totals within 10 % of each other - for up to 32 rows per kv-head (16 at head
 * dim 64; keys-on-M kernel, chunks of at least 128 tokens: "tcgen05-keys-round" in
 * ss_last_chunk_kernel) and for more rows up to 128 (rows-on-M kernel: "tcgen05-round"); and at
 * head dim 128 for more than 128 rows per kv-head unless the host knows the batch to be ragged
 * ("tcgen05-round").  A batch the host knows to be ragged (valid_len_host for every chunk with
 * lengths, no request empty) also takes one launch with up to 32 rows per kv-head (16 at head dim
 * 64): the tiles of a kv-head's requests are laid end to end and every CTA takes an equal share,
 * ending one request and beginning the next where its share says so; the shares are cut on the
 * host's lengths and scaled to those on the device, so in this launch lengths that are out of
 * date cost balance, not tokens (pass the device's values all the same: the separate calls drop
 * tokens that the hint leaves out) ("tcgen05-keys-round"; SS_HISTORY_WALK=never turns this off).
 * SS_HISTORY_LAUNCH=never|always in the environment overrides the routing.  Otherwise the
 * chunks are enqueued one by one.  The results agree with separate calls
 * up to the order of the fp32 sums (one launch merges per split, separate calls per chunk).
 * Stream capture: the one launch reads the chunks' tensor maps from one of four lists in the
 * workspace, sent when a list of buffers is first used.  Under a capture a list that is already
 * there is kept for the life of the context (a graph may replay the launch), and a list that is
 * not is not sent: those chunks are enqueued one by one.  So run a round once before capturing it.
 * SS_ERR_STATE outside an open round; an error leaves the round open (ss_verify_abort ends it). */
typedef struct {
  ss_tensor K, V;                 /* [B, H_kv, L_c, d] bf16, device                          */
  int32_t L_c;
  const int32_t* valid_len;       /* device [B], 0..L_c; NULL = all L_c                      */
  const int32_t* valid_len_host;  /* HOST copy of valid_len or NULL (scheduling hint)        */
} ss_chunk_desc;
ss_status ss_verify_chunks(ss_ctx* ctx, const ss_chunk_desc* chunks, int32_t n_chunks, void* stream);

/* a4. The on-GPU candidate segment (Section 4.2: the pass over the GPU-resident Active Tail and
 * Speculative Frontier; the mask M of Eq. 12): K_loc, V_loc [B, H_kv, T_loc, d].  Query i of
 * request b sees local token j iff
 *   SS_MASK_CHAIN:     j <= i + (T_loc - T_q)   (causal, inclusive; mask_bits ignored;
 *                      T_loc >= T_q, SS_ERR_ARG otherwise: the T_loc - T_q leading local
 *                      tokens - an Active Tail passed with the candidates - are seen by all)
 *   SS_MASK_TREE_BITS: bit j of mask_bits[b][i][j/64] is set (device uint64
 *                      [B, T_q, ceil(T_loc/64)]; row i = ancestors of node i and i itself). */
ss_status ss_verify_local(ss_ctx* ctx, ss_tensor K_loc, ss_tensor V_loc, int32_t T_loc,
                          ss_mask_kind kind, const uint64_t* mask_bits, void* stream);

/* A whole round with ONE host call (the paper has no counterpart for the call itself; it
 * computes Eq. 12 like begin + chunk* + local + finalize).  chunks is a HOST array of n_chunks
 * (>= 0) descriptors, read before the call returns; T_loc = 0 skips the local segment.  Same
 * tensors, checks and results as the separate calls: a large round is begin + ss_verify_chunks
 * + local + finalize.  A small round (at most 16 chunks and 32 tiles of 64 tokens in all, T_loc <=
 * 64) takes a single launch of the CUDA-core kernel that walks the chunks and the local
 * segment and finalizes in place (the token splits of a row tile run as one thread-block
 * cluster and merge their states through distributed shared memory), so that no partial state
 * goes through HBM and a tiny round costs one launch instead of n_chunks + 2.  SS_ERR_STATE while a round is open; on any
 * error nothing of the round is merged and the context is idle again. */
ss_status ss_verify_round(ss_ctx* ctx, ss_tensor Q, int32_t B, int32_t T_q, float scale,
                          const ss_chunk_desc* chunks, int32_t n_chunks, ss_tensor K_loc,
                          ss_tensor V_loc, int32_t T_loc, ss_mask_kind kind, const uint64_t* mask_bits,
                          void* O, float* LSE, void* stream);

/* Measurement aid (the paper has no counterpart): n_rounds rounds enqueued back to back by a
 * C caller - this function - and timed with two events on `stream`; *ms_total (HOST) receives
 * the device time of all of them.  single_call != 0: one ss_verify_round per round; 0: the
 * separate calls.  chunks holds n_sets consecutive groups of n_chunks descriptors and round i
 * uses group i % n_sets (rotating history buffers keep a small round from living in L2).
 * Synchronous.  It shows what a round costs without a binding's per-call overhead. */
ss_status ss_time_rounds(ss_ctx* ctx, ss_tensor Q, int32_t B, int32_t T_q, float scale,
                         const ss_chunk_desc* chunks, int32_t n_chunks, int32_t n_sets, ss_tensor K_loc,
                         ss_tensor V_loc, int32_t T_loc, ss_mask_kind kind, const uint64_t* mask_bits,
                         void* O, float* LSE, void* stream, int32_t n_rounds, int32_t single_call,
                         float* ms_total);

/* Checkpoint of a round (between begin and finalize).  export writes, for every query row in
 * [B, H_q, T_q] order, the merged state of everything seen so far: ml[row] = (m, l) with m in
 * the base-2 domain (maximum reference of score*scale*log2(e); -inf and l = 0 for an empty
 * row) and a[row][d] = sum exp2(s2 - m) v, both fp32 device buffers.  The round stays open.
 * import adds such a state to the open round as one more partial (Eq. 14 is associative and
 * order-free), e.g. the states other GPUs reduced over their share of the history chunks. */
ss_status ss_verify_export_state(ss_ctx* ctx, float* ml, float* a, void* stream);
ss_status ss_verify_import_state(ss_ctx* ctx, const float* ml, const float* a, void* stream);

/* a5. Merge all partial states (Eq. 14), O = a / l as bf16 (round to nearest even) into
 * O [B, H_q, T_q, d] (contiguous), LSE = m + ln l (natural log, of the scaled masked
 * scores) into LSE [B, H_q, T_q] fp32 (may be NULL).  Ends the round. */
ss_status ss_verify_finalize(ss_ctx* ctx, void* O, float* LSE, void* stream);

/* Drops the open round without producing an output (for a caller whose chunk or local call
 * failed, or that no longer wants the result).  Host-side only: kernels already enqueued run to
 * completion and their partial states are never merged; the next ss_verify_begin starts from the
 * identity state again.  With no round open it does nothing.  Returns SS_ERR_ARG for a NULL ctx. */
ss_status ss_verify_abort(ss_ctx* ctx);

/* a6. Commit-gather (Section 4.1: accepted candidates join the committed prefix).  For each
 * request b and k < accept_cnt[b]: row accept_idx[b][k] of K_loc/V_loc (all kv heads) is
 * copied, bit for bit, to row dst_off[b] + k of K_dst/V_dst [B, H_kv, cap, d].  Nothing else
 * is written.  accept_idx is [B, T_loc] int32, accept_cnt and dst_off are [B] int32, all on
 * the device.  Independent of the round state; may be called at any time. */
ss_status ss_commit_gather(ss_ctx* ctx, ss_tensor K_loc, ss_tensor V_loc, int32_t B,
                           int32_t T_loc, const int32_t* accept_idx, const int32_t* accept_cnt,
                           ss_tensor K_dst, ss_tensor V_dst, int32_t cap, const int32_t* dst_off,
                           void* stream);

/* Read (and clear) the device status word after synchronising `stream`, waiting at most
 * timeout_ms (<= 0: wait without limit).  SS_OK, SS_ERR_DEVICE_FLAG (bits in *dev_bits if
 * non-NULL) or SS_ERR_TIMEOUT. */
ss_status ss_poll_status(ss_ctx* ctx, void* stream, int32_t timeout_ms, uint32_t* dev_bits);

/* a7. Streamed round (Section 4.2, pipelined KV transfers): the committed history lives in
 * pinned HOST memory and crosses the host link once per round through two device staging
 * buffers; copies run on a copy stream while the attention stream works on the other buffer.
 *
 * Host layout of request b: for chunk j = 0..ceil(hist_len[b]/L_c)-1 a block of
 * [2 (K,V)][H_kv][L_c][d] bf16 at hist[b] + j * 2*H_kv*L_c*d elements (last block partial:
 * only the first valid tokens of each head row are read).
 * Device staging: stage_k[s], stage_v[s], s = 0,1, each [B, H_kv, batch_chunks*L_c, d]
 * contiguous; one fill carries batch_chunks adjacent chunks (a transfer batch) and is
 * consumed by one chunk-attention call.  Requests sorted by decreasing length keep the
 * active requests of late fills a prefix of the batch, but any order is correct.
 * After the attention the accepted rows are gathered into commit_k/commit_v
 * [B, H_kv, T_q, d] (device) at row 0 and the buffers copied to host_commit_k/v (pinned
 * HOST, same shape).  O_host / LSE_host (pinned HOST, may be NULL) receive the outputs.
 * Synchronous: returns when the round is complete. */
typedef struct {
  int32_t B, T_q, L_c;
  float scale;
  const void* const* hist;   /* HOST array [B] of pinned HOST pointers                    */
  const int32_t* hist_len;   /* HOST [B]                                                  */
  int32_t batch_chunks;      /* adjacent chunk indices per staging-buffer fill (>= 1)     */
  void* stage_k[2];          /* device, each [B, H_kv, batch_chunks * L_c, d]             */
  void* stage_v[2];
  int32_t scratch_fills;     /* capacity of the two scratch arrays, in fills              */
  int32_t* valid_len_host;   /* pinned HOST scratch [scratch_fills * B]                   */
  int32_t* valid_len_dev;    /* device scratch      [scratch_fills * B]                   */
  ss_tensor Q, K_loc, V_loc; /* device; T_loc = T_q                                       */
  ss_mask_kind mask_kind;
  const uint64_t* mask_bits; /* device                                                    */
  void* O;                   /* device [B,H_q,T_q,d] bf16                                 */
  float* LSE;                /* device [B,H_q,T_q]                                        */
  const int32_t* accept_idx; /* device [B,T_q]; NULL skips the commit step                */
  const int32_t* accept_cnt; /* device [B]                                                */
  const int32_t* zero_off;   /* device [B] of zeros (destination offsets)                 */
  void* commit_k;            /* device [B,H_kv,T_q,d]                                     */
  void* commit_v;
  void* host_commit_k;       /* pinned HOST, same shape; receives the whole buffer        */
  void* host_commit_v;
  void* O_host;              /* pinned HOST or NULL                                       */
  float* LSE_host;           /* pinned HOST or NULL                                       */
  int32_t copy_only;         /* 1: issue the same copies but no attention (control run)   */
  /* optional on-GPU Active Tail (committed KV not yet offloaded): attended to as one more chunk */
  ss_tensor tail_K, tail_V;  /* device [B, H_kv, tail_Lc, d]; tail_K.ptr NULL = none           */
  int32_t tail_Lc;
  const int32_t* tail_len;   /* device [B] valid tokens of the tail                           */
  int32_t commit_cap;        /* token capacity of commit_k / commit_v rows (0 = T_q); with a
                                tail, commit_k/v may be the tail buffers and zero_off their
                                lengths, so accepted rows are appended to the tail in place   */
  int32_t stage_fused;       /* 1: stage_k[s] is ONE buffer [B][2 (K,V)][H_kv][batch_chunks*L_c][d]
                                (stage_v ignored), the host block's own order, so every
                                (request, chunk) block crosses the link in one copy instead of
                                two: copies twice as large reach a few % more of the link.
                                2: stage_k[s] is [B][batch_chunks][2 (K,V)][H_kv][L_c][d], the
                                host's block sequence itself: a fill moves the batch_chunks
                                adjacent blocks of a request with ONE copy (plus one for a
                                partial block) and is consumed by batch_chunks chunk calls of
                                L_c tokens; scratch_fills then counts chunk calls, not fills  */
} ss_stream_desc;

typedef struct {
  double ms_total;      /* host wall time of the round                                    */
  float ms_device;      /* first copy enqueued -> last D2H done, CUDA events              */
  int64_t h2d_bytes;    /* valid K/V bytes moved host -> device                           */
  int64_t d2h_bytes;
  int32_t chunk_calls;
  int32_t copies;
} ss_stream_stats;

/* SS_ERR_STATE, touching nothing, while the caller has a round open on this context. */
ss_status ss_stream_round(ss_ctx* ctx, const ss_stream_desc* desc, ss_stream_stats* stats);

/* Several layers back to back through the same two staging buffers (Section 4.2, pipelined KV
 * transfers and prefetching; the modes mirror the paper's ablation of streaming designs):
 *   SS_LAYERS_PREFETCH  stream-and-reduce with cross-layer prefetch: the copy stream starts the
 *                       next layer's first fills as soon as a staging buffer frees, while the
 *                       current layer's last attention, finalize and commit still run;
 *   SS_LAYERS_STREAM    stream-and-reduce, layer by layer: a layer's copies start only when the
 *                       previous layer's work is done;
 *   SS_LAYERS_RESTORE   restore-then-verify baseline: the whole history of a layer is copied into
 *                       restore_k / restore_v (device, [B, H_kv, restore_tokens, d]) and only then
 *                       attended to; layers run strictly one after the other.  With restore_v
 *                       NULL, restore_k is one buffer [B][2 (K,V)][H_kv][restore_tokens][d]
 *                       and every (request, chunk) block is restored with one copy.
 * Every layer has its own descriptor (history, Q, local KV, outputs); all layers use the same
 * B, T_q, L_c, batch_chunks and staging buffers.  Layers may share the valid_len scratch arrays
 * only if their history lengths are identical.  Synchronous; `total` covers all layers. */
typedef enum { SS_LAYERS_PREFETCH = 0, SS_LAYERS_STREAM = 1, SS_LAYERS_RESTORE = 2 } ss_layers_mode;
typedef struct {
  int32_t n_layers;            /* <= 256                                                   */
  const ss_stream_desc* layers; /* HOST array [n_layers]                                   */
  int32_t mode;                /* ss_layers_mode                                           */
  void* restore_k;             /* device; SS_LAYERS_RESTORE only                           */
  void* restore_v;             /* NULL: restore_k holds K and V (see above)                */
  int64_t restore_tokens;      /* token capacity of a restore buffer row                   */
} ss_layers_desc;
ss_status ss_stream_layers(ss_ctx* ctx, const ss_layers_desc* layers, ss_stream_stats* total);
/* Commit-aware KV tiering (Section 4.1).  Per request: Sealed History [0, H) in pinned host
 * memory (chunk-block layout of ss_stream_round), Active Tail [H, C) in a device buffer
 * [B, H_kv, tail_capacity, d] (token t at index t - H).  ss_tier_commit advances C by the rows a
 * commit-gather appended; ss_tier_migrate computes the Eq. 9 end point
 * E = max{H, g * floor(max(0, C - T) / g)} per request and starts the asynchronous copy of
 * [H, E) to the host; ss_tier_poll advances H to E only once that copy is confirmed and then
 * moves the surviving tails to the front of the other tail buffer (all requests swap together).
 * Rejected candidates live past C and never reach the host, so there is no host-side rollback.
 * Host logic only; every copy is enqueued on the given stream.  len_dev (device [B]) always holds
 * C - H: the valid length of the tail chunk and the offset the next commit-gather appends at.
 * len_host is pinned HOST scratch of 4 * B int32. */
typedef struct ss_tier ss_tier;
typedef struct {
  int32_t B, H_kv, d, L_c;
  int32_t tail_target;   /* T: committed tokens kept on the GPU                                */
  int32_t granularity;   /* g: offload batch, H stays a multiple of it                         */
  int32_t tail_capacity; /* tokens per tail buffer row, >= T + g (+ a round of accepted rows)  */
} ss_tier_config;
ss_status ss_tier_create(ss_tier** out, const ss_tier_config* cfg, void* const* host_hist,
                         const int64_t* host_capacity_tokens, void* tail_k0, void* tail_v0,
                         void* tail_k1, void* tail_v1, int32_t* len_dev, int32_t* len_host);
ss_status ss_tier_destroy(ss_tier* tier);
/* Set the boundaries (HOST [B] each; H multiple of g, tail data already at index t - H of buffer 0). */
ss_status ss_tier_reset(ss_tier* tier, const int32_t* H, const int32_t* C, void* stream);
/* Read the boundaries (any pointer may be NULL); pending_E = end point of the copy in flight. */
ss_status ss_tier_get(ss_tier* tier, int32_t* H, int32_t* C, int32_t* pending_E, int32_t* cur_buffer);
/* Current tail view and the device array of tail lengths. */
ss_status ss_tier_tail(ss_tier* tier, ss_tensor* K, ss_tensor* V, const int32_t** tail_len_dev);
ss_status ss_tier_commit(ss_tier* tier, const int32_t* cnt_host, void* stream);
ss_status ss_tier_migrate(ss_tier* tier, void* stream, int32_t* n_requests);
ss_status ss_tier_poll(ss_tier* tier, int32_t wait, void* stream, int32_t* advanced);
int64_t ss_tier_d2h_bytes(ss_tier* tier);

/* I/O-aware dynamic verification width (Section 4.2): q* = argmin_q T_round(q) / U(q) over the
 * candidate widths, from running means of the rounds observed at each width.  Host logic only.
 * T_round = t_draft + max(t_transfer, t_compute) + t_other (overlapped transfer and compute are
 * counted once); means are exponential moving averages with weight `ema` (the first observation
 * is taken as is); every width is tried `sample_rounds` times, in list order, before any estimate
 * is trusted; afterwards the width changes only if the best width's cost per committed token is
 * below the current one's by more than `switch_threshold` (relative).  Times are floats in any
 * one unit; `committed` is the number of tokens the round committed. */
typedef struct ss_width ss_width;
typedef struct {
  int32_t n_widths;       /* 1..8                                                         */
  int32_t widths[8];      /* candidate set, e.g. {2, 4, 6, 8}                             */
  int32_t sample_rounds;  /* >= 1                                                         */
  float switch_threshold; /* >= 0, e.g. 0.05                                              */
  float ema;              /* in (0, 1]                                                    */
} ss_width_config;
typedef struct {
  float t_draft, t_transfer, t_compute, t_other;
  int32_t committed;
} ss_width_obs;
ss_status ss_width_create(ss_width** out, const ss_width_config* cfg);
ss_status ss_width_destroy(ss_width* w);
ss_status ss_width_observe(ss_width* w, int32_t q, const ss_width_obs* obs); /* end of a round at width q */
int32_t ss_width_next(ss_width* w);                                          /* width of the next round  */
ss_status ss_width_estimate(ss_width* w, int32_t q, double* t_round, double* committed, double* cost,
                            int32_t* n_obs);

/* Cohort builder (Section 4.2, cohort batching).  Tasks that one batched kernel can process
 * (same layer, width, dtype, n_kv, d_h, chunk_size) are grouped; inside a cohort requests are
 * ordered by decreasing history length (stable), cohorts keep the order of their first task and
 * are cut into pieces of at most max_batch.  order [n] receives the task indices cohort by
 * cohort, cohort_start [n + 1] the start of each cohort in `order` (and the total at the end).
 * Returns the number of cohorts, -1 on invalid arguments.  HOST pointers. */
typedef struct {
  int32_t layer, width, dtype, n_kv, d_h, chunk_size;
  int32_t request_id, hist_len;
} ss_task;
int32_t ss_cohort_build(const ss_task* tasks, int32_t n, int32_t max_batch, int32_t* order,
                        int32_t* cohort_start);


/* A whole round (one history chunk + local segment -> O, LSE) that allocates nothing and
 * needs no context or workspace.  The paper has no counterpart: this exists for callers that
 * cannot call cudaMalloc where they need attention (code in a region that must not
 * synchronise the device, plug-ins that do not own the process's memory pool, start-up paths
 * that run before the host framework's allocator exists).  The per-row partial states live in
 * a fixed SS_STATIC_SCRATCH_BYTES array inside the library's device image; each GPU that
 * loads the library holds it until the process exits.
 *  - Same tensors, layouts, masks and results as begin/chunk/local/finalize with one chunk
 *    call (K/V [B,H_kv,L_c,d], L_c may be 0 to skip the history; T_loc may be 0 to skip the
 *    local segment, not both).  The CUDA-core chunk kernel is used.
 *  - Returns SS_ERR_CAPACITY, enqueuing nothing, when the round's partial states
 *    (2 * splits * B * H_kv * T_q * G rows of (d + 2) floats, splits <= 16) do not fit.
 *  - The first call on a device looks up the array's device address (with that device
 *    current; host threads may race to it); make that first call before any stream capture.
 *    Any call does, even one that is rejected for its arguments: ss_verify_round_static(NULL,
 *    NULL) is a valid warm-up (it returns SS_ERR_ARG).  No call allocates or frees.
 *  - Shapes are limited like the regular entry points' (T_q * H_q / H_kv <= 4096,
 *    B * H_q * T_q < 2^31: SS_ERR_SHAPE); mask_kind must be one of the two kinds and a chain
 *    mask needs T_loc >= T_q (SS_ERR_ARG).
 *  - All calls share the array: it keeps the last call's contents (the call clears what must
 *    start at zero), and calls whose kernels may overlap on the GPU race - serialise them.
 *  - `status` (optional DEVICE word, OR-ed with SS_DEV_* bits) receives device-detected
 *    problems; with NULL they are only clamped. */
#define SS_STATIC_SCRATCH_BYTES (4u << 20)
typedef struct {
  int32_t B, H_q, H_kv, d, T_q, T_loc, L_c;
  float scale;
  ss_tensor Q;              /* [B, H_q, T_q, d]                                          */
  ss_tensor K, V;           /* [B, H_kv, L_c, d]; ignored when L_c == 0                  */
  const int32_t* valid_len; /* device [B] or NULL                                        */
  ss_tensor K_loc, V_loc;   /* [B, H_kv, T_loc, d]; ignored when T_loc == 0              */
  ss_mask_kind mask_kind;
  const uint64_t* mask_bits;
  void* O;                  /* device [B, H_q, T_q, d] bf16                              */
  float* LSE;               /* device [B, H_q, T_q] or NULL                              */
  uint32_t* status;         /* device word or NULL                                       */
} ss_static_round;
ss_status ss_verify_round_static(const ss_static_round* round, void* stream);

const char* ss_strerror(ss_status s);
/* sizeof(ss_stream_desc) as compiled, for bindings that mirror the struct. */
size_t ss_sizeof_stream_desc(void);
/* Last CUDA error code seen by this context (cudaError_t as int), 0 if none. */
int32_t ss_last_cuda_error(ss_ctx* ctx);
/* Tracing.  While enabled, CTA (0,0,0) of every tensor-core chunk kernel stamps the SM clock
 * at fixed points of its tile loop into a region of the workspace: words
 * [role][tile < 32][event < 8], role 0 = TMA producer, 1 = MMA issuer, 2 = softmax lane 0;
 * event 0 is the role's first stamp for that tile (the softmax thread reaching the tile, the
 * MMA issuer finding the tile's K landed), the other events are the kernel's own wait / issue
 * points (see the kernel sources).  Enabling clears the region (synchronous).
 * ss_trace_read synchronises nothing: call it after the stream is idle; it copies up to
 * max_words 64-bit words to HOST memory and returns the count. */
ss_status ss_trace_enable(ss_ctx* ctx, int32_t on);
int32_t ss_trace_read(ss_ctx* ctx, uint64_t* out, int32_t max_words);
/* Per-CTA log of the tensor-core chunk kernels (a measurement aid; the paper has no
 * counterpart).  `log` is a DEVICE buffer of 4 * (capacity + 1) 64-bit words that the caller
 * owns and zeroes: word 0 counts the entries, entry i occupies words 4 (i + 1) .. 4 (i + 1) + 3:
 * the CTA's start and end on the GPU's nanosecond timer, (SM id << 32 | the context's launch
 * number), (linear block id << 32 | tiles processed).  Entries past `capacity` are counted but
 * not stored.  log = NULL switches it off.  Takes effect from the next chunk call. */
ss_status ss_cta_log_set(ss_ctx* ctx, uint64_t* log, int32_t capacity);
/* Self-test of the bounded waits (the paper has no counterpart): one small kernel whose 64
 * threads wait, with the chunk kernels' own wait routine and a limit of limit_ms (1..1000), on
 * a barrier that nothing will ever complete.  Every thread must give up: *gave_up (DEVICE
 * uint32, zeroed by the caller) counts them, SS_DEV_WAIT_EXPIRED is raised in the context's
 * status word (read and cleared with ss_poll_status) and the context stays usable. */
ss_status ss_selftest_wait_expiry(ss_ctx* ctx, int32_t limit_ms, uint32_t* gave_up, void* stream);
/* Measurement aid (the paper has no counterpart): read n segments of DEVICE memory once, in
 * one kernel, with streaming 16-byte loads from every SM, and XOR-fold them into the 64-bit
 * DEVICE word *sink (the caller zeroes it or ignores it; it exists so that the loads cannot be
 * dropped).  srcs and bytes are HOST arrays of n <= 64 entries (SS_ERR_CAPACITY above), read
 * before the call returns; every segment 16-byte aligned with a length that is a multiple of
 * 16, sink 8-byte aligned (SS_ERR_ALIGN otherwise).  Timed by the caller with events on
 * `stream`, it gives the read bandwidth a kernel that streams memory once can reach on this
 * GPU in its current clock state. */
ss_status ss_probe_read(const void* const* srcs, const size_t* bytes, int32_t n, uint64_t* sink,
                        void* stream);
/* Counters of a context (the paper has no counterpart; its width controller, Section 4.2,
 * consumes the transfer and compute times of a round, which the last_* fields provide).
 * The last_* fields describe the most recent ss_stream_round of a context created with
 * SS_FLAG_STREAM_TIMING and are 0 otherwise; they are device-event times in nanoseconds. */
typedef struct {
  int64_t launches;      /* kernels launched since creation                                      */
  int64_t rounds;        /* rounds finalized                                                     */
  int64_t rows;          /* query rows finalized (B * H_q * T_q summed over the rounds)          */
  int64_t chunk_calls;   /* chunk calls of any kind                                              */
  int64_t kv_bytes;      /* K/V bytes those calls covered: the valid tokens where the call had a
                            host copy of the lengths (or no lengths at all), else every token
                            of the chunk (an upper bound)                                        */
  int64_t last_round_ns;     /* first copy enqueued -> last device-to-host copy done             */
  int64_t last_transfer_ns;  /* copy stream: first history copy -> last history copy done        */
  int64_t last_chunk_ns;     /* attention stream: sum over the chunk calls of their kernel time  */
  int64_t last_tail_ns;      /* local segment + finalize + commit-gather + copies to the host    */
  int64_t last_wait_ns;      /* last_round_ns - last_chunk_ns - last_tail_ns: the attention
                                stream waiting for transfers (the paper's exposed transfer time)  */
} ss_stats;
ss_status ss_get_stats(ss_ctx* ctx, ss_stats* out);
/* Number of kernels this context has launched since creation. */
int64_t ss_launch_count(ss_ctx* ctx);
/* "simt", "tcgen05" (rows on M), "tcgen05-keys" (keys on M), "tcgen05-round" / "tcgen05-keys-round"
 * (the same two over a list of chunks in one launch) or "simt-round" (a small round in one
 * launch): the chunk kernel the last chunk call, ss_verify_chunks or ss_verify_round used;
 * "none" before. */
const char* ss_last_chunk_kernel(ss_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* SPECSTREAM_H_ */
