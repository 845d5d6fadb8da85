/*
 * mukv.h -- C ABI of the MuKV compression + retrieval library for NVIDIA B200 (sm_100a).
 *
 * The library implements the data-parallel path of MuKV ("Multi-Grained KV Cache
 * Compression for Long Streaming Video Question-Answering"):
 *
 *   mukv_compress_chunk   Sec. 3.3 (Eq. 1-4, top-kappa selection, storing the kept KV
 *                         slices of all layers with their timestamps) and Eq. 5 of
 *                         Sec. 3.4 (mean-pooled block representations), applied to one
 *                         streaming chunk of frames after the LLM prefill.
 *   mukv_retrieve         Sec. 3.4 (Eq. 6-8): question pooling, cosine scoring against the
 *                         segment-level and frame-level block keys, top-2k candidates,
 *                         global-query rerank, final top-k.
 *   mukv_gather           Sec. 3.5 (Eq. 9): builds R_k, R_v, the contiguous decode context,
 *                         from the selected blocks.
 *
 * Conventions
 *   - Pointers named d_* are DEVICE pointers, h_* are HOST pointers.  Tensors of the cache
 *     dtype (Q, K, V, question tokens, decode buffers), the store and the workspace must be
 *     16-byte aligned; int32 / float index and score arrays need their natural 4-byte alignment.
 *   - Ownership: the caller owns every device buffer (store, workspace, inputs, outputs).
 *     The library allocates no device memory; a context holds host metadata only.
 *   - Ordering: all device work is enqueued on the stream given to the call and the call
 *     returns after enqueueing.  Host-visible counters (frames stored) advance at enqueue
 *     time; outputs are valid once the stream has reached that point.
 *   - Errors: every entry point returns a mukv_status.  Argument errors are detected on the
 *     host before anything is enqueued and leave the store unchanged.  No C++ exception
 *     crosses this boundary.  mukv_last_error() gives a readable message.
 *   - Threading: one context is used by one host thread at a time, and the calls on one context
 *     must also be ordered on the device (the same stream, or streams joined by events): every
 *     call, mukv_retrieve included, keeps intermediate results in the context's workspace.
 *     mukv_retrieve and mukv_gather do not modify the store.
 *   - A launch failure in the middle of mukv_compress_chunk (MUKV_E_CUDA after part of the call
 *     was enqueued) leaves the chunk half stored: the context then answers MUKV_E_STATE to every
 *     call except mukv_reset, mukv_get_stats and mukv_destroy.
 *
 * Tensor layouts are token-major; element type is mukv_config.dtype (bf16 or fp32):
 *     Q   [n_frames][P][Hq][D]        queries of the chunk's visual tokens in the scoring layer (the
 *                                     last layer by default); [Ls][n_frames][P][Hq][D] when
 *                                     n_score_layers = Ls > 1, ordered like the layers of K
 *     K,V [L][n_frames][P][Hkv][D]    keys / values of every layer
 * Query head h attends with key head h / (Hq / Hkv) (grouped-query attention).
 */
#ifndef MUKV_H_
#define MUKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct mukv_ctx mukv_ctx;          /* opaque, library-owned host object */
typedef void* mukv_stream;                 /* a cudaStream_t (NULL = legacy default stream) */

typedef enum {
  MUKV_OK = 0,
  MUKV_E_INVALID = -1,      /* null pointer, negative count, bad enum */
  MUKV_E_SHAPE = -2,        /* configuration outside the supported shapes */
  MUKV_E_DTYPE = -3,
  MUKV_E_ALIGN = -4,        /* device pointer not 16-byte aligned */
  MUKV_E_CAPACITY = -5,     /* store / workspace / per-call limit exceeded */
  MUKV_E_STATE = -6,        /* first_frame does not continue the stream, nothing stored, ... */
  MUKV_E_CUDA = -7,         /* a CUDA runtime call failed; message in mukv_last_error */
  MUKV_E_UNSUPPORTED = -8
} mukv_status;

typedef enum { MUKV_BF16 = 0, MUKV_FP32 = 1 } mukv_dtype;

/* Retrieval variants of Sec. 3.4 / the retrieval-mode ablation:
 * PARALLEL = stage 1 only (top-k by cosine); HIER = frames only inside the selected
 * segments; SEMI = the paper's method (stage 1 top-2k, Eq. 8 rerank, top-k). */
typedef enum { MUKV_RETR_PARALLEL = 0, MUKV_RETR_HIER = 1, MUKV_RETR_SEMI = 2 } mukv_retr_mode;

#define MUKV_MAX_QUESTIONS 128   /* questions per mukv_retrieve / mukv_gather call */
#define MUKV_MAX_TOPK 256        /* upper bound for k_seg, k_frm (2*k candidates <= 512) */
#define MUKV_MAX_TOKENS 256      /* upper bound for P (tokens per frame) */
#define MUKV_MAX_PATCH_SPLIT 4   /* upper bound for patch_split (16 super patches per frame) */

typedef struct {
  int32_t n_layers;              /* L                                                   */
  int32_t n_q_heads;             /* Hq, a multiple of n_kv_heads                        */
  int32_t n_kv_heads;            /* Hkv                                                 */
  int32_t head_dim;              /* D: 64 or 128                                        */
  int32_t tokens_per_frame;      /* P <= MUKV_MAX_TOKENS                                */
  int32_t keep_per_frame;        /* kappa = floor(rho * P), computed by the caller      */
  int32_t frames_per_segment;    /* frames pooled into one segment-level entry          */
  int32_t max_frames_per_chunk;  /* upper bound for n_frames of one compress call       */
  int32_t attn_causal;           /* 0: softmax over the whole frame; 1: keys j <= i     */
  int32_t keep_low_freq;         /* 0: high frequency scores are kept (paper default)   */
  float   alpha;                 /* Eq. 4 weight of the attention signal                */
  float   tie_eps;               /* scores within tie_eps of the k-th count as tied     */
  int32_t dtype;                 /* mukv_dtype of Q, K, V and of the stored pages       */
  int32_t patch_split;           /* s: patch-level blocks = the kept tokens inside each of
                                    the s x s super patches of a frame (Sec. 3.2); 0 = no
                                    patch level; at most 4                               */
  int32_t grid_width;            /* tokens per row of the frame's token grid (only read
                                    when patch_split > 0; must divide P)                 */
  int32_t n_score_layers;        /* Ls: Eq. 1-3 are averaged over Ls consecutive layers
                                    (the layer-choice ablation's "last-5 fusion": 5);
                                    0 counts as 1                                        */
  int32_t score_layer_offset;    /* layers between the last scoring layer and the end of
                                    the model: 0 = the last layer (paper default), 1 =
                                    penultimate, L/2 = middle; offset + Ls <= L           */
  int32_t keep_per_segment;      /* 0: every frame keeps keep_per_frame tokens (frame-
                                    level selection).  kappa_v > 0: segment-level selection
                                    (Sec. 3.3, "I_v in R^O"): Eq. 4 and the top-kappa_v run
                                    over all tokens of a segment, a frame keeps a variable
                                    number; see mukv_compress_chunk                      */
  int64_t max_frames;            /* capacity of the store, in frames                    */
  int32_t past_frames;           /* W: the queries of a chunk also attend to the kept keys
                                    of the W most recent frames stored before the chunk
                                    (Sec. 3.2: past KV of the same granularity); P + W *
                                    kappa <= 256; not with keep_per_segment; 0 = none.  A
                                    bf16 context stays on the tensor-core kernel while
                                    ceil8(P) + W * ceil8(kappa) <= 256 (the cached keys are
                                    rows of its key tile), else it scores on the multiply-
                                    add kernels, as every fp32 context does                */
  int32_t reserved;              /* set to 0                                            */
} mukv_config;

typedef struct {
  int64_t frames;                /* frames stored so far                                */
  int64_t segments;              /* segment entries present (last one may be partial)   */
  int64_t kept_tokens;           /* frames * kappa                                      */
  int64_t page_bytes;            /* bytes of one frame's page                           */
  int64_t store_bytes_used;      /* pages written so far, in bytes                      */
  int64_t refined_frames;        /* frames whose selection was redone in double         */
  int64_t refined_questions;     /* reserved (retrieval always scores in double)        */
  int64_t kernel_launches;       /* kernels launched by this context since creation     */
  int32_t device_status;         /* 0, or the first device-side event code recorded:
                                    3, 4, 5  a bounded wait inside the tensor-core scoring kernel
                                             ran out (producer, MMA issuer, epilogue): the chunk's
                                             scores are not to be trusted;
                                    6        the blocks of the double-precision pass waited in
                                             vain for one another: flagged frames were not stored;
                                    7        a frame's scores were not finite (Inf/NaN inputs):
                                             its kappa lowest token ids were kept            */
  int32_t reserved;
} mukv_stats;

/* Bytes the caller must provide for the compressed store / the scratch workspace.
 * Return 0 if the configuration is invalid. */
size_t mukv_store_bytes(const mukv_config* cfg);
size_t mukv_workspace_bytes(const mukv_config* cfg);

/* Creates a context over caller-owned device memory.  d_store and d_workspace must stay
 * valid until mukv_destroy; both are cleared where needed by stream-ordered memsets on the
 * legacy default stream followed by a device synchronise (creation is not a hot call).
 * Errors: INVALID (null), SHAPE/DTYPE (configuration), ALIGN, CAPACITY (buffers too small). */
mukv_status mukv_create(const mukv_config* cfg, void* d_store, size_t store_bytes,
                        void* d_workspace, size_t workspace_bytes, mukv_ctx** out);
void mukv_destroy(mukv_ctx* ctx);

/* Forgets every stored frame (capacity and buffers are kept) and clears the counters behind
 * mukv_get_stats (refined_frames, device_status).  The host-side frame counter is reset at once;
 * the device-side counters are cleared by a memset enqueued on `stream`, so the call must be
 * ordered after the context's earlier work like any other call. */
mukv_status mukv_reset(mukv_ctx* ctx, mukv_stream stream);

/* Options of a context.  They exist for tests and experiments; the defaults are what the
 * parity guarantees are stated for.
 *   MUKV_OPT_FLAG_MARGIN  frames whose lowest kept and highest dropped fused score differ by less
 *                         than tie_eps + margin are re-scored in double precision.  The built-in
 *                         margin (3e-6) can only be raised: smaller values return MUKV_E_INVALID.
 *   MUKV_OPT_SCORE_PATH   0 (default): bf16 chunks are scored on the tensor cores, fp32 chunks by
 *                         the multiply-add kernel;  1: the multiply-add kernel for every dtype.
 * Takes effect from the next mukv_compress_chunk. */
typedef enum { MUKV_OPT_FLAG_MARGIN = 0, MUKV_OPT_SCORE_PATH = 1 } mukv_option;
mukv_status mukv_set_option(mukv_ctx* ctx, int32_t option, double value);

/* Sec. 3.3 + Eq. 5.  Compresses frames first_frame .. first_frame+n_frames-1.
 *   d_q [n_frames][P][Hq][D] ([Ls][n_frames][P][Hq][D] with Ls scoring layers), d_k / d_v
 *   [L][n_frames][P][Hkv][D]: inputs, read only.
 *   first_frame must equal the number of frames already stored (timestamps are the
 *   absolute frame indices); 1 <= n_frames <= max_frames_per_chunk.
 *   d_kept_out  [n_frames][kappa] int32, ascending kept token ids per frame, or NULL.
 *   d_scores_out [3][n_frames][P] float: I_att (Eq. 1), I_fft (Eq. 3), fused I (Eq. 4), or NULL.
 * Per frame the call scores every token, keeps the kappa best (ties within tie_eps go to
 * the lowest index), copies their K/V rows of all layers into the frame's page, writes the
 * frame-level entry (float mean of the kept rows per layer, K and V) and refreshes the
 * entry of every segment the chunk touches (mean over the frames present so far).  With
 * frame-level selection that last step is owed to the store until it is next needed: the
 * next compress call, mukv_retrieve / mukv_retrieve3, mukv_gather3, mukv_store_region or
 * mukv_export_header pools the entries before anything reads them (the library's own kernel,
 * on the stream of the call that needs them).
 * Frames whose selection lies too close to a tie boundary for single precision are
 * re-scored in double precision on the device before they are stored.
 * With keep_per_segment = kappa_v > 0 the selection is made per segment: first_frame must be a
 * multiple of frames_per_segment and the chunk must hold whole segments (a last, shorter one ends
 * the stream and keeps kappa_v * frames / frames_per_segment tokens, rounded down); the min-max of
 * Eq. 4 and the ranking run over all tokens of a segment (bf16 chunks: scored on the tensor cores
 * and ranked in single precision where the margin of mukv_set_option allows, else, like fp32
 * chunks, in double precision); frame t keeps n_t
 * tokens (region 10), its page is [L][2][n_t][Hkv][D], kept ids are stored and returned as
 * [frames][P] int32 padded with -1 (d_kept_out must have that size), frames_per_segment * P <= 4096,
 * no patch level.  Such a store is read with mukv_retrieve / mukv_retrieve3 and mukv_gather3
 * (k_patch = 0); mukv_gather and mukv_compress_chunk_scored answer MUKV_E_UNSUPPORTED.
 * A frame whose fused scores are not all finite (Inf or NaN among its inputs) has no ranking:
 * its kappa lowest token ids are kept and device_status 7 is recorded.
 * Errors: INVALID, ALIGN, STATE (first_frame), CAPACITY (n_frames, store full), CUDA. */
mukv_status mukv_compress_chunk(mukv_ctx* ctx, const void* d_q, const void* d_k, const void* d_v,
                                int32_t n_frames, int64_t first_frame,
                                int32_t* d_kept_out, float* d_scores_out, mukv_stream stream);

/* Like mukv_compress_chunk, but each frame's tokens are ranked by numbers the caller supplies
 * instead of Eq. 1-4: d_select_scores [n_frames][P] float (device), higher = kept first, ties and
 * near-ties (within tie_eps) to the lowest token id.  This is how the "Rand(50%)" row of the paper's
 * compression-ablation table is reproduced (uniform random scores, kappa = P/2), and it lets a
 * caller plug in an indicator of its own.  No queries are needed.  The ranking runs in double
 * precision on the given floats, so it equals the exact rule; scores that are not finite make the
 * frame keep its kappa lowest ids (device_status 7).  Errors: as mukv_compress_chunk. */
mukv_status mukv_compress_chunk_scored(mukv_ctx* ctx, const float* d_select_scores, const void* d_k,
                                       const void* d_v, int32_t n_frames, int64_t first_frame,
                                       int32_t* d_kept_out, mukv_stream stream);

/* Sec. 3.4.  Serves nq questions in one batch.
 *   d_qtok      [sum Nq][Hq][D] last-layer query tokens of all questions, concatenated.
 *   h_q_offsets [nq+1] token offsets of each question in d_qtok (host, ascending, [0]=0).
 *   h_t_limit   [nq] or NULL: question i sees frames with id < t_limit[i] and the segments
 *               whose last stored frame is visible; NULL = everything stored.
 *   k_seg, k_frm  blocks to select per granularity (<= MUKV_MAX_TOPK); top_n = number of
 *               segment keys averaged into the global query (0 = k_seg); lambda_frm = Eq. 8
 *               coherence factor for frames (segments use 0).
 *   d_seg_idx [nq][k_seg], d_frm_idx [nq][k_frm]: selected ids ascending, unused slots -1.
 *   d_seg_score / d_frm_score: matching scores (stage-1 cosine for segments, final score
 *               for frames), or NULL.   d_counts [nq][2]: number of valid (segments, frames).
 * Errors: INVALID, ALIGN, CAPACITY (nq, k, question length, workspace), STATE (empty store). */
mukv_status mukv_retrieve(mukv_ctx* ctx, const void* d_qtok, const int32_t* h_q_offsets,
                          const int64_t* h_t_limit, int32_t nq,
                          int32_t k_seg, int32_t k_frm, int32_t top_n, float lambda_frm,
                          int32_t mode,
                          int32_t* d_seg_idx, int32_t* d_frm_idx,
                          float* d_seg_score, float* d_frm_score, int32_t* d_counts,
                          mukv_stream stream);

/* Sec. 3.4 over all three granularities (patch-, frame- and segment-level blocks), each with its
 * own k_g and lambda_g; the paper's values are k_g = {20, 32, 12}, lambda_g = {0.3, 0.3, 0}.
 * Stage 1 ranks every visible block of a granularity by cosine (Eq. 7) and keeps 2 k_g candidates;
 * stage 2 re-scores them against the mean of the top_n segment keys (Eq. 8) and keeps k_g
 * (lambda_g = 0: the k_g best of stage 1).  PARALLEL stops after stage 1; HIER looks for frame- and
 * patch-level blocks only inside the selected segments.  A patch-level block is (frame, super
 * patch), id = frame * S + super patch with S = patch_split^2; super patches that kept no token are
 * no blocks.  The store must have been created with patch_split > 0 when k_patch > 0.
 *   d_patch_idx [nq][k_patch] / d_patch_score: like the frame outputs; may be NULL when k_patch = 0.
 *   d_counts [nq][3]: valid (segments, frames, patch blocks).
 * Other arguments and errors as mukv_retrieve. */
typedef struct {
  int32_t k_patch, k_frm, k_seg;
  float lambda_patch, lambda_frm, lambda_seg;
  int32_t top_n;                 /* segment keys averaged into the global query; 0 = k_seg */
  int32_t mode;                  /* mukv_retr_mode */
} mukv_retr_params;
mukv_status mukv_retrieve3(mukv_ctx* ctx, const void* d_qtok, const int32_t* h_q_offsets,
                           const int64_t* h_t_limit, int32_t nq, const mukv_retr_params* params,
                           int32_t* d_seg_idx, int32_t* d_frm_idx, int32_t* d_patch_idx,
                           float* d_seg_score, float* d_frm_score, float* d_patch_score,
                           int32_t* d_counts, mukv_stream stream);

/* Sec. 3.4 (first paragraph) / Sec. 3.5: the decode context when the selected blocks of all three
 * granularities are loaded.  For question i, per layer l, K then V:
 *   d_decode + i*decode_stride_bytes : [L][2][tok_cap][Hkv][D] in the store dtype, with
 *   tok_cap = mukv_decode3_tokens(ctx, k_seg, k_frm, k_patch).  Token slots, in this order: one
 *   summary token per selected segment (the segment's pooled entry, Eq. 5, rounded to the store
 *   dtype), the kept tokens of the selected frames, the kept tokens of the selected patch-level
 *   blocks; every group ascending by block id.  Only the first d_ntok[i] slots are written.
 *   d_seg_idx / d_frm_idx / d_patch_idx / d_counts: as written by mukv_retrieve3 (device).
 *   d_ntok [nq] int32: valid token slots per question.   d_tok_meta [nq][tok_cap][2] int32 or NULL:
 *   (frame id, token id) per slot, (-1 - segment id, -1) for a summary token.
 * Errors: INVALID, ALIGN, CAPACITY (nq, k, stride too small), STATE (k_patch > 0 without patch level). */
int64_t mukv_decode3_tokens(const mukv_ctx* ctx, int32_t k_seg, int32_t k_frm, int32_t k_patch);
mukv_status mukv_gather3(mukv_ctx* ctx, const int32_t* d_seg_idx, const int32_t* d_frm_idx,
                         const int32_t* d_patch_idx, const int32_t* d_counts, int32_t nq,
                         int32_t k_seg, int32_t k_frm, int32_t k_patch, void* d_decode,
                         int64_t decode_stride_bytes, int32_t* d_ntok, int32_t* d_tok_meta,
                         mukv_stream stream);

/* Sec. 3.5.  For question i and layer l the kept K rows of the selected frames (ascending
 * frame id, ascending token id inside a frame) are concatenated, then the V rows:
 *   d_decode + i*decode_stride_bytes : [L][2 (K,V)][k_frm*kappa][Hkv][D] in the store dtype.
 * Only the first counts[i][1]*kappa token slots of each [l][K|V] plane are written.
 *   d_frm_idx [nq][k_frm], d_counts [nq][2]: as written by mukv_retrieve (device memory).
 *   d_tok_meta [nq][k_frm*kappa][2] int32 (frame id, token id) per slot, or NULL.
 * Errors: INVALID, ALIGN, CAPACITY (nq, k_frm, stride too small). */
mukv_status mukv_gather(mukv_ctx* ctx, const int32_t* d_frm_idx, const int32_t* d_counts,
                        int32_t nq, int32_t k_frm, void* d_decode, int64_t decode_stride_bytes,
                        int32_t* d_tok_meta, mukv_stream stream);

/* Device-side views into the store, for inspection and tests (do not write through them).
 * which: 0 pages (dtype)           [max_frames][L][2][kappa][Hkv][D]
 *        1 kept ids (int32)        [max_frames][kappa]
 *        2 frame entries (float)   [max_frames][L][2][C]
 *        3 segment entries (float) [max_segments][L][2][C]
 *        4 frame keys (float)      [max_frames][C]
 *        5 segment keys (float)    [max_segments][C]
 *        6 frame timestamps (int64)[max_frames]
 *        7 page table (int64 byte offsets from the store base) [max_frames]
 *        8 patch-level keys (float) [max_frames][S][C]     (patch_split > 0)
 *        9 patch-level token counts (int32) [max_frames][S]
 *       10 tokens kept per frame (int32) [max_frames]       (keep_per_segment > 0; region 1 is then
 *          [max_frames][P], padded with -1, and region 0 is packed pages of different lengths)
 * Returns NULL for an unknown region; *bytes (if not NULL) receives the region size.
 * Segment entries and keys (regions 3, 5) of the chunk of the last compress call are pooled lazily
 * (by the next compress call, or by whatever reads them first): this call, like
 * mukv_export_header, launches that pooling on the stream of that compress call if it is still
 * owed and waits for that stream, so what the pointer shows is complete; NULL also if that fails. */
void* mukv_store_region(const mukv_ctx* ctx, int32_t which, size_t* bytes);

/* Moving a store (the paper's "offline memory" outlives the questions; it prints no format).
 * The store buffer is position independent: every reference inside it is an offset from its
 * base.  mukv_export_header fills a small plain header (configuration, frames stored); the caller
 * copies the store's bytes wherever it likes (cudaMemcpy to another buffer, another device, the
 * host) once the stream has finished (mukv_export_header itself waits for the stream of the last
 * compress call when that call's segment entries were still to be pooled: see mukv_store_region;
 * it returns MUKV_E_CUDA if that fails).  mukv_import builds a context over such a copy: like
 * mukv_create, but the store's contents are kept and the stream continues at header->frames.
 * Errors of mukv_import: INVALID (null, bad magic / version), SHAPE/DTYPE, ALIGN, CAPACITY
 * (store_bytes below header->store_bytes, workspace too small). */
#define MUKV_STORE_MAGIC 0x564B754Du   /* "MuKV" */
#define MUKV_STORE_VERSION 1u
typedef struct {
  uint32_t magic, version;
  mukv_config cfg;
  int64_t frames;
  uint64_t store_bytes;            /* what mukv_store_bytes(&cfg) returned */
} mukv_store_header;
mukv_status mukv_export_header(const mukv_ctx* ctx, mukv_store_header* out);
mukv_status mukv_import(const mukv_store_header* header, void* d_store, size_t store_bytes,
                        void* d_workspace, size_t workspace_bytes, mukv_ctx** out);

/* Reads counters.  Copies a few device words: synchronises the given stream. */
mukv_status mukv_get_stats(mukv_ctx* ctx, mukv_stats* out, mukv_stream stream);

/* Optional per-kernel timing for benchmarks.  While enabled, every kernel launch of this
 * context is bracketed by a pair of CUDA events on the call's stream (host objects; no device
 * memory).  mukv_profile_read waits for the recorded events, adds up the elapsed milliseconds
 * and the launch counts per kernel kind since the last read, and forgets them.
 * Kinds: 0 score, 1 tail (double-precision pass of flagged frames; segment-level selection),
 *        2 compact+pool, 3 segment pool, 4 question pool, 5 index scan, 6 rank, 7 gather. */
#define MUKV_PROF_KINDS 8
mukv_status mukv_profile_enable(mukv_ctx* ctx, int32_t on);
mukv_status mukv_profile_read(mukv_ctx* ctx, double* ms, int64_t* launches);

/* Scores frames without any caller-provided scratch.  (The paper has no counterpart: this entry
 * point exists for the deployment case below, it computes what mukv_compress_chunk computes
 * for its d_kept_out / d_scores_out arguments and stores nothing.)
 *
 * Who needs it: code that must not, or cannot, obtain device memory of its own -- for example
 * a plug-in inside a serving process that handed all free device memory to its cache pool at
 * start-up, or a loop that is not allowed to call the allocator while it runs.  Such a caller
 * cannot build the workspace a mukv_ctx needs, but it may still want to know which tokens of a
 * frame the method would keep.
 *
 *   cfg        shapes and method parameters; n_layers, frames_per_segment, max_frames,
 *              max_frames_per_chunk, the scoring-layer and the patch-level fields are ignored
 *              (whatever they hold): the one layer the caller passes is scored.  Limits: n_frames <= MUKV_NOALLOC_MAX_FRAMES,
 *              n_q_heads <= MUKV_NOALLOC_MAX_Q_HEADS, n_kv_heads <= MUKV_NOALLOC_MAX_KV_HEADS,
 *              tokens_per_frame <= MUKV_MAX_TOKENS; larger requests return MUKV_E_CAPACITY.
 *   d_q        [n_frames][P][Hq][D] last-layer queries;  d_k_last [n_frames][P][Hkv][D] last-layer
 *              keys (device, 16-byte aligned, cfg->dtype).
 *   d_kept_out [n_frames][kappa] int32 ascending kept token ids, or NULL;
 *   d_scores_out [3][n_frames][P] float (I_att, I_fft, fused I), or NULL; not both NULL.
 *
 * The scratch (about 1.9 MB: per-head partial sums in float and double, arrival counters, the
 * list of frames that need the double-precision pass) is a fixed array inside the library; every
 * device that loads the library holds it until the process exits.  The call performs no
 * cudaMalloc / cudaFree and uses no allocating routine; it enqueues one small memset (the
 * counters must start at zero, the rest of the array is overwritten before it is read) and two
 * kernels on `stream`.  The first call on each device also looks up the array's device address
 * and raises the kernels' shared-memory limit; make that first call outside any stream capture.
 * All calls on a device share the one array: two calls whose kernels may overlap on the device
 * (different streams without an ordering between them) race.  Messages of failures are read
 * with mukv_last_error(NULL). */
#define MUKV_NOALLOC_MAX_FRAMES 16
#define MUKV_NOALLOC_MAX_Q_HEADS 32
#define MUKV_NOALLOC_MAX_KV_HEADS 8
mukv_status mukv_score_frames_noalloc(const mukv_config* cfg, const void* d_q, const void* d_k_last,
                                      int32_t n_frames, int32_t* d_kept_out, float* d_scores_out,
                                      mukv_stream stream);

/* Message of the last failure on this context (valid until the next call on it);
 * with ctx == NULL, the message of the last failed mukv_create on this thread. */
const char* mukv_last_error(const mukv_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* MUKV_H_ */
