/*
 * aspd.h -- C ABI of the B200 (sm_100a) branch-isolated attention library.
 *
 * The library implements one step of one attention layer of ASPD's Hybrid Decoding
 * Engine (Section 3.3 of the paper) under the model-side rules of Section 3.2
 * (Eq. 1-4): during a parallel segment every branch decodes its next token against the
 * shared prefix KV plus its own branch's KV only, all branches sharing position IDs per
 * timestep; when the segment ends, serial decoding continues over the merged cache,
 * which is reused as it lies (nothing is copied or re-encoded).
 *
 * Conventions
 *   - "host"/"device" on every pointer says where the memory lives.  The caller owns
 *     every buffer it passes; buffers must stay valid until the stream has passed the
 *     call.  The library owns only plans.
 *   - Every function returns 0 (ASPD_OK) or a negative aspd_status_t; nothing throws,
 *     aborts or synchronises the device unless stated.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *   - Token order: the new tokens of a step are ordered request-major, then branch, then
 *     token inside the branch.  q, out, k_new, v_new and pos all use that order.
 *   - Layouts: q, out [n_new][n_q_heads][head_dim]; k_new, v_new [n_new][n_kv_heads]
 *     [head_dim]; element type per aspd_shape_t.dtype.  The K and V pools are
 *     [n_pool_pages][n_kv_heads] tiles of page_size x head_dim elements each
 *     (aspd_pool_bytes gives the size); the order of elements INSIDE a tile is private to
 *     the library -- read tokens back with aspd_debug_read_token.  Pools must be zero-filled
 *     (or at least hold no NaN/Inf bit patterns) before their first use: the rows of a partly
 *     filled page that no token has been written to yet are multiplied by a weight of exactly 0.
 *     Device buffers (q, out, k_new, v_new, the pools) must start on a 16-byte boundary (the
 *     kernels move them in 16-byte pieces); a call given one that does not returns
 *     ASPD_ERR_INVALID_ARG and launches nothing.
 *   - Positions are 0-based.  Query head h uses KV head h / (n_q_heads / n_kv_heads).
 *     RoPE pairs element i with i + head_dim/2 and uses inv_freq[i] = theta^(-2i/head_dim)
 *     (the paper leaves the encoding open; this is the rotate-half convention of the
 *     models it fine-tunes).
 */
#ifndef ASPD_H_
#define ASPD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  ASPD_OK = 0,
  ASPD_ERR_INVALID_ARG = -1,    /* null pointer, negative count, wrong mode              */
  ASPD_ERR_BAD_DESCRIPTOR = -2, /* overlapping regions, slot beyond the page table, ...  */
  ASPD_ERR_UNSUPPORTED = -3,    /* head_dim / page_size / dtype outside what is built     */
  ASPD_ERR_CUDA = -4,           /* a CUDA runtime call or a launch failed                 */
  ASPD_ERR_TIMEOUT = -5,        /* a bounded device-side wait ran out (see aspd_plan_status) */
  ASPD_ERR_NOMEM = -6,          /* host or device allocation failed at plan creation      */
  ASPD_ERR_TOO_LARGE = -7       /* a size exceeds a stated maximum                        */
} aspd_status_t;

enum { ASPD_MODE_BRANCH = 0, ASPD_MODE_SERIAL = 1 };
enum { ASPD_DTYPE_F32 = 0, ASPD_DTYPE_BF16 = 1 };
/* aspd_branch_t.q_len of a region that belongs to an EARLIER stage (a merged branch, or the serial
 * tokens written between two parallel stages): every token of the step sees all of it. */
enum { ASPD_Q_SHARED = -1 };
/* aspd_branch_t.pos_start value that makes the library derive the paper's shared position-ID rule
 * itself (Eq. 4: stage_start = the number of tokens before the stage). */
enum { ASPD_POS_AUTO = -1 };
enum { ASPD_KERNEL_AUTO = 0, ASPD_KERNEL_GENERIC = 1, ASPD_KERNEL_MMA = 2 };

/* One request (host memory).  Logical slot s of the request lives in physical page
 * page_ids[page_begin + s / page_size], row s % page_size. */
typedef struct {
  int32_t prefix_len;   /* P: shared main-branch tokens at logical slots [0, P)            */
  int32_t n_branches;   /* N >= 0                                                           */
  int32_t branch_begin; /* first entry of this request in the branch array                  */
  int32_t page_begin;   /* first entry of this request in page_ids[]                        */
  int32_t n_pages;      /* length of this request's page table                              */
  int32_t tail_off;     /* first logical slot of the main-branch tokens written after the
                           segment closed (page-aligned); used by serial mode              */
  int32_t tail_len;     /* their number, including the token appended this step            */
} aspd_request_t;

/* One parallel branch (host memory). */
typedef struct {
  int32_t kv_off;    /* first logical slot of the branch (page-aligned)                     */
  int32_t kv_len;    /* tokens of the branch in the cache AFTER this step's append          */
  int32_t pos_start; /* position ID of the branch's first token.  ASPD_POS_AUTO: the library applies
                        Eq. 4 itself -- stage_start = the number of tokens before the stage = the
                        request's prefix_len plus the kv_len of all its ASPD_Q_SHARED regions, the same
                        for every branch of the stage (branches share the ID of a timestep).  Any
                        value >= 0 is taken as given (position-ID variants of the ablation).  Ignored
                        for ASPD_Q_SHARED regions and in serial mode.                              */
  int32_t q_len;     /* query tokens this step = the LAST q_len tokens (0: finished branch of the
                        current stage, invisible to the other branches; ASPD_Q_SHARED: region of an
                        earlier stage, visible to every branch -- Eq. 3, different stages)       */
} aspd_branch_t;

typedef struct {
  int32_t n_q_heads, n_kv_heads;
  int32_t head_dim;  /* 64 or 128 */
  int32_t page_size; /* tokens per page: 16 (8, 32 also accepted by the generic kernel) */
  int32_t dtype;     /* ASPD_DTYPE_* : element type of q, out, k_new, v_new and the pools */
  float rope_theta;
  float sm_scale;    /* Eq. 1's 1/sqrt(d_k), as a parameter */
} aspd_shape_t;

/* Optional knobs of plan creation (NULL = all automatic). */
typedef struct {
  int32_t kernel;       /* ASPD_KERNEL_* */
  int32_t chunk_tokens; /* cut work items at least every this many keys (multiple of
                           page_size); 0 = only at the CTA boundaries                      */
  int32_t n_ctas;       /* size of the persistent grid; 0 = auto                           */
  int32_t host_only;    /* 1: build the work list on the host only (no CUDA call at all);
                           such a plan serves aspd_plan_info / aspd_plan_items only        */
  int32_t stable_cache; /* 1: the caller promises that, when an attention call of this plan is
                           made, nothing still in flight on the stream writes K/V pages the plan
                           reads, except this step's own new rows (written by aspd_kv_append with
                           this plan, or by the fused step).  True for a decode loop, where a
                           layer's pools are only touched by that layer's own step.  The kernel
                           may then start fetching such pages before the previous kernel on the
                           stream has finished.  0 (default): full stream ordering for the pools */
  int32_t mask;         /* ASPD_MASK_*: attention mask of a parallel step (default: branch-invisible) */
  int32_t updatable;    /* 1: leave room in the plan's tables (25 %) for aspd_plan_update                */
  int32_t combine;      /* ASPD_COMBINE_*: where a7 (the merge of a token's split-K records) runs        */
  int32_t wide_rows;    /* plans that deal whole streams to the tensor-core kernel: query rows of a row
                           block, 128 (one tile) or 256 (two tiles scored against every K/V tile the CTA
                           fetches); 0 = automatic (256 when a request has more query tokens than one
                           tile holds)                                                                */
  int32_t mma_m;        /* stream-K plans of the tensor-core kernel: M of its MMAs, 128 (the at most 64 query
                           rows of a row block are replicated to fill 128 accumulator rows), 64 (half the
                           tensor work; the accumulators then use 16 lanes of each quadrant) or 96, which
                           stands for both: scores at M = 128, P.V at M = 64; 0 = automatic (96)        */
} aspd_tuning_t;

/* a7 of a stream-K plan of the tensor-core kernel.  KERNEL: the separate combine launch (what AUTO
 * takes: it measured faster on every workload of the benchmark).  FUSED: one launch per layer --
 * every CTA counts the records of a (token, KV head) as it stores its own, and the CTA that stores
 * the last one merges them all, in record order, and writes the output (no CTA ever waits for
 * another); a key stream that lies inside one CTA is normalised and written by that CTA without
 * any record.  Both give the same bits.  FUSED is honoured where the plan allows it (not the
 * generic kernel, which keeps the combine launch, and not plans that deal whole streams, which
 * need no merge at all); aspd_plan_info_t.single_launch says what the plan does. */
enum { ASPD_COMBINE_AUTO = 0, ASPD_COMBINE_KERNEL = 1, ASPD_COMBINE_FUSED = 2 };

/* Attention mask of a parallel step.  BRANCH_INVISIBLE is the paper's mask (its Eq. 2-3).  SHARED
 * is the visible mask of its attention-mask ablation, read as "only the order of the position IDs
 * remains": a new token at offset k of its branch also sees the first k tokens of every other
 * branch of its stage (branches with q_len = 0 included) -- what exists when the branches decode
 * in lockstep.  Serial steps are the same under both.  SHARED plans never fuse the append into the
 * attention pass and never deal whole streams. */
#define ASPD_MASK_BRANCH_INVISIBLE 0
#define ASPD_MASK_SHARED 1

/* One split-K work item of a plan, as aspd_plan_items reports it.  The pages a request's
 * step must read form one key stream (prefix, then the branches that have queries, or every
 * branch and the tail in serial mode); an item is a run of pages of that stream for one KV
 * head and one block of query tokens.  Key k of the stream is row k % page_size of stream page
 * k / page_size. */
typedef struct {
  int32_t q_tok0;     /* first new token (step order) of the item's row block               */
  int32_t n_q_tok;    /* tokens in the block; rows = n_q_tok * (n_q_heads / n_kv_heads) <= max_rows_per_item */
  int32_t kv_head;
  int32_t page0;      /* index of the item's first page in the plan's stream-page list       */
  int32_t n_pages;    /* pages of the item                                                   */
  int32_t key0;       /* stream key index of the item's first key                            */
  int32_t part_slot;  /* which partial record of (token, KV head) this item writes           */
  int32_t request;
  int32_t row_block;  /* index of the item's block of query tokens among all blocks of the step */
  int32_t n_parts;    /* items the key stream of (row block, KV head) was cut into = records per row */
} aspd_item_t;

typedef struct {
  int32_t n_new;            /* new tokens (= query tokens) of the step                      */
  int32_t n_items;          /* split-K work items                                           */
  int32_t n_partials;       /* partial (m, l, O) records, summed over (token, KV head)      */
  int32_t n_stream_pages;   /* entries of the stream-page list                             */
  int32_t kernel;           /* ASPD_KERNEL_* actually chosen                                */
  int32_t chunk_tokens;     /* forced maximum keys per item (0: none)                       */
  int32_t n_ctas;           /* CTAs of the persistent grid = shares the streams are cut into */
  int32_t fused_append;     /* 1: aspd_branch_step / aspd_serial_step write the new rows inside the
                               attention pass; 0: they run the append kernel first               */
  int32_t direct_output;    /* 1: one item per (token, KV head) and the attention kernel writes the
                               output itself (no records, no combine launch)                     */
  int32_t max_rows_per_item;/* query rows (tokens x group heads) an item may carry: 64, 128 or 256  */
  int32_t dealt;            /* 1: whole streams dealt to the CTAs (every row block has a page list of its
                               own, so n_stream_pages counts shared pages once per row block); 0: stream-K cuts */
  int32_t single_launch;    /* 1: the attention kernel merges the split-K records itself (ASPD_COMBINE_FUSED): the
                               attention and step calls are one launch; 0: a combine launch follows      */
  int32_t mma_m;            /* M of the tensor-core kernel's MMAs in this plan: 128, 64 or 96 (see aspd_tuning_t;
                               0: generic kernel)                                                          */
  int32_t reserved;
  int64_t workspace_bytes;  /* device memory the plan holds                                 */
  int64_t kv_tokens_read;   /* cached tokens the step must read (each once)                 */
  int64_t algorithmic_bytes;/* K+V of those tokens + q in + out + appended K/V              */
} aspd_plan_info_t;

typedef struct aspd_plan aspd_plan_t;

const char* aspd_strerror(int status);

/* Bytes of one pool (K or V) with n_pages pages; 0 if the shape is unsupported. */
size_t aspd_pool_bytes(const aspd_shape_t* shape, int64_t n_pages);

/* Number of new tokens of a step: sum of q_len (branch mode) or n_req (serial mode). */
int aspd_count_new_tokens(const aspd_request_t* req /*host*/, const aspd_branch_t* br /*host*/,
                          int n_req, int mode);

/*
 * Position ID and logical slot of every new token (Eq. 4; Section 3.3: positions grow by
 * one per token inside a branch, and the first serial token after a segment takes its index
 * in the complete sequence).  Pure host integer code, no CUDA.
 *   branch mode: i-th query of a branch -> pos_start + kv_len - q_len + i, with pos_start derived
 *                per Eq. 4 where the descriptor says ASPD_POS_AUTO; slot kv_off + kv_len - q_len + i
 *   serial mode: prefix_len + sum of kv_len + tail_len - 1, slot tail_off + tail_len - 1
 * pos_out, slot_out, req_out: host arrays of aspd_count_new_tokens entries (req_out may be NULL).
 */
int aspd_positions(const aspd_request_t* req, const aspd_branch_t* br, int n_req, int mode,
                   int32_t* pos_out, int32_t* slot_out, int32_t* req_out);

/*
 * Mask membership as integers (Eq. 2-3 in descriptor form): vis_out[t * n_slots + s] = 1 iff
 * new token t may attend logical slot s of its own request.  Host only, for tests.
 */
int aspd_visible_slots(const aspd_request_t* req, const aspd_branch_t* br, int n_req, int mode,
                       int n_slots, uint8_t* vis_out /*host*/);

/* aspd_visible_slots under either attention mask (ASPD_MASK_*): with ASPD_MASK_SHARED a new token at
 * offset k of its branch also attends the slots at offsets below k of the stage's other branches
 * (the paper's attention-mask ablation).  Serial mode is the same under both.  Host only, for tests. */
int aspd_visible_slots_masked(const aspd_request_t* req, const aspd_branch_t* br, int n_req, int mode, int mask,
                              int n_slots, uint8_t* vis_out /*host*/);

/*
 * Validate the descriptors and build the step's plan: new-token table, query RoPE table,
 * split-K work list over (request, KV head, key chunk), partial-result workspace.  One plan
 * serves every layer of the step.  All device allocation of the library happens here
 * (unless tuning->host_only); copies are enqueued on `stream`.
 *   page_ids      host, concatenated page tables
 *   n_pool_pages  pages in each pool; every page id must be < n_pool_pages and unique
 *   q_pos         host, optional (NULL = derive as aspd_positions does): RoPE position of
 *                 each new token's query
 * Errors: ASPD_ERR_BAD_DESCRIPTOR for overlapping or out-of-table regions, unaligned kv_off /
 * tail_off, q_len > kv_len, serial mode with tail_len < 1, duplicate or out-of-pool page ids.
 */
int aspd_plan_create(const aspd_shape_t* shape, const aspd_request_t* req, const aspd_branch_t* br,
                     const int32_t* page_ids, int n_req, int64_t n_pool_pages, int mode,
                     const int32_t* q_pos, const aspd_tuning_t* tuning, void* stream,
                     aspd_plan_t** plan_out);
/*
 * Destroys the plan.  Work of the plan that is still in flight need not be waited for: the plan's
 * device block is parked with an event recorded on every stream the plan was used on, and a later
 * aspd_plan_create reuses a parked block of fitting size after making its own stream wait for
 * those events (so a decode loop that makes a plan per step neither allocates nor synchronises in
 * steady state).  Up to 8 blocks and 2 GiB in total are kept per process; what does not fit is
 * freed at once (cudaFree, which waits for the device).
 */
int aspd_plan_destroy(aspd_plan_t* plan);
/*
 * Re-plans an existing device plan for the NEXT step of the same batch, in place: same requests and
 * branches decoding (the number of new tokens, the grid and the kernel variant must come out the
 * same), lengths as given by the new descriptors.  The tables are rebuilt on the host and uploaded
 * on `stream` to the addresses they already have, so kernel launches recorded in a CUDA graph with
 * this plan stay valid: a decode loop captures one step once and per step calls aspd_plan_update
 * and replays the graph, on one stream.  Create the plan with tuning->updatable = 1 so that the
 * length-dependent tables have room to grow.
 * Returns ASPD_ERR_UNSUPPORTED when the new step needs another launch sequence (other number of
 * new tokens, grid, kernel variant, fused or separate append) and ASPD_ERR_TOO_LARGE when a table
 * has outgrown its room; the plan is unchanged then and the caller makes a new one (and a new graph).
 */
int aspd_plan_update(aspd_plan_t* plan, const aspd_request_t* req, const aspd_branch_t* br, const int32_t* page_ids,
                     int n_req, const int32_t* q_pos /*host, optional*/, void* stream);
/* Frees the parked device blocks (e.g. before handing the GPU's memory to someone else). */
int aspd_release_cached_memory(void);
int aspd_plan_info(const aspd_plan_t* plan, aspd_plan_info_t* info /*host*/);
/* Copy up to max_items work items to `items` (host); returns the number of items. */
int aspd_plan_items(const aspd_plan_t* plan, aspd_item_t* items, int max_items);
/* First work item of every CTA of the persistent grid: CTA c owns items [first[c], first[c + 1])
 * of aspd_plan_items (host array of n_ctas + 1 entries). Returns n_ctas. */
int aspd_plan_cta_ranges(const aspd_plan_t* plan, int32_t* first /*host*/, int max_entries);
/* The plan's stream-page list: physical page and number of valid rows of every page the step
 * reads (host arrays of n_stream_pages entries each). */
int aspd_plan_stream_pages(const aspd_plan_t* plan, int32_t* page_ids /*host*/, int32_t* n_valid /*host*/,
                           int max_pages);
/* Per new token, the stream keys it may attend: [0, pe) and [lo, hi) (host arrays of n_new). */
int aspd_plan_token_ranges(const aspd_plan_t* plan, int32_t* pe, int32_t* lo, int32_t* hi, int max_tokens);
/* Plans with ASPD_MASK_SHARED: per new token its offset k in its branch (it also attends keys of
 * other branches at offsets below k), and per stream page the page's index inside its branch
 * (host arrays of n_new and n_stream_pages entries).  ASPD_ERR_INVALID_ARG for other plans. */
int aspd_plan_shared_mask_tables(const aspd_plan_t* plan, int32_t* below /*host*/, int32_t* page_in_branch /*host*/);
/* Device status word of the plan (synchronises `stream`): ASPD_OK, or the first error a kernel
 * recorded since the plan was created: ASPD_ERR_TIMEOUT from a bounded wait; in a library built
 * with -DASPD_DEBUG_BOUNDS also ASPD_ERR_BAD_DESCRIPTOR from a kernel that met a page id or row
 * outside the pool (it skips the access).  aspd_plan_update leaves the word as it is. */
int aspd_plan_status(aspd_plan_t* plan, void* stream);

/*
 * a3: K' = RoPE(k_new, pos), V' = v_new, written into the paged cache at the slots the plan
 * derived from the descriptors (Section 3.3: KV of parallel tokens joins the one shared
 * cache).  pos: device int32[n_new], caller-given position IDs (aspd_positions for ASPD;
 * other values implement position-ID variants).  RoPE in fp32 with the angle reduced in
 * fp64; bf16 stores round to nearest even.
 */
int aspd_kv_append(aspd_plan_t* plan, const void* k_new /*device*/, const void* v_new /*device*/,
                   const int32_t* pos /*device*/, void* k_pool /*device*/, void* v_pool /*device*/,
                   void* stream);

/*
 * a4-a7: parallel-mode attention (Eq. 1 under the mask of Eq. 2-3).  Query i of branch b
 * attends the prefix [0, P) and tokens 0 .. kv_len - q_len + i of its own branch; the prefix
 * is read once per KV head for all branches' query heads.  Split-K partials are merged by
 * log-sum-exp.  The plan must have been created in ASPD_MODE_BRANCH.  q is raw (un-rotated).
 */
int aspd_branch_attn(aspd_plan_t* plan, const void* q /*device*/, const void* k_pool /*device*/,
                     const void* v_pool /*device*/, void* out /*device*/, void* stream);

/*
 * a9: serial-mode attention after the segment closed: one query per request attends the
 * prefix, every token of every branch and the tail up to itself (the main branch sees the
 * whole history, Section 3.2).  The plan must have been created in ASPD_MODE_SERIAL.
 */
int aspd_serial_attn(aspd_plan_t* plan, const void* q /*device*/, const void* k_pool /*device*/,
                     const void* v_pool /*device*/, void* out /*device*/, void* stream);

/*
 * The two halves of either attention call, for callers (and profilers) that want them
 * apart: a4-a6, the split-K pass that leaves one un-normalised (max, sum, O) record per work
 * item and query row in the plan's workspace; and a7, the log-sum-exp merge of a token's
 * records into `out`.  aspd_branch_attn / aspd_serial_attn are exactly these two in sequence
 * (plans with 256-row blocks, whose kernel only writes final outputs, return
 * ASPD_ERR_UNSUPPORTED from aspd_attn_partials).
 */
int aspd_attn_partials(aspd_plan_t* plan, const void* q /*device*/, const void* k_pool /*device*/,
                       const void* v_pool /*device*/, void* stream);
int aspd_attn_combine(aspd_plan_t* plan, void* out /*device*/, void* stream);
/* The first half of aspd_branch_step / aspd_serial_step alone, for plans whose step fuses the append
 * (aspd_plan_info_t.fused_append = 1 and direct_output = 0): the attention pass that first writes
 * the step's new K/V rows and then leaves the (max, sum, O) records; aspd_attn_combine completes
 * it.  ASPD_ERR_UNSUPPORTED for other plans.  For profilers and the benchmark's kernel timing. */
int aspd_step_partials(aspd_plan_t* plan, const void* q /*device*/, const void* k_new /*device*/,
                       const void* v_new /*device*/, void* k_pool /*device*/, void* v_pool /*device*/, void* stream);

/*
 * a3 + a4-a7 (or a3 + a9) in one call: the step's new K/V rows are written into the cache by the
 * attention pass itself, just before it reads the pages they live in (each CTA writes the rows of
 * the pages it is about to read; CTAs that share a page write identical bytes), so no separate
 * append launch is needed.  The position IDs are the plan's (aspd_positions, or q_pos if given);
 * results equal aspd_kv_append followed by aspd_branch_attn / aspd_serial_attn up to the last bit
 * of the cos/sin evaluation.  k_new, v_new as for aspd_kv_append.
 */
int aspd_branch_step(aspd_plan_t* plan, const void* q /*device*/, const void* k_new /*device*/,
                     const void* v_new /*device*/, void* k_pool /*device*/, void* v_pool /*device*/,
                     void* out /*device*/, void* stream);
int aspd_serial_step(aspd_plan_t* plan, const void* q /*device*/, const void* k_new /*device*/,
                     const void* v_new /*device*/, void* k_pool /*device*/, void* v_pool /*device*/,
                     void* out /*device*/, void* stream);

/*
 * The whole step (a3-a7 or a3 + a9, by the plan's mode) from HOST buffers: copies q, k_new,
 * v_new to staging memory the plan owns, runs the step, copies out back, all on `stream`, then
 * synchronises it.  The pools stay on the device (they are the state).
 *   - When pos equals the position IDs the plan derived (aspd_positions, or its q_pos), which is
 *     compared on the host, the step is aspd_branch_step / aspd_serial_step (new rows written by
 *     the attention pass where the plan allows) and pos is not copied; otherwise pos goes up too
 *     and the step is aspd_kv_append with those positions followed by the attention call.
 *   - When k_new starts where q ends and v_new where k_new ends (one packed host buffer), one copy
 *     moves all three.
 */
int aspd_step_host(aspd_plan_t* plan, const void* q /*host*/, const void* k_new /*host*/,
                   const void* v_new /*host*/, const int32_t* pos /*host*/, void* k_pool /*device*/,
                   void* v_pool /*device*/, void* out /*host*/, void* stream);

/*
 * The same without the final synchronisation: everything is enqueued on `stream` and the call
 * returns.  The host buffers must be page-locked and stay valid (out: unread) until the stream
 * has passed the call.  The staging memory belongs to the plan, so calls with the same plan are
 * ordered by using one stream for them; to overlap the copies of one call with the kernels of
 * another, give the calls different plans and different streams (e.g. the layers of a model
 * alternating between two plans of the same step).
 */
int aspd_step_host_async(aspd_plan_t* plan, const void* q /*host*/, const void* k_new /*host*/,
                   const void* v_new /*host*/, const int32_t* pos /*host*/, void* k_pool /*device*/,
                   void* v_pool /*device*/, void* out /*host*/, void* stream);

/*
 * Attention of a step for callers that must not allocate device memory (the paper has no
 * counterpart; this is a convenience of the library).
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a memory pool that owns
 * the whole device, in a latency-critical serving loop whose allocator may not be re-entered,
 * or in a process that was handed a fixed memory budget -- and therefore cannot create a
 * device plan with aspd_plan_create, which allocates the plan's tables and split-K workspace.
 *
 * `plan` is a HOST-ONLY plan (aspd_tuning_t.host_only = 1; building it makes no CUDA call).
 * The call copies the plan's tables into a scratch array that is compiled into the library
 * (a file-scope __device__ array of ASPD_STATIC_SCRATCH_BYTES bytes; every GPU that loads the
 * library holds that much memory until the process exits), runs the same split-K pass and
 * combine as aspd_branch_attn / aspd_serial_attn (by the plan's mode) with all scratch inside
 * that array, and writes `out`.  It calls no cudaMalloc / cudaFree and no allocating library
 * routine.  q, k_pool, v_pool, out are device buffers as for aspd_branch_attn.
 *
 *  - Plans whose tables plus workspace exceed ASPD_STATIC_SCRATCH_BYTES (less its last 256 bytes,
 *    which hold the status word) are rejected with ASPD_ERR_TOO_LARGE before anything is launched.
 *  - The first call on a device looks the array's device address up (once per device, with
 *    that device current; host threads are serialised on that look-up).  The array's memory is
 *    taken when the CUDA module that holds it is loaded, which with lazy loading may be this first
 *    call; make it outside any stream capture.
 *  - The tables are copied from pageable host memory that lives only as long as the call, so the
 *    host may wait inside the call until earlier work on the stream has drained, and a call on a
 *    stream that is being captured returns ASPD_ERR_UNSUPPORTED and enqueues nothing.
 *  - All calls share the one array, which keeps the previous call's contents; every call
 *    rewrites the tables and clears the status word it needs.  Two calls that overlap on the GPU
 *    (different streams, or different host threads) race on it: serialise them.
 *  - A bounded device-side wait that ran out is recorded in the array's status word, which
 *    aspd_static_status reads (it synchronises `stream`; ASPD_OK, or ASPD_ERR_TIMEOUT, of the last
 *    call on the current device).
 */
#define ASPD_STATIC_SCRATCH_BYTES (8u << 20)
int aspd_attn_static(const aspd_plan_t* plan /*host-only*/, const void* q /*device*/, const void* k_pool /*device*/,
                     const void* v_pool /*device*/, void* out /*device*/, void* stream);
int aspd_static_status(void* stream);

/* Read one cached token (physical page, row, KV head) back as head_dim floats (host).
 * Synchronises `stream`.  For tests. */
int aspd_debug_read_token(const aspd_shape_t* shape, const void* pool /*device*/, int64_t page,
                          int row, int kv_head, float* out /*host*/, void* stream);

/*
 * Move cached keys to new position IDs in place: K'(pos + delta) = RoPE(K'(pos), delta).  The
 * paper's "Same-Re" variant renumbers the positions of a finished parallel segment sequentially
 * and pays for it with a re-prefill of the KV cache (its position-ID ablation); because rotations
 * compose, re-rotating the cached keys does the same with one read and one write per key and no
 * model pass.  Token t is row rows[t] of physical page pages[t] (all KV heads); delta[t] may be
 * negative.  pages, rows, delta: device int32[n].  V is untouched.  Each call rounds the keys to
 * the storage dtype once more.  A token must not be listed twice in one call.
 */
int aspd_k_rerotate(const aspd_shape_t* shape, void* k_pool /*device*/, const int32_t* pages /*device*/,
                    const int32_t* rows /*device*/, const int32_t* delta /*device*/, int n, void* stream);

/*
 * The same for whole ranges of logical slots, which is what Same-Re renumbering moves: range i is
 * (page-table base, first slot, count, delta) -- `count` consecutive slots from `first` of the
 * request whose page table starts at page_table[base], all moved by `delta` positions (a finished
 * branch moves as a whole: delta = the tokens of the branches listed before it).  The kernel
 * derives page and row itself, so no per-token index arrays exist or are read.
 *   page_table  device int32, the concatenated page tables (as aspd_plan_create's page_ids)
 *   ranges      HOST int32[n_ranges][4]; they travel in the launch parameters, 512 per launch
 * The ranges of one call must not overlap (every key is read and written once, by one block).
 * ASPD_ERR_BAD_DESCRIPTOR for a negative base, slot or count.
 */
int aspd_k_rerotate_ranges(const aspd_shape_t* shape, void* k_pool /*device*/, const int32_t* page_table /*device*/,
                           const int32_t* ranges /*host*/, int n_ranges, void* stream);

/*
 * The same for the K pools of several layers in one launch (a finished segment is renumbered in
 * every layer of the model at once; the layers share the page tables, so the same slots move in
 * each).  k_pools: HOST array of n_layers device pointers, read before the call returns; 64 pools
 * per launch.  Pools must not overlap.  Same results, bit for bit, as n_layers calls of
 * aspd_k_rerotate_ranges; one launch of n_layers times the blocks instead of n_layers short ones.
 */
int aspd_k_rerotate_ranges_layers(const aspd_shape_t* shape, void* const* k_pools /*host array of device pointers*/,
                                  int n_layers, const int32_t* page_table /*device*/,
                                  const int32_t* ranges /*host*/, int n_ranges, void* stream);

/*
 * Failure-path check: runs the library's bounded device-side wait on a barrier nobody ever
 * arrives on, with a limit of `limit_cycles` SM clock cycles (at most 4e9).  The kernel gives up
 * when the limit passes and reports ASPD_ERR_TIMEOUT through *status_out (host); the context
 * stays usable.  This is the same wait every hand-off of the tensor-core kernel uses.
 * Synchronises `stream`.
 */
int aspd_debug_bounded_wait(int64_t limit_cycles, int32_t* status_out /*host*/, void* stream);

/*
 * Checking builds (-DASPD_DEBUG_BOUNDS; python -m paper_2508_08895_b200.build --debug-bounds): the
 * kernels compare every page id they are about to use with the number of pool pages and every row
 * with the page size; on a violation they record ASPD_ERR_BAD_DESCRIPTOR in the plan's status word
 * and leave the access out (a read is redirected to page 0) -- nothing traps or faults.  Plans
 * the library built never violate (aspd_plan_create validates on the host), so to see the check
 * work this call LOWERS the page count the kernels of `plan` compare against (n_pages <= the plan's
 * n_pool_pages; the pools themselves stay as large as they are, so nothing is out of bounds).
 * Other builds return ASPD_ERR_UNSUPPORTED.
 */
int aspd_debug_pool_limit(aspd_plan_t* plan, int64_t n_pages);

/*
 * Development aid of the tensor-core attention kernel.  In a library built with -DASPD_TC_PROFILE,
 * CTA `cta` of every later launch stamps its clock at the pipeline events of its first 64 tiles
 * into device_buf[0 .. 1024) and every CTA stamps the global timer (ns) into device_buf[1024 +
 * 8 * blockIdx ..): at entry, after set-up, after its last record, after the final barrier, then
 * (plans that merge inside the kernel) records stored / fenced / counted of its last announced
 * item, and after its merges (device memory of at least 1024 + 8 * n_ctas int64, caller-owned and
 * zero-filled; NULL switches the stamps off).  Other builds return
 * ASPD_ERR_UNSUPPORTED.
 */
int aspd_debug_profile(void* device_buf /*device*/, int cta);

#ifdef __cplusplus
}
#endif
#endif /* ASPD_H_ */
