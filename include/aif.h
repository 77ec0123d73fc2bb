/*
 * libaif -- C ABI of the B200 (sm_100a) pre-ranking scoring pass of AIF, the Asynchronous Inference
 * Framework for pre-ranking (Sections 2-4 of the paper).
 *
 * The calls follow the paper's split of one request (Section 2, Figure 2b):
 *   - item side, nearline (Section 3.2, 3.4):  aif_item_nearline_refresh writes precomputed item vectors
 *     (and their BEA weights / LSH signatures) into an item table that lives in GPU memory;
 *   - user side, online-asynchronous (Section 3.1, 3.3): aif_user_precompute runs, on a side stream and
 *     in parallel with retrieval, the user-side network (eqs. 1-3), copies the user-side part of the
 *     cross features into a pre-cache and caches the user's partial product of the first MLP layer;
 *   - real time (Section 3.1 "Real-Time Prediction Phase", Section 4): aif_score / aif_score_batch take
 *     candidate ids and return logits.
 *
 * Conventions
 *   - Every function returns an int: AIF_OK (0) or a negative AIF_ERR_* code.  Nothing throws, aborts or
 *     traps the GPU.  Argument, shape and version errors are returned at once.  What only the GPU can
 *     see (a candidate id outside the table, a bounded device-side wait that ran out) sets a bit in a device status
 *     word, the affected logits are NaN, and aif_poll_status reports it.  AIF_STATUS_TIMEOUT stays set until it is
 *     polled, and while it is set the kernel-per-layer path answers NaN: poll after a timeout before scoring on.
 *   - "device" pointers are GPU global memory, "host" pointers are ordinary host memory; the comment of
 *     each argument says which.  The caller owns every buffer it passes; the context owns the item
 *     table, the weight copies, the user-state arena and its scratch memory.
 *   - aif_stream is a cudaStream_t passed as a plain pointer (NULL = the default stream).  All work is
 *     stream-ordered; no call synchronises the device unless its comment says so.
 *   - Storage type (aif_config.dtype): AIF_F32 or AIF_BF16.  It is the element type of the item table, of
 *     the user-side tensors, of the cross pre-cache and of the weights.  Biases, the cached partial
 *     product, accumulators, softmax statistics and logits are always fp32.
 *   - Matrices are row-major.  A weight W of a layer y = W x + b is [out x in].
 *   - One context is bound to the CUDA device that was current when it was created.  Calls on one
 *     context must not overlap in time on different host threads.
 */
#ifndef AIF_H_
#define AIF_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    AIF_OK = 0,
    AIF_ERR_ARG = -1,       /* NULL or out-of-range argument */
    AIF_ERR_SHAPE = -2,     /* size not supported by the configuration (L > L_max, n < 0, ...) */
    AIF_ERR_OOM = -3,       /* device allocation failed, or no free user-state slot */
    AIF_ERR_CUDA = -4,      /* a CUDA runtime call failed; the runtime's error string is in aif_last_error */
    AIF_ERR_VERSION = -5,   /* user state was computed under other weights than the loaded ones */
    AIF_ERR_NOT_READY = -6, /* weights not loaded, or user state not computed */
    AIF_ERR_BAD_ID = -7,    /* (status bit only) candidate or refresh id outside [0, M) */
    AIF_ERR_TIMEOUT = -8    /* (status bit only) a bounded device-side wait ran out */
};

/* bits of the device status word */
enum { AIF_STATUS_BAD_ID = 1u, AIF_STATUS_TIMEOUT = 2u };

enum { AIF_F32 = 0, AIF_BF16 = 1 };
enum { AIF_BUCKET_MOD = 0, AIF_BUCKET_HASH = 1 };
enum { AIF_NORM_NONE = 0, AIF_NORM_MEAN = 1 };
enum { AIF_PATH_AUTO = 0, AIF_PATH_SIMT = 1, AIF_PATH_TENSOR = 2 };
enum { AIF_USER_RAW = 0, AIF_USER_PROJECTED = 1 };

/* Interaction blocks of the real-time model.  The first two are the base model; the last three are the
 * paper's approximations (Algorithm 1; eqs. 6-9). */
enum {
    AIF_BLK_ATT = 1,      /* dense target attention: softmax(e S^T / sqrt(d)) S (Section 4.2, first paragraph) */
    AIF_BLK_CROSS = 2,    /* cross features indexed from the user's pre-cache (Section 3.3) */
    AIF_BLK_BEA = 4,      /* v = w_hat V (Algorithm 1, line 4) */
    AIF_BLK_LSH_DIN = 8,  /* LSH similarity (eqs. 6-7) weighting the projected sequence (eq. 8) */
    AIF_BLK_SIMTIER = 16  /* histogram of LSH similarities over n_tiers tiers (eq. 9) */
};

typedef void *aif_stream;
typedef struct aif_ctx aif_ctx;
typedef struct aif_user_state aif_user_state;

/*
 * Model and table geometry.  The input of the scoring MLP is the concatenation, in this column order,
 *   [ u (d) | e (d) | att (d) | cross f=0..F-1 (F*dc) | v_bea (d) | lsh_din (d) | simtier (n_tiers) ]
 * with the columns of disabled blocks absent; aif_input_width returns the total.
 */
typedef struct {
    uint32_t struct_size;          /* sizeof(aif_config), checked */
    int32_t dtype;                 /* AIF_F32 | AIF_BF16 */
    int64_t M;                     /* rows of the item table, 0 < M < 2^31 */
    int32_t d;                     /* width of item and user vectors; multiple of 32; <= 256 */
    int32_t dU;                    /* width of the raw user embeddings of eq. 1; multiple of 4 */
    int32_t L_max;                 /* longest behaviour sequence a user state can hold */
    int32_t F, B, dc;              /* cross fields, buckets per field, width of one cross embedding (multiple of 8) */
    int32_t n_hidden;              /* 1..4 hidden layers (ReLU); the output layer is 1 wide */
    int32_t hidden[4];             /* widths, each a multiple of 8 and <= 1024 */
    int32_t bucket_mode;           /* AIF_BUCKET_MOD: id % B;  AIF_BUCKET_HASH: aif_mix64(id, f) % B */
    int32_t blocks;                /* mask of AIF_BLK_* */
    int32_t n_bridge;              /* n of Algorithm 1 (<= 16) */
    int32_t lsh_bits;              /* d' of eq. 5: signature bits, multiple of 32, <= 256 */
    int32_t n_tiers;               /* N of eq. 9 (<= 16): equal-width tiers over [0,1], the last one closed */
    int32_t lsh_din_norm;          /* AIF_NORM_NONE: eq. 8 as printed (a sum); AIF_NORM_MEAN: divided by L */
    int32_t simtier_norm;          /* AIF_NORM_NONE: raw counts; AIF_NORM_MEAN: counts divided by L */
    int32_t emit_sigmoid;          /* 0: logits; 1: sigmoid(logit) */
    int32_t max_user_states;       /* slots of the user-state arena (the paper sizes its pool at 2-3x the
                                      requests in flight, Section 5.3) */
    int32_t mini_batch;            /* candidates per mini-batch (Section 1: e.g. 1000); work tiles never
                                      straddle a mini-batch boundary; 0 = one batch per request */
    int32_t path;                  /* AIF_PATH_AUTO: tensor-core kernels when dtype and shapes allow, else
                                      the CUDA-core kernels; _SIMT / _TENSOR force one (TENSOR: AIF_ERR_SHAPE
                                      if unsupported) */
    int32_t n_categories;          /* 0: the sequence blocks (attention, LSH-DIN, SimTier) see the whole behaviour
                                      sequence.  1..4096: they see only the sub-sequence of the candidate's category
                                      (Section 3.3, SIM-hard: <user, category, sub-sequence>), see aif_category.  Needs
                                      the tensor-core kernels (AIF_ERR_SHAPE otherwise); mini_batch is then ignored
                                      (scores do not depend on it) */
    int32_t versioned_table;       /* 1: the item table (and its sidecars) exists twice.  A full refresh (ids == NULL) is
                                      written into the copy that is not being read and published as a whole: scoring
                                      calls made before the refresh call keep reading the old copy, calls made after it
                                      wait for the refresh and read the new one; no call ever sees a half-written table
                                      (Section 3.4: full updates of the index table under serving).  Costs the table's
                                      memory a second time.  0: one copy, the caller orders refreshes against scoring */
    int64_t max_batch_candidates;  /* upper bound of the candidates of one aif_score / aif_score_batch call;
                                      sizes the context's scratch memory */
} aif_config;

/* Device pointers to the weights, all in storage type unless stated.  Copied by aif_load_weights. */
typedef struct {
    uint32_t struct_size;
    const void *W[4];      /* W[k]: [hidden[k] x in_k]; in_0 = aif_input_width (full concatenation) */
    const float *b[4];     /* fp32 [hidden[k]] */
    const void *w_out;     /* [hidden[n_hidden-1]] */
    const float *b_out;    /* fp32 [1] */
    /* user-side network, eqs. 1-2; may all be NULL if only AIF_USER_PROJECTED states are used */
    const void *W_profile; /* [d x dU] */
    const void *W_seq;     /* [d x dU] */
    const void *W_a;       /* [d x d]   FFN(x) = ReLU(x W_a^T + b_a) W_b^T + b_b */
    const float *b_a;      /* fp32 [d] */
    const void *W_b;       /* [d x d] */
    const float *b_b;      /* fp32 [d] */
    /* user side of Algorithm 1 (steps 1-2); may be NULL when every caller supplies bea_V itself */
    const void *bridges;   /* B [n_bridge x d] */
    const void *W_f;       /* [d x d]: V_k = W_f (sum_j W_kj U_j), this library's reading of f(U, W | Theta_u) */
} aif_weights;

/* Device pointers to one user's inputs, storage type unless stated. */
typedef struct {
    uint32_t struct_size;
    int32_t mode;            /* AIF_USER_RAW: profile [dU] and seq [L x dU] are raw embeddings, eqs. 1-3 are
                                computed.  AIF_USER_PROJECTED: profile is the combined user vector u [d] and seq is
                                the projected sequence U^_seq [L x d] (a state computed elsewhere and shipped in). */
    const void *profile;
    const void *seq;
    const void *cross_raw;   /* [F x B x dc] user-side part of the cross features; NULL if block off */
    const void *bea_V;       /* [n_bridge x d] user-side BEA vectors (Algorithm 1, step 2), computed elsewhere; NULL if
                                the block is off or bea_U is given instead */
    const uint8_t *seq_sig;  /* [L x lsh_bits/8] packed signatures of the sequence items, first bit = MSB of
                                byte 0 (Section 4.2); NULL if both LSH blocks are off */
    const void *bea_U;       /* [bea_m x d] user-side feature embeddings U of Algorithm 1: with bea_V == NULL the call
                                computes W = Softmax(B U^T / sqrt(d)) and V from them (needs bridges and W_f) */
    const int32_t *seq_cat;  /* int32 [L]: category in [0, n_categories) of every sequence item, the parsed form of the
                                long-term sequence (Section 3.3); required iff n_categories > 0.  An entry outside the
                                range drops that item from every sub-sequence and sets AIF_STATUS_BAD_ID */
    int32_t bea_m;           /* 1 <= bea_m <= 1024 */
} aif_user_inputs;

typedef struct {
    uint64_t score_calls, candidates_scored, precompute_calls, refresh_calls, rows_refreshed;
    uint64_t bad_id_events, timeout_events;   /* accumulated from polled status words */
    int32_t user_states_in_use, user_states_high_water;
    uint64_t model_version, table_version;
    int64_t device_bytes;                     /* memory held by the context */
    int32_t tensor_path;                      /* 1 if aif_score runs the tensor-core kernels */
} aif_stats;

/* Width of the concatenated MLP input for a configuration (see aif_config). */
int aif_input_width(const aif_config *cfg);

/* The 64-bit mix behind AIF_BUCKET_HASH: the splitmix64 output function applied to
 * id * 0x9E3779B97F4A7C15 + field.  Host function; the kernels compute the same value. */
uint64_t aif_mix64(uint64_t id, uint64_t field);

/* Category of an item when n_categories > 0 (Section 3.3 selects sub-sequences by the candidate's category; like the
 * cross-feature attribute it is derived from the id here): id % n_categories (AIF_BUCKET_MOD) or
 * aif_mix64(id, AIF_CATEGORY_FIELD) % n_categories (AIF_BUCKET_HASH).  Host function; the kernels compute the same. */
#define AIF_CATEGORY_FIELD 3239
int64_t aif_category(int64_t id, int32_t n_categories, int32_t bucket_mode);

/* Creates a context on the current CUDA device: allocates the item table (M x d, plus M x n_bridge BEA
 * weights and M x lsh_bits/8 signature bytes when those blocks are on), the user-state arena, the status
 * word and scratch memory.  The table starts zeroed.  cfg: host.  Synchronises the device once. */
int aif_create(const aif_config *cfg, aif_ctx **out);

/* Frees everything the context owns.  Synchronises the device.  User-state handles die with it. */
int aif_destroy(aif_ctx *ctx);

/* Copies the weights in (device to device, on `stream`), derives the layouts the kernels want, and bumps
 * model_version: user states computed earlier are refused by aif_score with AIF_ERR_VERSION, which is the
 * version-consistency rule of Section 3.4.  w: host struct of device pointers. */
int aif_load_weights(aif_ctx *ctx, const aif_weights *w, aif_stream stream);

/* Item side, nearline (eq. 4 produces `rows` upstream; Section 3.4 asks for full and incremental updates).
 * ids == NULL: full refresh, rows i -> table row i for i < n (n <= M).  Otherwise incremental: rows i ->
 * table row ids[i]; an id outside [0, M) is skipped and sets AIF_STATUS_BAD_ID.  Duplicate ids in one call
 * leave either row.  ids: device int32 [n].  rows: device [n x d] storage type.  bea_w: device [n x n_bridge]
 * storage type, lsh_sig: device [n x lsh_bits/8]; required iff their blocks are on.  Bumps table_version.
 * The caller orders the call against scoring (same stream, or an event).
 * With versioned_table a full refresh needs no such ordering: it fills the spare copy (rows beyond n are carried over
 * from the live one) on `stream` and becomes the live copy for every scoring call made after this call returns; those
 * calls wait on the device for the refresh to finish.  The copy it overwrites is the one that was live before the
 * previous full refresh: scoring calls made before that previous refresh must have finished by now.  Incremental
 * refreshes write into the live copy and are ordered by the caller as before. */
int aif_item_nearline_refresh(aif_ctx *ctx, const int32_t *ids, int64_t n, const void *rows, const void *bea_w,
                              const uint8_t *lsh_sig, aif_stream stream);

/* Weights of the item side of the nearline pipeline.  Device pointers, storage type unless noted; copied in by
 * aif_load_item_weights.
 *   eq. 4 (Section 3.2) "dimensionality reduction": I^ = W_i1 ReLU(W_i0 I + b_i0) + b_i1, widths dI -> hI -> d (the
 *     paper says "a multi-layer perceptron" and no more; one ReLU hidden layer and a linear output is this library's reading)
 *   Algorithm 1 step 3: w^ = Softmax(I_id B^T / sqrt(d)): `bridges` = B [n_bridge x d] (needed iff the BEA block is on)
 *   eq. 5 (Section 4.2): signature bits = [M W_hash^T > 0]: `W_hash` [lsh_bits x d_mm] (needed iff an LSH block is on) */
typedef struct {
    uint32_t struct_size;
    int32_t dI, hI, d_mm;
    const void *W_i0;     /* [hI x dI] */
    const float *b_i0;    /* [hI] fp32 */
    const void *W_i1;     /* [d x hI] */
    const float *b_i1;    /* [d] fp32 */
    const void *bridges;  /* [n_bridge x d] or NULL */
    const void *W_hash;   /* [lsh_bits x d_mm] or NULL */
} aif_item_weights;

/* Copies the item-side weights in (device to device, on `stream`) and sizes the scratch of
 * aif_item_nearline_compute.  Does not touch model_version: cached user states do not depend on these weights.
 * Errors: AIF_ERR_ARG (NULL, struct_size), AIF_ERR_SHAPE (widths < 1, not multiples of 4), AIF_ERR_OOM. */
int aif_load_item_weights(aif_ctx *ctx, const aif_item_weights *w, aif_stream stream);

/* Item side, nearline, as a compute call (Section 3.2: the nearline job that fills the item table for every candidate,
 * run again whenever the model or the features change; Section 3.4: full and incremental updates): from raw item
 * features to the table rows that aif_item_nearline_refresh would have been handed.
 *   I_raw  device [n x dI] storage type: concatenated item embeddings; gives the item vectors I^ (eq. 4)
 *   I_id   device [n x d] storage type or NULL: item id embeddings for the BEA weights (Algorithm 1 step 3); NULL: the
 *          freshly computed I^ takes their place.  Read only when the BEA block is on.
 *   M_mm   device [n x d_mm] storage type: multi-modal embeddings for the signatures (eq. 5); required iff an LSH block is on
 * ids == NULL: rows i -> table row i (n <= M); otherwise rows i -> table row ids[i] with the rules of
 * aif_item_nearline_refresh.  Bumps table_version.  Needs aif_load_item_weights first (AIF_ERR_NOT_READY).
 * On bf16 contexts whose widths are multiples of 64 the two layers and the hash projections run on the tensor cores;
 * a signature bit whose projection is within rounding of zero may then differ from an evaluation in another order. */
int aif_item_nearline_compute(aif_ctx *ctx, const int32_t *ids, int64_t n, const void *I_raw, const void *I_id,
                              const void *M_mm, aif_stream stream);

/* User side, online-asynchronous (Section 3.1 eqs. 1-3, Section 3.3 "User-Side Pre-Processing").  Takes a free
 * slot of the arena and fills it on `side_stream`: u, S = U^_seq [L x d], the cross pre-cache T, V, the
 * sequence signatures, and p_u = W1[:, user columns] u + b1 (fp32), so that the real-time phase never touches
 * the user columns of the first layer again.  With categories on it also lays the projected sequence (and its
 * signatures) out a second time grouped by category, every sub-sequence padded with zero rows to a multiple of 128:
 * this is the pre-cache of parsed sub-sequences for all of the user's categories that Section 3.3 builds in parallel
 * with retrieval.  Records a "ready" event that aif_score waits on.
 * in: host struct of device pointers; the inputs must stay valid until the work on side_stream is done.
 * request_key: the caller's request identity (Section 3.4 keys the cached state by request), kept in the handle.
 * Calls with AIF_USER_RAW inputs share scratch of the context (the attention rows of eq. 2): issue them on one side
 * stream, or order them with events, so that two of them never run on the GPU at the same time.
 * Errors: AIF_ERR_SHAPE (L < 1 or L > L_max), AIF_ERR_OOM (no free slot), AIF_ERR_NOT_READY (no weights). */
int aif_user_precompute(aif_ctx *ctx, uint64_t request_key, const aif_user_inputs *in, int32_t L,
                        aif_user_state **out, aif_stream side_stream);

/* Returns the slot to the arena.  The caller makes sure no scoring work that uses it is still in flight. */
int aif_user_release(aif_ctx *ctx, aif_user_state *state);

/* Key given to aif_user_precompute (host query, no device work). */
uint64_t aif_user_request_key(const aif_user_state *state);

/* Copies parts of a user state to caller memory for inspection (tests, transport): any of u_out (device fp32
 * [d]), S_out (device, storage type [L x d]) and pu_out (device fp32 [hidden[0]]) may be NULL. */
int aif_user_state_export(aif_ctx *ctx, const aif_user_state *state, float *u_out, void *S_out, float *pu_out,
                          aif_stream stream);

/* Real-time phase: scores n candidates of one request.  cand_ids: device int32 [n]; logits: device fp32 [n]
 * (sigmoid outputs when emit_sigmoid).  `stream` first waits for the state's ready event.  May be called once
 * per request or once per mini-batch; the result of a candidate does not depend on which.  n = 0 is a no-op.
 * An id outside [0, M) gives NaN and sets AIF_STATUS_BAD_ID.  No host-device copy happens inside.
 * Errors: AIF_ERR_VERSION, AIF_ERR_NOT_READY, AIF_ERR_SHAPE (n > max_batch_candidates), AIF_ERR_ARG. */
int aif_score(aif_ctx *ctx, const aif_user_state *state, const int32_t *cand_ids, int32_t n, float *logits,
              aif_stream stream);

/* Many requests in one launch.  states: host array [n_req]; offsets: host int64 [n_req + 1], ascending, request
 * r owns cand_ids[offsets[r] .. offsets[r+1]) and the same range of logits (both device).  The small request
 * table is staged through pinned memory owned by the context (one asynchronous copy per call).
 * Errors: AIF_ERR_SHAPE also when the launch needs more 128-candidate tiles than the context's tile table holds (it is
 * sized from max_batch_candidates, mini_batch and max_user_states, so only a call beyond those limits can get there). */
int aif_score_batch(aif_ctx *ctx, int32_t n_req, const aif_user_state *const *states, const int32_t *cand_ids,
                    const int64_t *offsets, float *logits, aif_stream stream);

/* aif_score for callers whose buffers live in host memory: brings host_ids (host) to the device, scores, leaves the
 * logits in host_logits (host), all on `stream`; returns after the stream has drained.  If both buffers are page-locked
 * and mapped into the device's address space (cudaHostAlloc / cudaHostRegister; pinned torch tensors are), a small
 * kernel reads the ids across the bus and the last scoring kernel writes the logits straight into host_logits;
 * otherwise both are staged with cudaMemcpyAsync through buffers of the context.  This is the end-to-end form the
 * benchmark times. */
int aif_score_host(aif_ctx *ctx, const aif_user_state *state, const int32_t *host_ids, int32_t n,
                   float *host_logits, aif_stream stream);

/* aif_score_batch for callers whose buffers live in host memory (Section 3.1: the real-time phase is handed candidate ids
 * by the retrieval service and hands scores back to it): host_ids (host int32, all requests concatenated) are copied to the
 * device on `stream`, scored in one launch, and the logits copied back into host_logits (host fp32); returns after the
 * stream has drained.  Page-locked buffers make both copies asynchronous transfers of the copy engine; pageable ones are
 * staged by the runtime.  states, offsets: as for aif_score_batch.  Errors as for aif_score_batch. */
int aif_score_batch_host(aif_ctx *ctx, int32_t n_req, const aif_user_state *const *states, const int32_t *host_ids,
                         const int64_t *offsets, float *host_logits, aif_stream stream);

/* Scoring for callers that cannot allocate device memory.  (The paper has no counterpart to this call; it exists
 * for deployment reasons only.)  Some hosts of this library never get to call cudaMalloc after start-up: a plug-in
 * inside a serving process whose memory pool has already claimed the whole GPU, or a request thread that is not
 * allowed to enter the driver's allocator because an allocation can stall every stream of the device.  A context
 * normally keeps the activations that pass between its scoring kernels in memory it allocated in aif_create, sized
 * by max_batch_candidates.  This call runs the same tensor-core kernel chain as aif_score but keeps those
 * activations in a fixed array that is part of the library image instead, so it allocates nothing and does not
 * depend on max_batch_candidates.  It calls no cudaMalloc, cudaFree or other allocating routine.
 *
 * Limits: n <= AIF_NOALLOC_MAX_CANDIDATES, and the model's activations (dense interaction columns plus all hidden
 * layers but the last, 2 bytes each) must fit AIF_NOALLOC_ROW_BYTES per candidate; beyond either the call returns
 * AIF_ERR_SHAPE and aif_last_error says which.  It also returns AIF_ERR_SHAPE on a context that runs the CUDA-core
 * kernel (fp32 storage or unsupported shapes): that kernel has no scratch, use aif_score.  The array costs
 * (AIF_NOALLOC_MAX_CANDIDATES + 128) * AIF_NOALLOC_ROW_BYTES = 4.5 MiB on every GPU that loads the library, until
 * the process exits.
 *
 * The first call on each device looks up the array's device address (once, with that device current); make that
 * first call before any stream capture begins.  All calls on a device share the one array, and it keeps whatever the
 * previous call left there: every element a call reads it has written itself earlier in the same call, so nothing
 * needs clearing, but two calls that overlap on the GPU (different streams, or different contexts) race on it.
 * Order them on one stream or with events.  Arguments and results are those of aif_score. */
#define AIF_NOALLOC_MAX_CANDIDATES 1024
#define AIF_NOALLOC_ROW_BYTES 4096
int aif_score_noalloc(aif_ctx *ctx, const aif_user_state *state, const int32_t *cand_ids, int32_t n, float *logits,
                      aif_stream stream);

/* The gather stage alone (Section 1, "indexing the model embedding matrices"): rows_out[i] = table[ids[i]].
 * ids: device int32 [n]; rows_out: device [n x d] storage type.  Bad ids give zero rows and the status bit.
 * Exists so that the gather can be measured against HBM bandwidth by itself. */
int aif_gather_rows(aif_ctx *ctx, const int32_t *ids, int64_t n, void *rows_out, aif_stream stream);

/* The same for the sidecars that nearline updates write beside the item vectors: bea_w_out[i] = the BEA weight row
 * (device [n x n_bridge] storage type), sig_out[i] = the signature (device [n x lsh_bits/8]) of item ids[i]; a NULL
 * output is skipped, an output whose block is off is AIF_ERR_ARG.  Bad ids give zero rows and the status bit. */
int aif_gather_sidecars(aif_ctx *ctx, const int32_t *ids, int64_t n, void *bea_w_out, uint8_t *sig_out, aif_stream stream);

/* Copies the user-side BEA vectors V [n_bridge x d] (storage type) of a state to V_out (device), ordered after the
 * state's user-side call.  AIF_ERR_ARG when the BEA block is off. */
int aif_user_state_export_bea(aif_ctx *ctx, const aif_user_state *state, void *V_out, aif_stream stream);

/* Reads and clears the device status word (synchronises the device).  bits: host. */
int aif_poll_status(aif_ctx *ctx, uint32_t *bits);

int aif_get_stats(aif_ctx *ctx, aif_stats *out);

/* Per-kernel timing of scoring calls, for roofline measurements.  While on, every scoring call brackets each of
 * its kernels with CUDA events on the call's stream (a few microseconds of overhead per kernel, so leave it off
 * for throughput runs).  aif_get_kernel_timing synchronises on the last scoring call and returns, for that call,
 * the number of kernels (<= 8), their names (static strings) and their durations in milliseconds.
 * names / ms: host arrays of 8 entries. */
int aif_set_kernel_timing(aif_ctx *ctx, int on);
int aif_get_kernel_timing(aif_ctx *ctx, int32_t *n, const char **names, float *ms);

/* Self-test of the failure path of the device-side waits (Section 3.4's consistency requirement is enforced on the
 * host; this is its device-side companion).  Every wait inside the tensor-core kernels is bounded: when a producer
 * never delivers, the waiting thread gives up after a fixed number of clock cycles, the kernel sets AIF_STATUS_TIMEOUT
 * and returns normally.  This call launches one tiny kernel on `stream` whose single wait can never be satisfied and
 * whose bound is limit_cycles (1 .. 2e9 SM clock cycles); afterwards aif_poll_status reports AIF_STATUS_TIMEOUT and the
 * context remains fully usable.  Nothing faults, traps or hangs. */
int aif_selftest_bounded_wait(aif_ctx *ctx, int64_t limit_cycles, aif_stream stream);

/* Number of kernels this library has launched in this process (all contexts). */
uint64_t aif_kernel_launches(void);

const char *aif_strerror(int code);

/* Text of the last CUDA runtime error seen by this thread's most recent failing call ("" if none). */
const char *aif_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* AIF_H_ */
