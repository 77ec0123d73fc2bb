// Internal declarations of libaif: context layout, device-side descriptors, kernel launchers.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <vector>

#include "../../include/aif.h"

namespace aif {

constexpr int kMaxHidden = 4;
constexpr int kSimtTile = 8;        // candidates per block in the CUDA-core scoring kernel
constexpr int kSimtThreads = 256;
constexpr int kTcTile = 128;        // candidates per tile in the tensor-core kernels (UMMA M)

// One user-state slot as the kernels see it.  Pointers are fixed when the arena is laid out; only L changes.
struct SlotDev {
    const void *u;          // [d] storage type
    const float *u32;       // [d] fp32
    const void *S;          // [L x d] storage type: projected behaviour sequence
    const void *T;          // [F x B x dc] storage type: cross pre-cache
    const void *V;          // [n_bridge x d] storage type
    const uint8_t *sigS;    // [L x lsh_bits/8]
    const uint8_t *sigE;    // [L x lsh_bits] the same signatures with one E4M3 byte per bit, +1.0 / -1.0 (tensor-core LSH), or nullptr
    const float *p_u;       // [H1] fp32: W1[:, user columns] u + b1
    const void *pu_hl;      // [2][H1] bf16: p_u split into high parts and remainders (bias operand of the tensor cores)
    // categories on: the sequence a second time, grouped by category, every sub-sequence padded with zero rows to a multiple
    // of 128 (the pre-cache of parsed sub-sequences, Section 3.3)
    const void *Sg;         // [Lg x d] storage type, Lg = grouped_rows(L_max, n_categories)
    const uint8_t *sigEg;   // [Lg x lsh_bits] +-1 bytes, or nullptr
    const int32_t *cat_off; // [n_categories] first row of every sub-sequence in Sg
    const int32_t *cat_len; // [n_categories] items of every sub-sequence
    const float *k_norm;    // largest Euclidean norm of a row of S (set with the slot; NaN or inf rows make it so)
    int32_t L;
    int32_t pad_;
};

// One request of a scoring launch.
struct ReqDev {
    int32_t slot;
    int32_t n;            // candidates
    int64_t off;          // first candidate in ids / logits
    int32_t tile_begin;   // first tile of this request in the launch
    int32_t pad_;
};

struct ModelDev {
    int32_t d, F, B, dc, n_hidden, hidden[kMaxHidden];
    int32_t bucket_mode, blocks, n_bridge, lsh_bits, n_tiers, lsh_din_norm, simtier_norm, emit_sigmoid;
    int32_t k1;           // candidate-dependent input columns = input width - d
    int32_t mini_batch;
    int64_t M;
    const void *E;
    const void *bea_w;
    const uint8_t *sig;
    const void *Wt[kMaxHidden];   // transposed weights [in x out] storage type; Wt[0] = full first layer incl. user rows
    const float *b[kMaxHidden];
    const void *w_out;
    const float *b_out;
};

// One 128-candidate tile of a launch over several requests, looked up once per launch (k_tile_table) so that no kernel
// role has to search the request table per tile.
struct TileDev {
    int32_t slot;
    int32_t cnt;     // candidates in the tile
    int64_t pos0;    // position of its first candidate in ids / logits
    int32_t L;       // keys of the tile: the request's sequence length, or the length of its category's sub-sequence
    int32_t key0;    // first key row (0, or where the category's sub-sequence begins in the grouped sequence)
    int32_t pad_[2];
};

struct ScoreLaunch {
    const SlotDev *slots;   // device array of all slots
    const ReqDev *reqs;     // device array [n_req], or nullptr: use `single`
    ReqDev single;
    int32_t n_req;
    int32_t n_tiles;
    int64_t total;          // candidates of the launch
    int32_t max_L;          // longest behaviour sequence among the launch's requests (host-side hint)
    const int32_t *ids;
    float *logits;
    uint32_t *status;
    const TileDev *tiles;   // [n_tiles] (tensor-core tiles), or nullptr: search `reqs` per tile
    // categories on: tiles are formed on the device from the candidates grouped by (request, category).  n_tiles above is
    // then an upper bound that sizes grids, the count is read from n_tiles_dev; ids are the grouped candidates, and
    // out_index[p] is where the logit of grouped position p belongs in the caller's array.
    const int32_t *n_tiles_dev;
    const int32_t *out_index;
    int32_t grouped;        // 1: key blocks come from the grouped sequence
};

struct HostSlot {
    bool in_use = false;
    bool ready = false;
    int32_t L = 0;
    uint64_t key = 0;
    uint64_t model_version = 0;
    cudaEvent_t ev = nullptr;
    mutable bool ev_seen_done = false;   // the user-side call that recorded `ev` is known to have completed
    SlotDev dev{};
    // scratch for the user-side network
    float *prof_hat = nullptr;   // [d]
    float *partial = nullptr;    // [kUserPartials x d]
    float *ppart = nullptr;      // [kProfParts x (d + 2)]: per key slice, unnormalised attention row, maximum, sum
    int32_t *cat_map = nullptr;  // [L_max]: row of every sequence item in the grouped sequence (scratch of the grouping)
    int32_t *cat_hist = nullptr; // [ceil(L_max / 1024) x n_categories]: per 1024-item block, items of every category
};

constexpr int kUserPartials = 1184;
constexpr int kProfParts = 256;      // warps (key slices) of the profile-attention launch   // warps of the self-attention launch (148 SMs x 8)

// Optional per-kernel timing of the last scoring call (events on the call's stream).
struct KernelTiming {
    static constexpr int kMax = 8;
    bool on = false;
    int n = 0;
    cudaEvent_t ev[kMax + 1] = {};
    const char *names[kMax] = {};
};

struct PinnedRing {
    static constexpr int kSlots = 8;
    ReqDev *host[kSlots] = {};
    ReqDev *dev[kSlots] = {};
    cudaEvent_t ev[kSlots] = {};
    bool used[kSlots] = {};
    int next = 0;
    int capacity = 0;   // requests per slot
};

}  // namespace aif

struct aif_user_state {
    aif_ctx *ctx;
    int32_t index;
};

struct aif_ctx {
    aif_config cfg;
    int device = 0;
    size_t el = 4;
    int input_width = 0;
    bool weights_loaded = false;
    bool tensor_path = false;
    uint64_t model_version = 0, table_version = 0;
    int64_t device_bytes = 0;

    void *E = nullptr;          // the live copy of the item table and its sidecars: what every reader takes at call time
    void *bea_w = nullptr;
    uint8_t *sig = nullptr;
    void *E_alt = nullptr;      // versioned_table: the spare copy, target of the next full refresh
    void *bea_w_alt = nullptr;
    uint8_t *sig_alt = nullptr;
    // largest Euclidean norm of an item vector ever written to the table (device, only raised): with the slot's k_norm a
    // bound on every attention score of a request, which lets the attention kernel drop its running maximum
    float *e_norm = nullptr;
    cudaEvent_t table_ev = nullptr;   // end of the last full refresh of a versioned table
    mutable bool table_ev_pending = false;

    // weights
    void *Wt[aif::kMaxHidden] = {};      // [in x out]
    void *Wk[aif::kMaxHidden] = {};      // [out x in] (K-major), first layer: candidate-dependent columns only, K padded
    float *b[aif::kMaxHidden] = {};
    void *w_out = nullptr;
    float *b_out = nullptr;
    void *Wprofile_t = nullptr, *Wseq_t = nullptr, *Wa_t = nullptr, *Wb_t = nullptr;
    void *Wseq_k = nullptr, *Wa_k = nullptr;   // W_seq [d x dU], W_a [d x d] as given (K-major): operands of the tensor-core user side
    float *zero_bias = nullptr;                // [256] zeros
    void *ffn_rows = nullptr;                  // [L_max + 128][d] bf16: hidden FFN activations of the user state being computed
    float *b_a = nullptr, *b_b = nullptr;
    bool user_weights = false;
    void *bridges = nullptr, *W_f = nullptr;   // user side of Algorithm 1: B [n_bridge x d], W_f [d x d]
    bool bea_user_weights = false;

    char *arena = nullptr;
    size_t slot_bytes = 0;
    aif::SlotDev *slots_dev = nullptr;
    std::vector<aif::HostSlot> slots;
    std::vector<aif_user_state> handles;
    uint32_t *status = nullptr;

    // scratch owned by the context
    int32_t *ids_stage = nullptr;     // device staging of host ids (aif_score_host)
    float *logits_stage = nullptr;
    void *tc_plan = nullptr;          // tensor-core path: packed weights, tensor maps, activation scratch
    void *tc_att_plan = nullptr;      // tensor-core attention: tensor map over the arena's S regions
    void *nearline_plan = nullptr;    // item-side weights and scratch of aif_item_nearline_compute
    void *tc_fused_plan = nullptr;    // single-launch scoring: the second layer's bias split into two bf16 rows
    void *tc_lsh_plan = nullptr;      // tensor-core LSH blocks: tensor maps over the arena's S and +-1 signature regions
    void *sim_plan = nullptr;         // categories on: scratch of the grouping passes (aif_sim.cu)
    size_t grouped_rows = 0;          // rows of a slot's grouped sequence
    aif::PinnedRing ring;

    aif_stats stats{};
    mutable aif::KernelTiming timing;
    std::vector<void *> allocations;
};

namespace aif {

extern std::atomic<uint64_t> g_launches;
inline void count_launch(int n = 1) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }

// A named host-side range (NVTX) around the launches of a stage or of an entry point: a timeline tool shows the kernels under
// the stage's name.  With no tool attached a range costs two calls through an empty hook.
struct StageRange {
    explicit StageRange(const char *name);
    ~StageRange();
    StageRange(const StageRange &) = delete;
    StageRange &operator=(const StageRange &) = delete;
};

// Timing marks: begin(st) before the first kernel of a scoring call, mark(name, st) after each kernel.
void timing_begin(const aif_ctx *ctx, cudaStream_t st);
void timing_mark(const aif_ctx *ctx, const char *name, cudaStream_t st);

ModelDev make_model(const aif_ctx *ctx);

// aif_simt.cu
cudaError_t launch_scatter_rows(const aif_ctx *ctx, const int32_t *ids, int64_t n, const void *rows, const void *bea_w,
                                const uint8_t *sig, cudaStream_t st);
// *out = max(*out, largest row norm) over rows ids[0..n) of `rows` (ids == nullptr: rows 0..n); ids outside [0, M) skipped
cudaError_t launch_row_norm_max(const aif_ctx *ctx, const void *rows, const int32_t *ids, int64_t n, int64_t M, float *out, cudaStream_t st);
cudaError_t launch_stage_ids(const int32_t *mapped_src, int32_t *dst, int n, cudaStream_t st);
cudaError_t launch_gather_rows(const aif_ctx *ctx, const int32_t *ids, int64_t n, void *out, cudaStream_t st);
cudaError_t launch_gather_sidecars(const aif_ctx *ctx, const int32_t *ids, int64_t n, void *bea_w_out, uint8_t *sig_out, cudaStream_t st);
cudaError_t launch_transpose(const void *in, void *out, int rows, int cols, size_t el, cudaStream_t st);
cudaError_t launch_score_simt(const aif_ctx *ctx, const ScoreLaunch &sl, cudaStream_t st);
cudaError_t launch_user_network(const aif_ctx *ctx, HostSlot &hs, int slot_index, const aif_user_inputs *in, int L,
                                cudaStream_t st);
int simt_tiles_for(const aif_ctx *ctx, int n);

// tensor-core path (aif_tc.cu)
bool tc_supported(const aif_config &cfg);
cudaError_t tc_prepare_context(aif_ctx *ctx);
void tc_destroy_context(aif_ctx *ctx);
// tensor-core attention (aif_tc_att.cu)
bool tc_att_supported(const aif_config &cfg);
cudaError_t tc_att_prepare(aif_ctx *ctx);
void tc_att_destroy(aif_ctx *ctx);
// eq. 2's attention rows softmax(S S^T / sqrt(d)) S of one user state with the same kernel (queries = the sequence rows);
// *rows_out: [L x d] bf16 in scratch of the attention plan, valid until the next call
cudaError_t launch_self_att_tc(const aif_ctx *ctx, int slot_index, int L, cudaStream_t st, const void **rows_out);
cudaError_t launch_att_tc(const aif_ctx *ctx, const ScoreLaunch &sl, cudaStream_t st, void *X, int x_stride, size_t x_rows);
// LSH similarity, LSH-DIN and SimTier on the tensor cores (aif_tc_lsh.cu)
bool tc_lsh_supported(const aif_config &cfg);
cudaError_t tc_lsh_prepare(aif_ctx *ctx);
void tc_lsh_destroy(aif_ctx *ctx);
cudaError_t launch_expand_signatures(const aif_ctx *ctx, const uint8_t *sig, int L, uint8_t *out, cudaStream_t st);
cudaError_t launch_lsh_tc(const aif_ctx *ctx, const ScoreLaunch &sl, cudaStream_t st, void *X, int x_stride, size_t x_rows, int x_din,
                          int x_tier);
// category sub-sequences (aif_sim.cu): the user-side grouping of a sequence, and the grouping of a launch's candidates by
// (request, category) into tiles
size_t sim_grouped_rows(int L_max, int n_categories);
cudaError_t sim_prepare(aif_ctx *ctx);
void sim_destroy(aif_ctx *ctx);
size_t sim_tile_capacity(const aif_ctx *ctx);
cudaError_t sim_group_sequence(const aif_ctx *ctx, HostSlot &hs, const int32_t *seq_cat, int L, cudaStream_t st);
// fills sl (ids, tiles, n_tiles upper bound, n_tiles_dev, out_index) for a launch whose original ids are sl.ids
cudaError_t sim_group_candidates(const aif_ctx *ctx, ScoreLaunch &sl, cudaStream_t st);
// whole scoring pass of a tile in one CTA (aif_tc_fused.cu); the tensor maps it shares with the other kernels
bool tc_fused_supported(const aif_config &cfg);
cudaError_t tc_fused_prepare(aif_ctx *ctx);
cudaError_t tc_fused_prepare_weights(aif_ctx *ctx, cudaStream_t st);
cudaError_t launch_request_fused(const aif_ctx *ctx, const ScoreLaunch &sl, cudaStream_t st);
const void *tc_weight_tmap(const aif_ctx *ctx, int k);   // CUtensorMap over the packed weights of hidden layer k
const void *tc_att_tmap(const aif_ctx *ctx);             // CUtensorMap over the S regions of the user-state arena
cudaError_t tc_prepare_weights(aif_ctx *ctx, const aif_weights *w, cudaStream_t st);
cudaError_t launch_score_tc(const aif_ctx *ctx, const ScoreLaunch &sl, int64_t total_candidates, cudaStream_t st);
// The same kernel chain with its intermediate activations in caller-chosen memory.
struct TcScratch {
    void *X;               // dense interaction columns, [rows x x_cols] bf16
    void *H[kMaxHidden];   // activations after hidden layer k (k < last), [rows x hidden[k]] bf16
    void *xb;              // cross-feature buckets, [rows x F] uint16
    void *tiles;           // tile table, [rows / 128 + requests] TileDev, or nullptr
    size_t rows;           // rows every array has room for
};
size_t tc_scratch_row_bytes(const aif_ctx *ctx);
void tc_scratch_layout(const aif_ctx *ctx, void *base, size_t rows, TcScratch *out);
cudaError_t launch_score_tc_scratch(const aif_ctx *ctx, const ScoreLaunch &sl, cudaStream_t st, const TcScratch &sc);
// One dense layer on the tensor cores (aif_tc.cu): out [rows x H] bf16 = act(A [rows x in_w] W^T + bias), or, with
// sign_bits, out [rows x H / 8] bytes = packed signs of A W^T.  in_w a multiple of 64; H <= 256 and a multiple of 32, or a
// multiple of 256.  W [H x in_w] bf16 row-major.
struct DenseLayer {
    const void *A;
    const void *W;
    const float *bias;   // [H]
    void *out;
    int32_t in_w, H;
    int32_t relu;        // 0: linear output
    int32_t sign_bits;
};
cudaError_t tc_dense_layer(const aif_ctx *ctx, const DenseLayer &L, int64_t rows, cudaStream_t st);
// the item-side tower in one kernel, hidden activations in tensor memory (aif_tc_tower.cu)
bool tc_tower_supported(int dI, int hI, int d);
cudaError_t tc_tower_prepare();
// norm_max (device, may be null): raised to an upper bound of the largest Euclidean norm of an output row
cudaError_t launch_item_tower_tc(const aif_ctx *ctx, const void *I_raw, const void *W0, const float *b0, const void *W1, const float *b1,
                                 void *out, int64_t n, int dI, int hI, float *norm_max, cudaStream_t st);
// item side of the nearline pipeline (aif_nearline.cu)
int nearline_load_weights(aif_ctx *ctx, const aif_item_weights *w, cudaStream_t st);
int nearline_compute(aif_ctx *ctx, const int32_t *ids, int64_t n, const void *I_raw, const void *I_id, const void *M_mm,
                     cudaStream_t st);
void nearline_destroy(aif_ctx *ctx);
// host-side checks shared by the scoring entry points (aif_api.cu)
int check_user_state(aif_ctx *ctx, const aif_user_state *st);
cudaError_t wait_table_ready(const aif_ctx *ctx, cudaStream_t st);   // orders st behind the last full refresh of a versioned table
void set_last_error(const char *text);
int tc_tiles_for(const aif_ctx *ctx, int n);
size_t tc_tile_capacity(const aif_ctx *ctx);   // entries of the context's tile table (launches over several requests)
cudaError_t launch_wait_selftest(const aif_ctx *ctx, long long limit_cycles, cudaStream_t st);

}  // namespace aif
