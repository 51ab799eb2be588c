/*
 * dasc.h -- C ABI of the B200 (sm_100a) implementation of the data-parallel
 * hot path of Decay-Aware State Compression (DASC): the compress / restore
 * cycle of linear-attention recurrent-state checkpoints in a prefix cache.
 *
 *   dasc_plan     host   static selection plan          (Section 3.3, 4.1, Eq. 2/3/6/7, App. B)
 *   dasc_pack     device retained units -> ragged pool  (Store path, Section 4.1, App. B Scheme 2)
 *   dasc_restore  device pool -> dense state, zero-fill (Load path, zero-fill policy, Section 4.2)
 *   dasc_refresh  device replay of the gated delta rule (Eq. 1; suffix-refresh policy, Section 4.2)
 *   dasc_pack_int8 / dasc_restore_int8
 *                 device the same copies with the INT8 checkpoint codec fused in (Appendix D, Eq. 10)
 *
 * Conventions
 *   - No exception crosses this boundary; every call returns a dasc_status_t.
 *   - "HOST" / "DEVICE" on a pointer says where the memory lives.  All device
 *     buffers are owned by the caller; the library owns only the plan object
 *     and the small index tables it uploads once in dasc_plan.
 *   - Device calls are asynchronous on `cuda_stream` (a cudaStream_t passed as
 *     void*; NULL = the legacy default stream), never synchronise, never
 *     allocate, and may be issued concurrently on several streams against one
 *     plan (a plan is immutable after creation).
 *   - Argument errors are detected on the host before any launch and leave
 *     the outputs untouched.
 *   - Device calls must be made with the plan's device current (cudaSetDevice);
 *     any other current device is refused with DASC_ERR_INVALID_ARG, because the
 *     plan's index tables live on that device.
 *   - State orientation: the paper writes the recurrent state as S in
 *     R^{d_v x d_k} with o = S q (Section 3.1).  This library stores the
 *     transpose, S[head][d_k][d_v], fp32, row-major, so that one KDA key
 *     channel S_{h,:,k} (the KDA selection unit of Section 4.1) is one
 *     contiguous row of d_v floats.  A dense state is addressed as
 *         state_base + req*req_stride + layer*layer_stride
 *                    + ((head*d_k + k)*d_v + v)            [floats]
 *     so both layer-major and request-major active-state pools work.
 *   - Selection units (Section 4.1): KDA -> one (head, key channel) row of
 *     d_v floats; GDN -> one complete value-head state of d_k*d_v floats.
 *     Unit index inside a layer: u = head*d_k + k (KDA), u = head (GDN).
 *   - Checkpoint pool (Appendix B, ragged layout): slot s holds, for layers
 *     in ascending order, the retained units of that layer in ascending unit
 *     index; layer l occupies units [o_l, o_{l+1}) with o_0 = 0 and
 *     o_{l+1} = o_l + r_l.  Slot s starts at pool_base + s*slot_stride floats.
 */
#ifndef DASC_H_
#define DASC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  DASC_OK = 0,
  DASC_ERR_INVALID_ARG = 1, /* null pointer, negative size, misaligned pointer or stride */
  DASC_ERR_SHAPE = 2,       /* shape outside what the kernels support */
  DASC_ERR_UNSUPPORTED = 3, /* valid request that this build does not implement */
  DASC_ERR_ALLOC = 4,       /* host or device allocation failed (dasc_plan only) */
  DASC_ERR_CUDA = 5,        /* a CUDA runtime call or launch failed */
  DASC_ERR_WORKSPACE = 6,   /* workspace missing, misaligned or too small */
  DASC_ERR_TIMEOUT = 7,     /* a bounded device-side wait ran out (reported by dasc_refresh_status) */
  DASC_ERR_DOMAIN = 8       /* log-decay outside the chunked kernel's range (reported by dasc_refresh_status) */
} dasc_status_t;

typedef enum { DASC_KDA = 0, DASC_GDN = 1 } dasc_kind_t;
typedef enum {
  DASC_SEL_THRESHOLD = 0, /* retained iff H_s > w_max, strictly (Section 4.1) */
  DASC_SEL_TOP_RATIO = 1, /* keep the ceil(keep_ratio*n) longest-horizon units of each scope group */
  DASC_SEL_EXPLICIT = 2   /* caller-supplied mask */
} dasc_sel_t;
typedef enum { DASC_SCOPE_HEAD = 0, DASC_SCOPE_LAYER = 1, DASC_SCOPE_MODEL = 2 } dasc_scope_t;
typedef enum { DASC_IO_BF16 = 0, DASC_IO_FP32 = 1 } dasc_io_dtype_t;
typedef enum {
  DASC_REFRESH_CONTINUE = 0,           /* start from the stored state, write every unit back */
  DASC_REFRESH_SCRATCH_MERGE_LOCAL = 1 /* start from zero, write back only the omitted units */
} dasc_refresh_mode_t;
typedef enum {
  DASC_ALGO_AUTO = 0,
  DASC_ALGO_SEQUENTIAL = 1, /* token-by-token fp32 kernel; any log-decay */
  DASC_ALGO_CHUNKED = 2     /* chunked (UT-transform) tensor-core kernel; see dasc_refresh */
} dasc_refresh_algo_t;

typedef struct dasc_plan_s dasc_plan_t; /* opaque */

/*
 * Plan description.  All pointers are HOST memory and are only read during
 * dasc_plan.  A_log and dt_bias hold one entry per selection unit, laid out
 * [n_layers][n_v_heads][units_per_head] with units_per_head = d_k (KDA) or
 * 1 (GDN); a caller whose model has one parameter per head broadcasts it.
 */
typedef struct {
  int32_t kind;                 /* dasc_kind_t */
  int32_t n_layers;             /* recurrent (linear-attention) layers only */
  int32_t n_v_heads;            /* value heads = number of head states per layer */
  int32_t n_k_heads;            /* key/query heads; divides n_v_heads; value head h reads key head h/(n_v_heads/n_k_heads) */
  int32_t d_k, d_v;             /* d_v must be a multiple of 4 (16-byte rows) */
  const float *A_log;           /* HOST, Eq. 2 */
  const float *dt_bias;         /* HOST, Eq. 2 */
  double a;                     /* fixed gate logit of the static metric; the paper uses -0.3 */
  double eps;                   /* Eq. 3; the paper uses 1e-3 */
  int32_t sel;                  /* dasc_sel_t */
  int32_t scope;                /* dasc_scope_t; TOP_RATIO only */
  double w_max;                 /* threshold of Section 4.1 and window cap of Eq. 7.  With TOP_RATIO or
                                   EXPLICIT, w_max <= 0 means: cap = next power of two of the largest
                                   omitted horizon. */
  double keep_ratio;            /* TOP_RATIO only, in [0, 1] */
  int32_t randomize;            /* != 0: replace each layer's selection by a seeded uniform draw of the
                                   same count r_l (the count-matched random control of Appendix C.3) */
  uint64_t seed;                /* for randomize */
  const uint8_t *explicit_mask; /* HOST, EXPLICIT only: [n_layers][units per layer], != 0 = retained */
  int64_t conv_bytes_per_ckpt;  /* B_conv of Eq. 6 (uncompressed convolution state), may be 0 */
} dasc_plan_desc_t;

/* Scalar results of a plan (Eq. 6, Eq. 7, Appendix B). */
typedef struct {
  int32_t kind, n_layers, n_v_heads, n_k_heads, d_k, d_v;
  int64_t units_per_layer;   /* n_l */
  int64_t unit_floats;       /* d_v (KDA) or d_k*d_v (GDN) */
  int64_t units_total;       /* sum_l n_l */
  int64_t units_retained;    /* sum_l r_l */
  int64_t r_max;             /* max_l r_l */
  int64_t slot_floats;       /* units_retained * unit_floats: the compact slot stride */
  int64_t dense_floats_per_layer; /* n_v_heads*d_k*d_v */
  double c_temp_rag;         /* Eq. 6: sum n_l / sum r_l        (inf if nothing is retained) */
  double c_temp_pad;         /* App. B: sum n_l / (L * R_max)   (inf if nothing is retained) */
  double c_ckpt_rag;         /* Eq. 6: (B_dense + B_conv) / (B_rag + B_conv) */
  double w_max_used;         /* window cap used by Eq. 7 */
  int64_t w_replay;          /* Eq. 7: max over omitted units of W_u; 0 if nothing is omitted */
  int32_t device;            /* CUDA device holding the index tables, -1 for a host-only plan */
} dasc_plan_info_t;

/*
 * Build the static selection plan (Section 4.1; it depends on model weights only,
 * so it is built once, before serving).
 * For every unit: g = -exp(A_log) * softplus(a + dt_bias) (Eq. 2),
 * H_s = ln(eps)/g (Eq. 3), all in fp64.  Selection per `sel`; TOP_RATIO keeps,
 * in each scope group of n units, the r = ceil(keep_ratio*n - 1e-9) units of
 * largest H_s, ties to the lower unit index.  Replay windows per Eq. 7:
 * W_u = clamp(next_pow2(H_s(u)), 4, w_max) with next_pow2 the smallest power
 * of two >= H_s, W_replay = max over omitted units.
 *
 * device >= 0: also uploads the index tables pack/restore/refresh need to
 * that CUDA device (the only device allocation this library ever makes).
 * device  < 0: host-only plan; the accessors work, device calls return
 * DASC_ERR_INVALID_ARG.
 * On error *out is NULL.
 */
dasc_status_t dasc_plan(const dasc_plan_desc_t *desc, int32_t device, dasc_plan_t **out);
void dasc_plan_destroy(dasc_plan_t *plan);

/*
 * A plan depends on model weights only (Section 4.1: built once offline), so it can be built where the weights are
 * and shipped to the serving processes.  dasc_plan_save writes a self-contained little-endian blob of
 * dasc_plan_save_bytes() bytes into the HOST buffer `buf` (scores, mask, windows and the scalar results; the index
 * tables are derived again on load); dasc_plan_load checks the blob (magic, version, sizes, that the counts it claims
 * are those of its mask) and rebuilds the plan, uploading its tables to `device` as dasc_plan does (device < 0: host
 * only).  A blob that fails a check gives DASC_ERR_INVALID_ARG and *out = NULL.
 */
dasc_status_t dasc_plan_save_bytes(const dasc_plan_t *plan, size_t *out);
dasc_status_t dasc_plan_save(const dasc_plan_t *plan, void *buf, size_t buf_bytes);
dasc_status_t dasc_plan_load(const void *buf, size_t bytes, int32_t device, dasc_plan_t **out);

/* Accessors.  Array outputs are HOST buffers the caller sized from dasc_plan_info:
 * horizon/mask/window: n_layers*units_per_layer entries, [layer][unit];
 * layer_counts: n_layers (r_l); layer_offsets: n_layers+1 (o_l). */
dasc_status_t dasc_plan_info(const dasc_plan_t *plan, dasc_plan_info_t *out);
dasc_status_t dasc_plan_horizon(const dasc_plan_t *plan, double *out);
dasc_status_t dasc_plan_mask(const dasc_plan_t *plan, uint8_t *out);
dasc_status_t dasc_plan_window(const dasc_plan_t *plan, int64_t *out);
dasc_status_t dasc_plan_layer_counts(const dasc_plan_t *plan, int64_t *out);
dasc_status_t dasc_plan_layer_offsets(const dasc_plan_t *plan, int64_t *out);

/*
 * Store path (Section 4.1; Appendix B, ragged layout): for each pair i,
 *     pool[dst_slot[i]][o_l + j] = unit j-th retained of layer l of request src_req[i]
 * as a bit copy (values are never interpreted; NaN payloads, -0.0 and
 * denormals survive).
 *   state_base  DEVICE, const, 16-byte aligned; strides in floats, multiples of 4.
 *   src_req     DEVICE int32[n_pairs]: request index of each source state.
 *   pool_base   DEVICE, 16-byte aligned.
 *   slot_stride floats between slots, multiple of 4, >= slot_floats; 0 = slot_floats.
 *   dst_slot    DEVICE int32[n_pairs]; destination slots must be distinct.
 * n_pairs == 0 is a no-op.  Source and pool must not overlap.
 */
dasc_status_t dasc_pack(const dasc_plan_t *plan, const float *state_base, int64_t layer_stride,
                        int64_t req_stride, const int32_t *src_req, float *pool_base,
                        int64_t slot_stride, const int32_t *dst_slot, int32_t n_pairs,
                        void *cuda_stream);

/*
 * Load path, zero-fill policy (Section 4.2: retained units are loaded exactly,
 * omitted units are left at zero).  For each pair i every float of the dense
 * state of request dst_req[i] (all layers, all heads) is written exactly once:
 * a retained unit gets the bits stored in slot src_slot[i], an omitted unit
 * gets +0.0f (all-zero bits).  Memory between the dense layers (when
 * layer_stride exceeds the dense layer size) is not touched.
 * Pointer, alignment and stride rules as for dasc_pack; dst_req must be distinct.
 */
dasc_status_t dasc_restore(const dasc_plan_t *plan, const float *pool_base, int64_t slot_stride,
                           const int32_t *src_slot, float *state_base, int64_t layer_stride,
                           int64_t req_stride, const int32_t *dst_req, int32_t n_pairs,
                           void *cuda_stream);

/*
 * Padded checkpoint layout (Appendix B, Scheme 1), the paper's comparison point for
 * the ragged layout: one contiguous pool [n_layers][n_slots][R_max][unit_floats]
 * fp32 with R_max = max_l r_l; entry (l, slot, j) holds the j-th retained unit of
 * layer l (ascending unit index) for j < r_l, and entries r_l .. R_max-1 are
 * padding that dasc_pack_padded never writes and dasc_restore_padded never reads.
 * The retained values are those of the ragged layout, so loading from either
 * layout gives the same state.
 *   dasc_padded_pool_floats  floats of such a pool for n_slots slots.
 *   pool_base  DEVICE, 16-byte aligned, at least that many floats.
 *   n_slots    the pool's slot count (> 0); slot indices must be < n_slots.
 * Everything else as for dasc_pack / dasc_restore.
 */
dasc_status_t dasc_padded_pool_floats(const dasc_plan_t *plan, int64_t n_slots, int64_t *out);
dasc_status_t dasc_pack_padded(const dasc_plan_t *plan, const float *state_base, int64_t layer_stride,
                               int64_t req_stride, const int32_t *src_req, float *pool_base,
                               int64_t n_slots, const int32_t *dst_slot, int32_t n_pairs,
                               void *cuda_stream);
dasc_status_t dasc_restore_padded(const dasc_plan_t *plan, const float *pool_base, int64_t n_slots,
                                  const int32_t *src_slot, float *state_base, int64_t layer_stride,
                                  int64_t req_stride, const int32_t *dst_req, int32_t n_pairs,
                                  void *cuda_stream);

/*
 * Complete-checkpoint accounting (host arithmetic only).
 * dasc_checkpoint_bytes: bytes of one checkpoint under a layout, temporal state
 *   plus the uncompressed convolution state B_conv that is stored alongside
 *   (Eq. 6, Appendix B): ragged sum_l r_l units, padded L * R_max units, dense
 *   sum_l n_l units, each unit_floats * 4 bytes, + conv_bytes.  Ratios of these
 *   are C_ckpt; dense / padded and dense / ragged differ by R_max / mean(r_l).
 * dasc_slot_budget (Appendix C.1): with per-rank temporal bytes b_r and the
 *   convolution bytes b_conv, N = floor(B / max_r (b_r + b_conv)) - 1; one slot
 *   is reserved by the allocator.  HOST pointers.
 */
typedef enum { DASC_LAYOUT_RAGGED = 0, DASC_LAYOUT_PADDED = 1, DASC_LAYOUT_DENSE = 2 } dasc_layout_t;
dasc_status_t dasc_checkpoint_bytes(const dasc_plan_t *plan, int32_t layout, int64_t conv_bytes, int64_t *out);
dasc_status_t dasc_slot_budget(int64_t budget_bytes, const int64_t *temporal_bytes_per_rank,
                               int32_t n_ranks, int64_t conv_bytes, int64_t *out);

/*
 * TP-balanced placement, second stage (Section 4.3), host arithmetic only: the TP
 * group is one storage pool with per-rank slot width C = ceil(sum_r U_r / T), U_r
 * the packed units of one checkpoint on rank r.  The packed units of all ranks,
 * taken in rank order, form one sequence, and the unit at global position p is
 * stored on rank p / C (the paper fixes C and that only remotely owned units move;
 * the assignment is this library's reading).
 *   units_per_rank  HOST int64[n_ranks]
 *   slot_width      HOST out: C
 *   send_counts     HOST out int64[n_ranks][n_ranks]: row r = how many of rank r's
 *                   units each rank stores, consecutive runs in rank order (the split
 *                   sizes of the variable-split all-to-all at Store; its transpose
 *                   is the Load transfer).  The diagonal entry stays on its rank.
 * dasc_pack_tp / dasc_restore_tp below move the units; the Python package also
 * carries a torch.distributed (library all-to-all) form of the same transfer.
 */
dasc_status_t dasc_tp_balance(const int64_t *units_per_rank, int32_t n_ranks, int64_t *slot_width,
                              int64_t *send_counts);

/*
 * TP-balanced placement, second stage, on the device (Section 4.3: at Store only
 * remotely owned units cross to another rank; Load applies the inverse transfer
 * before the compute-local layout is restored).  Rank `rank` of a TP group of
 * n_ranks packs its retained units as dasc_pack does, but the unit at global
 * position p = (sum of units_per_rank below `rank`) + (its index in this rank's
 * packed order) is stored in the pool of rank p / C at local unit index p % C,
 * C = ceil(sum_r U_r / T): the store goes straight into the owner's pool with
 * plain 16-byte stores (a push; for another GPU's pool the pointer is a peer
 * mapping, and nothing but this kernel's stores touches it).  dasc_restore_tp
 * is the inverse gather with the zero-fill of dasc_restore fused in.
 *   pool_bases      HOST array of n_ranks DEVICE pointers, 16-byte aligned: base
 *                   of every rank's pool as seen from this GPU.  n_ranks <= 16.
 *   units_per_rank  HOST int64[n_ranks]: U_r; entry `rank` must equal this plan's
 *                   units_retained (every rank has its own plan: its own heads).
 *   slot_stride     floats between a rank's slots, multiple of 4, >= C*unit_floats;
 *                   0 = C*unit_floats.  Slot s of a rank holds local units [0, C).
 * Ordering between ranks is the caller's: a Store is visible to the other ranks'
 * Loads once its stream has been synchronised and the ranks have met (a barrier
 * of the caller's process group).  All else as for dasc_pack / dasc_restore.
 */
dasc_status_t dasc_pack_tp(const dasc_plan_t *plan, const float *state_base, int64_t layer_stride,
                           int64_t req_stride, const int32_t *src_req, float *const *pool_bases,
                           const int64_t *units_per_rank, int32_t n_ranks, int32_t rank,
                           int64_t slot_stride, const int32_t *dst_slot, int32_t n_pairs,
                           void *cuda_stream);
dasc_status_t dasc_restore_tp(const dasc_plan_t *plan, float *const *pool_bases,
                              const int64_t *units_per_rank, int32_t n_ranks, int32_t rank,
                              int64_t slot_stride, const int32_t *src_slot, float *state_base,
                              int64_t layer_stride, int64_t req_stride, const int32_t *dst_req,
                              int32_t n_pairs, void *cuda_stream);

/*
 * TP-balanced placement, first stage (Section 4.3: a model-load-time permutation
 * redistributes linear-attention head bundles across TP ranks, an exact
 * re-indexing).  The paper does not state how the permutation is chosen; this
 * library's reading: every rank keeps the same number of bundles per layer (so
 * compute stays balanced), and bundles are placed greedily, layers in ascending
 * order, within a layer the bundle with the most retained units first (ties: the
 * lower index), each on the rank with the smallest payload so far that still
 * has room in this layer (ties: the lower rank).  Host arithmetic only.
 *   heads_per_bundle  value heads that must move together (1 for KDA; H_v/H_k
 *                     for GDN, where a key head and its value heads are coupled);
 *                     n_v_heads / heads_per_bundle must be a multiple of n_ranks.
 *   perm              HOST out int32[n_layers][n_bundles]: perm[l][i] = original
 *                     bundle at position i of layer l; rank r owns positions
 *                     [r*n_bundles/T, (r+1)*n_bundles/T), ascending original index.
 *   units_per_rank    HOST out int64[n_ranks]: U_r under this placement.
 */
dasc_status_t dasc_tp_head_permutation(const dasc_plan_t *plan, int32_t n_ranks, int32_t heads_per_bundle,
                                       int32_t *perm, int64_t *units_per_rank);

/*
 * The convolution state of a checkpoint (Section 4.1: stored uncompressed, in
 * bf16, beside the temporal state; B_conv of Eq. 6).  To this library it is an
 * opaque blob of conv_bytes per request:
 *     pool[dst_slot[i]] = conv[src_req[i]]   (store)      conv[dst_req[i]] = pool[src_slot[i]]   (load)
 * as bit copies.  Bases DEVICE and 16-byte aligned; conv_bytes and both strides
 * (bytes between requests / between slots, >= conv_bytes) multiples of 16.
 */
dasc_status_t dasc_conv_store(const void *conv_base, int64_t req_stride_bytes, const int32_t *src_req,
                              void *pool_base, int64_t slot_stride_bytes, const int32_t *dst_slot,
                              int64_t conv_bytes, int32_t n_pairs, void *cuda_stream);
dasc_status_t dasc_conv_load(const void *pool_base, int64_t slot_stride_bytes, const int32_t *src_slot,
                             void *conv_base, int64_t req_stride_bytes, const int32_t *dst_req,
                             int64_t conv_bytes, int32_t n_pairs, void *cuda_stream);

/*
 * INT8 checkpoint codec fused into the Store / Load copies (Appendix D, Eq. 10).
 * A row is the d_v values of one (layer, head, key channel) tuple; rows are the
 * plan's retained rows in ragged order (a retained GDN head contributes its d_k
 * rows).  Per row, in fp32 arithmetic:
 *     a = max_v |S|,  s = max(a, 1e-8) / 127,
 *     q = clip(round(S / s), -127, 127)     (round to nearest, ties to even)
 * and on load  S_hat = q * s  (one fp32 multiply); omitted rows are zero-filled
 * exactly as in dasc_restore.  Values must be finite (the formula says nothing
 * about NaN or infinity; their codes are unspecified).
 *
 * Slot layout in BYTES: [packed_rows][d_v] int8 codes, then [packed_rows] fp32
 * scales, packed_rows = sum_r for KDA and sum_r * d_k for GDN.
 *   dasc_int8_slot_bytes  bytes of one slot, rounded up to a multiple of 16.
 *   pool_base             DEVICE, 16-byte aligned.
 *   slot_stride_bytes     bytes between slots, multiple of 16, >= the slot
 *                         size; 0 = the slot size.
 * Everything else (state pointer, strides in floats, index arrays, n_pairs,
 * distinctness, stream, errors) as for dasc_pack / dasc_restore.
 * d_v must be a power of two between 4 and 128 (DASC_ERR_SHAPE otherwise).
 */
dasc_status_t dasc_int8_slot_bytes(const dasc_plan_t *plan, size_t *out);
dasc_status_t dasc_pack_int8(const dasc_plan_t *plan, const float *state_base, int64_t layer_stride,
                             int64_t req_stride, const int32_t *src_req, void *pool_base,
                             int64_t slot_stride_bytes, const int32_t *dst_slot, int32_t n_pairs,
                             void *cuda_stream);
dasc_status_t dasc_restore_int8(const dasc_plan_t *plan, const void *pool_base,
                                int64_t slot_stride_bytes, const int32_t *src_slot,
                                float *state_base, int64_t layer_stride, int64_t req_stride,
                                const int32_t *dst_req, int32_t n_pairs, void *cuda_stream);

/*
 * Suffix refresh: replay the gated delta rule (Eq. 1, transposed orientation)
 *     S_t = (I - beta_t k_t k_t^T) Diag(alpha_t) S_{t-1} + beta_t k_t v_t^T,   alpha_t = exp(g_t)
 *     o_t = q_scale * S_t^T q_t
 * over each request's token range, for layers [layer_begin, layer_end) and
 * all value heads, updating the fp32 states in place.  alpha_t is channel-wise
 * for KDA and one scalar per value head for GDN.
 *
 * Token streams (DEVICE, const), with Lc = layer_end - layer_begin and
 * T = total_tokens = cu_seqlens[n_req]:
 *   q, k   [Lc][T][n_k_heads][d_k]   bf16 or fp32 (io_dtype)
 *   v      [Lc][T][n_v_heads][d_v]   same dtype
 *   g      [Lc][T][n_v_heads][d_k]   fp32 log-decay, KDA;  [Lc][T][n_v_heads] for GDN
 *   beta   [Lc][T][n_v_heads]        fp32
 *   o      [Lc][T][n_v_heads][d_v]   o_dtype (bf16 or fp32, independent of io_dtype), out;
 *                                     NULL = outputs not wanted
 *   cu_seqlens DEVICE int32[n_req+1], ascending from 0: request r owns tokens
 *          [cu_seqlens[r], cu_seqlens[r+1]) of every layer; empty ranges are allowed.
 *   req_idx    DEVICE int32[n_req]: which dense state each request updates (distinct).
 *   max_seqlen an upper bound on any request's token count (sizes the launch).
 *
 * mode CONTINUE: S_0 is the state as stored (for instance just restored);
 *   every unit is written back.  This continues the recurrence.
 * mode SCRATCH_MERGE_LOCAL (the paper's suffix-refresh load policy, Section 4.2):
 *   S_0 = 0 in a scratch state; afterwards only the units the plan OMITS are
 *   copied into the stored state, retained units keep their stored values.
 *
 * algo SEQUENTIAL is exact fp32 arithmetic token by token and accepts any g <= 0.
 * algo CHUNKED processes 32-token chunks on the tensor cores (tf32 operands,
 *   fp32 accumulation and fp32 state); it needs d_k = d_v = 128 and bf16 q/k/v
 *   (DASC_ERR_SHAPE otherwise) and, for every channel and every half chunk of
 *   16 tokens, |sum g| <= 80 (decay factors are formed relative to the chunk
 *   midpoint in fp32).  That bound is checked on the device while the sums are
 *   formed.  A (request, layer, head) unit that breaks it is NOT written back:
 *   its stored state keeps the bits it had before the call, its outputs are
 *   unspecified, its index ((request*Lc + layer)*n_v_heads + head) is appended
 *   to the int32 list that starts 256 bytes into the workspace (length: third
 *   header word), and dasc_refresh_status reports DASC_ERR_DOMAIN.  Every other
 *   unit is complete.
 * algo AUTO runs CHUNKED when shape and dtype allow it, and then, on the same
 *   stream, replays with the exact kernel (a) the units that broke the bound,
 *   from their untouched stored states, and (b) requests of at most 8 tokens,
 *   where one tf32-rounded q.k product can exceed the output tolerance.  Under
 *   AUTO a call therefore completes for any g <= 0 and dasc_refresh_status
 *   stays DASC_OK; dasc_refresh_counters tells how many units took the exact
 *   path.  When shape or dtype rule the chunked kernel out, AUTO is SEQUENTIAL.
 *
 * workspace: DEVICE scratch of at least dasc_refresh_workspace_bytes() (256
 *   bytes of flags and counters + 4 bytes per unit of the call, for CHUNKED and
 *   AUTO), 256-byte aligned, private to this call until it completes; may be
 *   NULL when that size is 0.
 * Errors: bad arguments -> no launch.  A bounded device-side wait that runs
 *   out sets the first header word (DASC_ERR_TIMEOUT): the CTA that gave up
 *   skips the rest of its work and leaves its unit's stored state untouched.
 *   Read the flags with dasc_refresh_status after synchronising the stream.
 */
dasc_status_t dasc_refresh_workspace_bytes(const dasc_plan_t *plan, int32_t n_req, int32_t n_layers_in_call,
                                           int32_t algo, size_t *out);
dasc_status_t dasc_refresh(const dasc_plan_t *plan, float *state_base, int64_t layer_stride,
                           int64_t req_stride, const int32_t *req_idx, const void *q, const void *k,
                           const void *v, int32_t io_dtype, const float *g, const float *beta,
                           const int32_t *cu_seqlens, int32_t n_req, int64_t total_tokens,
                           int32_t max_seqlen, int32_t layer_begin, int32_t layer_end, float q_scale,
                           void *o, int32_t o_dtype, int32_t mode, int32_t algo, void *workspace,
                           size_t workspace_bytes, void *cuda_stream);
/* After the stream has been synchronised: DASC_OK; DASC_ERR_TIMEOUT if a
 * device-side wait of the last dasc_refresh that used `workspace` gave up;
 * else DASC_ERR_DOMAIN if that call left a unit unwritten because its
 * log-decay was outside the chunked kernel's range.  Copies the first 8
 * bytes device -> host (synchronous); pass workspace_bytes >= 8 (with 4 only
 * the time-out word is read).
 * dasc_refresh_counters (same conditions, 16 bytes): units the chunked kernel
 * handed over, and units the exact kernel replayed from that list. */
dasc_status_t dasc_refresh_status(const void *workspace, size_t workspace_bytes);
dasc_status_t dasc_refresh_counters(const void *workspace, size_t workspace_bytes, int32_t *handed_over,
                                    int32_t *replayed_exactly);
/* Test hook, not for production use: when `polls` != 0 the chunked kernel's
 * issuing warp gives its very first wait of every CTA only that many polls, so
 * that a test can watch a bounded wait run out (DASC_ERR_TIMEOUT, the unit left
 * unwritten, the context still usable).  0 restores the normal limit.  Process-wide. */
void dasc_debug_set_refresh_poll_limit(uint32_t polls);

/*
 * Load path, suffix-refresh policy as the paper states it (Section 4.2, with the
 * window of Eq. 7): after dasc_restore has loaded the retained units of a hit,
 * each request's last `window` tokens BEFORE the cache boundary are replayed
 * from a zero scratch state, and only the units the plan omits are copied from
 * the scratch state into the stored state (SCRATCH_MERGE_LOCAL); retained units
 * keep their exactly loaded values.  A request whose available prefix is
 * shorter than the window replays the whole prefix (Table 8: replayed tokens
 * per hit are the window clipped by the prefix).
 *   cu_seqlens   DEVICE int32[n_req+1]: request r's available prefix is tokens
 *                [cu_seqlens[r], cu_seqlens[r+1]) of the streams; the replayed
 *                range is [max(cu_seqlens[r], cu_seqlens[r+1] - window), cu_seqlens[r+1]).
 *   window       W_replay in tokens; <= 0 means the plan's own W_replay (Eq. 7).
 *                When that is 0 (nothing omitted) only window_begin is written.
 *   window_begin DEVICE int32[n_req], written by the call: first replayed token
 *                of each request (cu_seqlens[r+1] - window_begin[r] tokens are
 *                replayed); caller-owned, must stay valid until the call completes.
 *   q, o         outputs are not part of this policy: pass o = NULL, and then q
 *                may be NULL too and the kernels skip the output side entirely
 *                (state-only fast path).  With o != NULL outputs of the replayed
 *                tokens are written at their stream positions (from the scratch
 *                state, i.e. without the retained history).
 * Everything else as for dasc_refresh (mode is fixed; max_seqlen is the window).
 */
dasc_status_t dasc_refresh_window(const dasc_plan_t *plan, float *state_base, int64_t layer_stride,
                                  int64_t req_stride, const int32_t *req_idx, const void *q,
                                  const void *k, const void *v, int32_t io_dtype, const float *g,
                                  const float *beta, const int32_t *cu_seqlens, int32_t n_req,
                                  int64_t total_tokens, int64_t window, int32_t layer_begin,
                                  int32_t layer_end, float q_scale, void *o, int32_t o_dtype,
                                  int32_t algo, int32_t *window_begin, void *workspace,
                                  size_t workspace_bytes, void *cuda_stream);

/*
 * The paper has no counterpart to this call: it is dasc_refresh (chunked tensor-core kernel,
 * bf16 token streams, d_k = d_v = 128) for callers that cannot hand over a workspace because
 * they cannot allocate device memory at the point of the call.  The typical case is a serving
 * engine whose start-up code has carved all of the GPU's memory into weights, KV cache and
 * state pools: on the cache-hit path a cudaMalloc (or a framework allocator that may fall
 * back to one) can fail for lack of free memory or stall the device, and no spare buffer was
 * planned for this library.
 *
 * The kernel's scratch lives in a 4096-byte array that is part of the library image: every
 * GPU that loads libdasc holds those bytes until the process exits.  The first 256 bytes are
 * the header dasc_refresh_status reads (word 0: a wait timed out; word 1: a unit outside the
 * log-decay range was left unwritten), the remaining 3840 bytes hold the list of up to 960
 * unit indices that the chunked kernel hands to the exact kernel for that reason.  The kernel cannot do without the header: were it ever to outgrow the array
 * the call would return DASC_ERR_WORKSPACE; shapes the chunked kernel does not take get
 * DASC_ERR_SHAPE.  The call makes no cudaMalloc / cudaFree and uses no allocating library
 * routine.
 *
 * First call on a device: the library looks up the array's device address for the CURRENT
 * device, which must be the plan's device (DASC_ERR_INVALID_ARG otherwise), and remembers it.
 * Make that first call before any stream capture is begun, since the look-up is not a stream
 * operation.
 * All calls on one device share the array and it keeps the last call's contents; the call
 * clears the header words on `cuda_stream` before the kernel runs.  Two dasc_refresh_static
 * calls that overlap on the GPU (different streams, no ordering) race on the header and the
 * list: order them, or give one of them its own workspace through dasc_refresh.
 *
 * Arguments are those of dasc_refresh with io_dtype fixed to bf16, algo fixed to CHUNKED and
 * no workspace.  *scratch_out (may be NULL) receives the DEVICE address of the array: after
 * synchronising the stream, dasc_refresh_status(*scratch_out, 8) reports a time-out or a
 * log-decay outside the range (pass 8 bytes or more: with 4 only the time-out word is read).
 * Units outside the chunked kernel's log-decay range are replayed by the exact kernel on the
 * same stream, as under DASC_ALGO_AUTO (that kernel needs no scratch beyond the list), so the
 * status stays DASC_OK for up to 960 such units per call; beyond that the surplus units keep
 * their stored states and the status is DASC_ERR_DOMAIN.  Short requests are not rerouted
 * here (algo is CHUNKED in every other respect).
 */
dasc_status_t dasc_refresh_static(const dasc_plan_t *plan, float *state_base, int64_t layer_stride,
                                  int64_t req_stride, const int32_t *req_idx, const void *q, const void *k,
                                  const void *v, const float *g, const float *beta, const int32_t *cu_seqlens,
                                  int32_t n_req, int64_t total_tokens, int32_t max_seqlen, int32_t layer_begin,
                                  int32_t layer_end, float q_scale, void *o, int32_t o_dtype, int32_t mode,
                                  void **scratch_out, void *cuda_stream);

const char *dasc_status_string(dasc_status_t status);
/* "major.minor.patch" of this library. */
const char *dasc_version(void);

#ifdef __cplusplus
}
#endif
#endif /* DASC_H_ */
