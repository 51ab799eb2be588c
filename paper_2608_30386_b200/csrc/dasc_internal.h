// Internal declarations shared by the translation units of libdasc.
#pragma once
#include <cstdint>
#include <vector>

#include "dasc.h"

// One entry per packed row: where in the dense state it comes from.
struct DascRowSrc {
  int32_t layer;  // layer index
  int32_t row;    // dense row inside the layer: head*d_k + k, a row of d_v floats
};

struct dasc_plan_s {
  dasc_plan_info_t info{};
  std::vector<double> horizon;       // [L][n_l]
  std::vector<uint8_t> mask;         // [L][n_l], 1 = retained
  std::vector<int64_t> window;       // [L][n_l], Eq. 7 W_u
  std::vector<int64_t> layer_count;  // r_l
  std::vector<int64_t> layer_offset; // o_l, L+1 entries

  // Row-granular tables (a row = d_v floats; a GDN unit is d_k consecutive rows).
  int64_t rows_per_layer = 0;        // n_v_heads * d_k
  int64_t packed_rows = 0;           // rows per slot
  std::vector<DascRowSrc> row_src;   // [packed_rows]
  std::vector<int32_t> row_pos;      // [L][rows_per_layer]: packed row or -1

  // Device copies (device >= 0 only).
  DascRowSrc *d_row_src = nullptr;
  int32_t *d_row_pos = nullptr;
  uint8_t *d_row_keep = nullptr;     // [L][rows_per_layer]: 1 = retained row
  int32_t *d_layer_row_off = nullptr;  // [L+1]: packed row at which each layer starts
};

// plan_host.cpp
dasc_status_t dasc_build_plan_host(const dasc_plan_desc_t *desc, dasc_plan_s *plan);
void dasc_plan_row_tables(dasc_plan_s *plan);  // row_src / row_pos / packed_rows from info + mask

// Section 4.3, second stage: where this rank's packed units live in the TP group's shared storage pool.
constexpr int DASC_TP_MAX_RANKS = 16;
struct DascTpPlacement {
  int32_t n_ranks;
  float *pool_base[DASC_TP_MAX_RANKS];  // DEVICE pool of each owner rank (a peer mapping for another GPU)
  int64_t unit_begin;                   // global position of this rank's first packed unit: sum of U_r over lower ranks
  int64_t width;                        // C = ceil(sum_r U_r / T)
};

// Launchers (pack_restore.cu, refresh_seq.cu, refresh_chunked.cu).  All return cudaError_t as int.
// layout: 0 ragged [slots][sum r_l] (pool_stride = floats between slots), 1 padded [L][n_slots][R_max][unit],
// 2 TP-balanced (`placement` set; pool_stride = floats between one rank's slots).
int dasc_launch_pack(const dasc_plan_s *plan, const float *state, int64_t layer_stride, int64_t req_stride,
                     const int32_t *src_req, float *pool, int64_t pool_stride, int64_t n_slots, const int32_t *dst_slot,
                     int32_t n_pairs, int layout, const DascTpPlacement *placement, void *stream);
int dasc_launch_restore(const dasc_plan_s *plan, const float *pool, int64_t pool_stride, int64_t n_slots,
                        const int32_t *src_slot, float *state, int64_t layer_stride, int64_t req_stride,
                        const int32_t *dst_req, int32_t n_pairs, int layout, const DascTpPlacement *placement,
                        void *stream);
// dst[dst_idx[i]] = src[src_idx[i]], blobs of blob_bytes (multiple of 16)
int dasc_launch_blob_copy(const void *src, int64_t src_stride_bytes, const int32_t *src_idx, void *dst,
                          int64_t dst_stride_bytes, const int32_t *dst_idx, int64_t blob_bytes, int32_t n_pairs,
                          void *stream);

// codec_int8.cu
int dasc_launch_pack_int8(const dasc_plan_s *plan, const float *state, int64_t layer_stride, int64_t req_stride,
                          const int32_t *src_req, void *pool, int64_t slot_stride_bytes, const int32_t *dst_slot,
                          int32_t n_pairs, void *stream);
int dasc_launch_restore_int8(const dasc_plan_s *plan, const void *pool, int64_t slot_stride_bytes,
                             const int32_t *src_slot, float *state, int64_t layer_stride, int64_t req_stride,
                             const int32_t *dst_req, int32_t n_pairs, void *stream);

// Refresh workspace (device): a header of 256 bytes followed by a list of unit indices.
//   word 0  a bounded device-side wait ran out
//   word 1  a unit left the chunked kernel's log-decay range and nothing replayed it (an error)
//   word 2  units the chunked kernel handed over (out of range, or shorter than its threshold): length of the list
//   word 3  units the token-by-token kernel replayed from the list
//   bytes 256...: int32 unit indices ((request * layers_in_call + layer) * H_v + head), in hand-over order
constexpr size_t kRefreshWsHeader = 256;
// Requests of at most this many tokens are replayed by the exact kernel under DASC_ALGO_AUTO: with only a handful of
// tokens every output is a sum of a few q.k products, so the tf32 rounding of one product can exceed the output
// tolerance, and the tensor-core kernel has no speed to offer at that length anyway.
constexpr int kShortSuffix = 8;

struct DascRefreshArgs {
  int32_t kind, H_v, H_k, d_k, d_v;
  float *state;
  int64_t layer_stride, req_stride;
  const int32_t *req_idx;
  const void *q, *k, *v;
  int32_t io_bf16;
  const float *g, *beta;
  const int32_t *cu_seqlens;
  const int32_t *tok_begin;  // device, [n_req], or null: first token of each request (null = cu_seqlens[r])
  int32_t n_req;
  int64_t total_tokens;
  int32_t max_seqlen;
  int32_t layer_begin, n_layers_in_call;
  float q_scale;
  void *o;
  int32_t o_bf16;
  int32_t mode;
  const uint8_t *row_keep;  // device, [L][rows_per_layer]
  int64_t rows_per_layer;
  void *workspace;          // header words as above (null only for the token-by-token kernel run on its own)
  size_t workspace_bytes;
  int32_t *unit_list;       // device, or null: where units are handed over (chunked) / taken from (token-by-token)
  int32_t unit_list_cap;    // entries the list can hold
  int32_t short_thr;        // chunked kernel: units of at most this many tokens are handed over; -1 = none
  int32_t from_list;        // token-by-token kernel: 1 = replay the listed units only, 0 = every unit of the grid
  int32_t domain_is_error;  // chunked kernel: an out-of-range unit also sets word 1
  uint32_t poll_limit_first_wait;  // test hook: poll limit of the issuing warp's very first wait (0 = the normal limit)
};
int dasc_launch_refresh_seq(const DascRefreshArgs &a, void *stream);
int dasc_launch_refresh_chunked(const DascRefreshArgs &a, void *stream);
size_t dasc_refresh_chunked_workspace_bytes(int32_t n_req, int32_t n_layers_in_call, int32_t H_v);
// Test hook (see dasc_debug_set_refresh_poll_limit in dasc.h).
extern uint32_t g_dasc_debug_poll_limit;
