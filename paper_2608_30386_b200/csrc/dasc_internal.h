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

// Launchers (pack_restore.cu, refresh_seq.cu, refresh_chunked.cu).  All return cudaError_t as int.
int dasc_launch_pack(const dasc_plan_s *plan, const float *state, int64_t layer_stride, int64_t req_stride,
                     const int32_t *src_req, float *pool, int64_t slot_stride, const int32_t *dst_slot,
                     int32_t n_pairs, void *stream);
int dasc_launch_restore(const dasc_plan_s *plan, const float *pool, int64_t slot_stride, const int32_t *src_slot,
                        float *state, int64_t layer_stride, int64_t req_stride, const int32_t *dst_req,
                        int32_t n_pairs, void *stream);

// pack_restore_padded.cu: pool [L][n_slots][R_max][unit]
int dasc_launch_pack_padded(const dasc_plan_s *plan, const float *state, int64_t layer_stride, int64_t req_stride,
                            const int32_t *src_req, float *pool, int64_t n_slots, const int32_t *dst_slot,
                            int32_t n_pairs, void *stream);
int dasc_launch_restore_padded(const dasc_plan_s *plan, const float *pool, int64_t n_slots, const int32_t *src_slot,
                               float *state, int64_t layer_stride, int64_t req_stride, const int32_t *dst_req,
                               int32_t n_pairs, void *stream);

// codec_int8.cu
int dasc_launch_pack_int8(const dasc_plan_s *plan, const float *state, int64_t layer_stride, int64_t req_stride,
                          const int32_t *src_req, void *pool, int64_t slot_stride_bytes, const int32_t *dst_slot,
                          int32_t n_pairs, void *stream);
int dasc_launch_restore_int8(const dasc_plan_s *plan, const void *pool, int64_t slot_stride_bytes,
                             const int32_t *src_slot, float *state, int64_t layer_stride, int64_t req_stride,
                             const int32_t *dst_req, int32_t n_pairs, void *stream);

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
  void *workspace;
  size_t workspace_bytes;
};
int dasc_launch_refresh_seq(const DascRefreshArgs &a, void *stream);
int dasc_launch_refresh_chunked(const DascRefreshArgs &a, void *stream);
size_t dasc_refresh_chunked_workspace_bytes(int32_t n_req, int32_t n_layers_in_call, int32_t H_v);
