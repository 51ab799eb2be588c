// Store / Load copies for the padded checkpoint layout (Appendix B, Scheme 1):
// pool [L][slots][R_max][unit], the first r_l entries of layer l valid, the rest padding that is
// neither written nor read.  Same row tables, vector width and launch shape as the ragged copies;
// only the pool address differs.  The paper keeps this layout as the comparison point for the
// ragged one (capacity gain R_max / mean r_l), and so does this library.
#include <cuda_runtime.h>

#include "dasc_internal.h"

namespace {

constexpr int kThreads = 256;
constexpr int kUnroll = 4;

__device__ __forceinline__ uint4 ld_stream(const uint4 *p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}
__device__ __forceinline__ void st_stream(uint4 *p, const uint4 &v) {
  asm volatile("st.global.L1::no_allocate.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z),
               "r"(v.w)
               : "memory");
}

// grid = (ceil(R_max * vecs_per_unit / (kThreads*kUnroll)), n_layers, pairs): one layer per block row, so the layer's
// first packed row is a per-block constant and no load depends on another table.  entry_stride4 = 16-byte vectors
// between consecutive (layer, slot) blocks of the pool: R_max rows of vecs_per_row vectors.
__global__ void __launch_bounds__(kThreads, 8) pack_padded_kernel(const uint4 *__restrict__ state, int64_t layer_stride4,
                                                               int64_t req_stride4, const int32_t *__restrict__ src_req,
                                                               uint4 *__restrict__ pool, int64_t n_slots,
                                                               int64_t entry_stride4, const int32_t *__restrict__ dst_slot,
                                                               const DascRowSrc *__restrict__ row_src,
                                                               const int32_t *__restrict__ layer_row_off,
                                                               uint32_t vecs_per_row, int32_t n_pairs) {
  const uint32_t base = blockIdx.x * (kThreads * kUnroll) + threadIdx.x;
  const int32_t layer = blockIdx.y;
  const uint32_t first = static_cast<uint32_t>(__ldg(layer_row_off + layer));
  const uint32_t layer_vecs = (static_cast<uint32_t>(__ldg(layer_row_off + layer + 1)) - first) * vecs_per_row;
  if (blockIdx.x * (kThreads * kUnroll) >= layer_vecs) return;
  const int2 *src_l = reinterpret_cast<const int2 *>(row_src) + first;  // {layer, dense row} of the layer's packed rows
  for (int32_t pair = blockIdx.z; pair < n_pairs; pair += gridDim.z) {
    const uint4 *src_base = state + static_cast<int64_t>(__ldg(src_req + pair)) * req_stride4 + layer * layer_stride4;
    uint4 *dst_base = pool + (layer * n_slots + __ldg(dst_slot + pair)) * entry_stride4;
    uint4 val[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const uint32_t i = base + u * kThreads;
      if (i < layer_vecs) {
        const uint32_t row = i / vecs_per_row;
        const uint32_t vec = i - row * vecs_per_row;
        val[u] = ld_stream(src_base + static_cast<int64_t>(__ldg(src_l + row).y) * vecs_per_row + vec);
      }
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const uint32_t i = base + u * kThreads;
      if (i < layer_vecs) st_stream(dst_base + i, val[u]);
    }
  }
}

// grid = (ceil(layer_vecs / (kThreads*kUnroll)), n_layers, pairs).
__global__ void __launch_bounds__(kThreads) restore_padded_kernel(const uint4 *__restrict__ pool, int64_t n_slots,
                                                                  int64_t entry_stride4,
                                                                  const int32_t *__restrict__ src_slot,
                                                                  uint4 *__restrict__ state, int64_t layer_stride4,
                                                                  int64_t req_stride4, const int32_t *__restrict__ dst_req,
                                                                  const int32_t *__restrict__ row_pos,
                                                                  const int32_t *__restrict__ layer_row_off,
                                                                  uint32_t layer_vecs, uint32_t rows_per_layer,
                                                                  uint32_t vecs_per_row, int32_t n_pairs) {
  const uint32_t base = blockIdx.x * (kThreads * kUnroll) + threadIdx.x;
  const int32_t layer = blockIdx.y;
  const int32_t *pos_l = row_pos + static_cast<int64_t>(layer) * rows_per_layer;
  const int32_t first = __ldg(layer_row_off + layer);  // packed row of the layer's first retained row
  for (int32_t pair = blockIdx.z; pair < n_pairs; pair += gridDim.z) {
    const uint4 *src_base = pool + (layer * n_slots + __ldg(src_slot + pair)) * entry_stride4;
    uint4 *dst_base = state + static_cast<int64_t>(__ldg(dst_req + pair)) * req_stride4 + layer * layer_stride4;
    uint4 val[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const uint32_t i = base + u * kThreads;
      val[u] = make_uint4(0u, 0u, 0u, 0u);  // omitted rows: +0.0f
      if (i < layer_vecs) {
        const uint32_t row = i / vecs_per_row;
        const uint32_t vec = i - row * vecs_per_row;
        const int32_t pos = __ldg(pos_l + row);
        if (pos >= 0) val[u] = ld_stream(src_base + static_cast<int64_t>(pos - first) * vecs_per_row + vec);
      }
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const uint32_t i = base + u * kThreads;
      if (i < layer_vecs) st_stream(dst_base + i, val[u]);
    }
  }
}

}  // namespace

int dasc_launch_pack_padded(const dasc_plan_s *plan, const float *state, int64_t layer_stride, int64_t req_stride,
                            const int32_t *src_req, float *pool, int64_t n_slots, const int32_t *dst_slot,
                            int32_t n_pairs, void *stream) {
  const uint32_t vpr = static_cast<uint32_t>(plan->info.d_v / 4);
  const uint64_t packed_vecs = static_cast<uint64_t>(plan->packed_rows) * vpr;
  if (packed_vecs == 0 || n_pairs == 0) return cudaSuccess;
  const int64_t rows_per_unit = plan->info.unit_floats / plan->info.d_v;
  const int64_t entry_stride4 = plan->info.r_max * rows_per_unit * vpr;
  const uint32_t per_block = kThreads * kUnroll;
  const uint64_t max_layer_vecs = static_cast<uint64_t>(entry_stride4);
  dim3 grid(static_cast<uint32_t>((max_layer_vecs + per_block - 1) / per_block),
            static_cast<uint32_t>(plan->info.n_layers), static_cast<uint32_t>(n_pairs < 65535 ? n_pairs : 65535));
  pack_padded_kernel<<<grid, kThreads, 0, static_cast<cudaStream_t>(stream)>>>(
      reinterpret_cast<const uint4 *>(state), layer_stride / 4, req_stride / 4, src_req, reinterpret_cast<uint4 *>(pool),
      n_slots, entry_stride4, dst_slot, plan->d_row_src, plan->d_layer_row_off, vpr, n_pairs);
  return static_cast<int>(cudaGetLastError());
}

int dasc_launch_restore_padded(const dasc_plan_s *plan, const float *pool, int64_t n_slots, const int32_t *src_slot,
                               float *state, int64_t layer_stride, int64_t req_stride, const int32_t *dst_req,
                               int32_t n_pairs, void *stream) {
  const uint32_t vpr = static_cast<uint32_t>(plan->info.d_v / 4);
  const uint64_t layer_vecs = static_cast<uint64_t>(plan->rows_per_layer) * vpr;
  if (n_pairs == 0) return cudaSuccess;
  const int64_t rows_per_unit = plan->info.unit_floats / plan->info.d_v;
  const int64_t entry_stride4 = plan->info.r_max * rows_per_unit * vpr;
  const uint32_t per_block = kThreads * kUnroll;
  dim3 grid(static_cast<uint32_t>((layer_vecs + per_block - 1) / per_block),
            static_cast<uint32_t>(plan->info.n_layers), static_cast<uint32_t>(n_pairs < 65535 ? n_pairs : 65535));
  restore_padded_kernel<<<grid, kThreads, 0, static_cast<cudaStream_t>(stream)>>>(
      reinterpret_cast<const uint4 *>(pool), n_slots, entry_stride4, src_slot, reinterpret_cast<uint4 *>(state),
      layer_stride / 4, req_stride / 4, dst_req, plan->d_row_pos, plan->d_layer_row_off,
      static_cast<uint32_t>(layer_vecs), static_cast<uint32_t>(plan->rows_per_layer), vpr, n_pairs);
  return static_cast<int>(cudaGetLastError());
}
