// Store / Load copy kernels: pack (gather retained rows into a checkpoint pool) and restore
// (scatter back with the zero-fill fused, every dense byte written once).  Pure HBM-bandwidth
// work: 128-bit streaming loads and stores, four independent loads in flight per thread, index
// tables small enough to live in L2.
//
// One pair of kernels serves three pool layouts; only the pool address of a packed row differs:
//   Ragged      (Appendix B, Scheme 2)  pool[slot][o_l + j]            the layout of the Store / Load path
//   Padded      (Appendix B, Scheme 1)  pool[l][slot][j], j < R_max    the paper's comparison layout
//   TpBalanced  (Section 4.3, stage 2)  the packed units of all TP ranks form one sequence; the unit at global
//               position p lives in the pool of rank p / C at local index p % C, C = ceil(sum_r U_r / T).
//               A rank stores straight into the owner's pool (plain 16-byte stores through a peer
//               mapping when the owner is another GPU) and loads from it on the way back.
// Also here: the indexed copy of the opaque convolution-state blob that is stored uncompressed beside the
// temporal state (Section 4.1, B_conv of Eq. 6).
#include <cuda_runtime.h>

#include "dasc_internal.h"

namespace {

constexpr int kThreads = 256;  // threads per block and loads in flight per thread: the best of a measured sweep
constexpr int kUnroll = 4;     // over {128..1024} x {2..16}

enum class Layout { Ragged, Padded, TpBalanced };

struct TpPools {
  uint4 *base[DASC_TP_MAX_RANKS];  // pool of each owner rank
  uint32_t unit_begin;             // global position of this rank's first packed unit
  uint32_t width;                  // C: units per rank and slot
  uint32_t unit_vecs;              // 16-byte vectors per unit
  int32_t unit_shift;              // log2(unit_vecs) when that is a power of two, else -1
  uint32_t width_magic;            // owner = umulhi(pos, width_magic) >> width_shift for every pos < 2^31 (width >= 2)
  uint32_t width_shift;
};

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

// Where vector `pv` (counted over the whole packed slot of this rank) of slot `slot` lives under the TP-balanced
// placement.
__device__ __forceinline__ uint4 *tp_address(const TpPools &tp, int64_t slot, int64_t slot_stride4, uint32_t pv) {
  // both divisions by multiplication or shift: they sit in front of every 16-byte access
  const uint32_t unit = tp.unit_shift >= 0 ? pv >> tp.unit_shift : pv / tp.unit_vecs;
  const uint32_t in_unit = pv - unit * tp.unit_vecs;
  const uint32_t pos = tp.unit_begin + unit;
  const uint32_t owner = tp.width > 1 ? __umulhi(pos, tp.width_magic) >> tp.width_shift : pos;
  const uint32_t local = pos - owner * tp.width;
  return tp.base[owner] + slot * slot_stride4 + static_cast<int64_t>(local) * tp.unit_vecs + in_unit;
}

// grid = (ceil(R_max * vecs_per_unit / (kThreads*kUnroll)), n_layers, pairs).  A "vec" is 16 bytes of a row.  One
// layer per block row: the layer's first packed row and its count are per-block constants, the source address
// needs the dense row only, and a block past its layer's count leaves at once.
// pool_stride4: vectors between slots (Ragged, TpBalanced) or between (layer, slot) entries (Padded).
template <Layout LAYOUT>
__global__ void __launch_bounds__(kThreads, 8) pack_kernel(const uint4 *__restrict__ state, int64_t layer_stride4,
                                                           int64_t req_stride4, const int32_t *__restrict__ src_req,
                                                           uint4 *__restrict__ pool, int64_t pool_stride4,
                                                           int64_t n_slots, const int32_t *__restrict__ dst_slot,
                                                           const DascRowSrc *__restrict__ row_src,
                                                           const int32_t *__restrict__ layer_row_off,
                                                           uint32_t vecs_per_row, int32_t n_pairs,
                                                           const __grid_constant__ TpPools tp) {
  const uint32_t base = blockIdx.x * (kThreads * kUnroll) + threadIdx.x;
  const int32_t layer = blockIdx.y;
  const uint32_t first = static_cast<uint32_t>(__ldg(layer_row_off + layer));
  const uint32_t layer_vecs = (static_cast<uint32_t>(__ldg(layer_row_off + layer + 1)) - first) * vecs_per_row;
  if (blockIdx.x * (kThreads * kUnroll) >= layer_vecs) return;
  const int2 *src_l = reinterpret_cast<const int2 *>(row_src) + first;  // {layer, dense row} of the layer's packed rows
  for (int32_t pair = blockIdx.z; pair < n_pairs; pair += gridDim.z) {
    const uint4 *src_base = state + static_cast<int64_t>(__ldg(src_req + pair)) * req_stride4 + layer * layer_stride4;
    const int64_t slot = __ldg(dst_slot + pair);
    uint4 *dst_base = nullptr;
    if (LAYOUT == Layout::Ragged) dst_base = pool + slot * pool_stride4 + static_cast<int64_t>(first) * vecs_per_row;
    if (LAYOUT == Layout::Padded) dst_base = pool + (layer * n_slots + slot) * pool_stride4;
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
      if (i < layer_vecs) {
        if (LAYOUT == Layout::TpBalanced)
          st_stream(tp_address(tp, slot, pool_stride4, first * vecs_per_row + i), val[u]);
        else
          st_stream(dst_base + i, val[u]);
      }
    }
  }
}

// grid = (ceil(layer_vecs / (kThreads*kUnroll)), n_layers, pairs).
template <Layout LAYOUT>
__global__ void __launch_bounds__(kThreads) restore_kernel(const uint4 *__restrict__ pool, int64_t pool_stride4,
                                                           int64_t n_slots, const int32_t *__restrict__ src_slot,
                                                           uint4 *__restrict__ state, int64_t layer_stride4,
                                                           int64_t req_stride4, const int32_t *__restrict__ dst_req,
                                                           const int32_t *__restrict__ row_pos,
                                                           const int32_t *__restrict__ layer_row_off,
                                                           uint32_t layer_vecs, uint32_t rows_per_layer,
                                                           uint32_t vecs_per_row, int32_t n_pairs,
                                                           const __grid_constant__ TpPools tp) {
  const uint32_t base = blockIdx.x * (kThreads * kUnroll) + threadIdx.x;
  const int32_t layer = blockIdx.y;
  const int32_t *pos_l = row_pos + static_cast<int64_t>(layer) * rows_per_layer;
  // Padded: packed row of the layer's first retained row (positions inside an entry count from it)
  const int32_t first = LAYOUT == Layout::Padded ? __ldg(layer_row_off + layer) : 0;
  for (int32_t pair = blockIdx.z; pair < n_pairs; pair += gridDim.z) {
    const int64_t slot = __ldg(src_slot + pair);
    const uint4 *src_base = nullptr;
    if (LAYOUT == Layout::Ragged) src_base = pool + slot * pool_stride4;
    if (LAYOUT == Layout::Padded) src_base = pool + (layer * n_slots + slot) * pool_stride4;
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
        if (pos >= 0) {
          if (LAYOUT == Layout::TpBalanced)
            val[u] = ld_stream(tp_address(tp, slot, pool_stride4, static_cast<uint32_t>(pos) * vecs_per_row + vec));
          else
            val[u] = ld_stream(src_base + static_cast<int64_t>(pos - first) * vecs_per_row + vec);
        }
      }
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const uint32_t i = base + u * kThreads;
      if (i < layer_vecs) st_stream(dst_base + i, val[u]);
    }
  }
}

// dst[dst_idx[i]] = src[src_idx[i]] for blobs of `vecs` 16-byte vectors; grid = (ceil(vecs / (kThreads*kUnroll)), pairs).
__global__ void __launch_bounds__(kThreads) blob_copy_kernel(const uint4 *__restrict__ src, int64_t src_stride4,
                                                             const int32_t *__restrict__ src_idx,
                                                             uint4 *__restrict__ dst, int64_t dst_stride4,
                                                             const int32_t *__restrict__ dst_idx, uint32_t vecs,
                                                             int32_t n_pairs) {
  const uint32_t base = blockIdx.x * (kThreads * kUnroll) + threadIdx.x;
  for (int32_t pair = blockIdx.y; pair < n_pairs; pair += gridDim.y) {
    const uint4 *s = src + static_cast<int64_t>(__ldg(src_idx + pair)) * src_stride4;
    uint4 *d = dst + static_cast<int64_t>(__ldg(dst_idx + pair)) * dst_stride4;
    uint4 val[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const uint32_t i = base + u * kThreads;
      if (i < vecs) val[u] = ld_stream(s + i);
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const uint32_t i = base + u * kThreads;
      if (i < vecs) st_stream(d + i, val[u]);
    }
  }
}

TpPools make_tp(const DascTpPlacement *p, int64_t unit_floats) {
  TpPools tp{};
  if (p) {
    for (int r = 0; r < p->n_ranks; ++r) tp.base[r] = reinterpret_cast<uint4 *>(p->pool_base[r]);
    tp.unit_begin = static_cast<uint32_t>(p->unit_begin);
    tp.width = static_cast<uint32_t>(p->width);
    tp.unit_vecs = static_cast<uint32_t>(unit_floats / 4);
    tp.unit_shift = -1;
    for (int sft = 0; sft < 31; ++sft)
      if ((1u << sft) == tp.unit_vecs) tp.unit_shift = sft;
    if (tp.width > 1) {
      // division of a 31-bit number by `width`: with s = ceil(log2 width), m = floor(2^(31+s) / width) + 1 < 2^32 and
      // floor(pos / width) = (pos * m) >> (31 + s) for every pos < 2^31
      uint32_t sft = 0;
      while ((uint64_t{1} << sft) < tp.width) ++sft;
      tp.width_magic = static_cast<uint32_t>((uint64_t{1} << (31 + sft)) / tp.width + 1);
      tp.width_shift = sft - 1;
    }
  }
  return tp;
}

dim3 copy_grid(uint64_t vecs_per_layer, const dasc_plan_s *plan, int32_t n_pairs) {
  const uint32_t per_block = kThreads * kUnroll;
  return dim3(static_cast<uint32_t>((vecs_per_layer + per_block - 1) / per_block), static_cast<uint32_t>(plan->info.n_layers),
              static_cast<uint32_t>(n_pairs < 65535 ? n_pairs : 65535));
}

}  // namespace

// layout: 0 ragged (pool_stride = floats between slots), 1 padded (n_slots slots), 2 TP-balanced (`tp` set,
// pool_stride = floats between a rank's slots).
int dasc_launch_pack(const dasc_plan_s *plan, const float *state, int64_t layer_stride, int64_t req_stride,
                     const int32_t *src_req, float *pool, int64_t pool_stride, int64_t n_slots, const int32_t *dst_slot,
                     int32_t n_pairs, int layout, const DascTpPlacement *placement, void *stream) {
  const uint32_t vpr = static_cast<uint32_t>(plan->info.d_v / 4);
  if (plan->packed_rows == 0 || n_pairs == 0) return cudaSuccess;
  const int64_t rows_per_unit = plan->info.unit_floats / plan->info.d_v;
  const int64_t entry_stride4 = plan->info.r_max * rows_per_unit * vpr;  // vectors of the fullest layer
  const dim3 grid = copy_grid(static_cast<uint64_t>(entry_stride4), plan, n_pairs);
  const TpPools tp = make_tp(placement, plan->info.unit_floats);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const uint4 *st = reinterpret_cast<const uint4 *>(state);
  uint4 *pl = reinterpret_cast<uint4 *>(pool);
  if (layout == 0)
    pack_kernel<Layout::Ragged><<<grid, kThreads, 0, s>>>(st, layer_stride / 4, req_stride / 4, src_req, pl, pool_stride / 4, 0,
                                                          dst_slot, plan->d_row_src, plan->d_layer_row_off, vpr, n_pairs, tp);
  else if (layout == 1)
    pack_kernel<Layout::Padded><<<grid, kThreads, 0, s>>>(st, layer_stride / 4, req_stride / 4, src_req, pl, entry_stride4,
                                                          n_slots, dst_slot, plan->d_row_src, plan->d_layer_row_off, vpr,
                                                          n_pairs, tp);
  else
    pack_kernel<Layout::TpBalanced><<<grid, kThreads, 0, s>>>(st, layer_stride / 4, req_stride / 4, src_req, nullptr,
                                                              pool_stride / 4, 0, dst_slot, plan->d_row_src,
                                                              plan->d_layer_row_off, vpr, n_pairs, tp);
  return static_cast<int>(cudaGetLastError());
}

int dasc_launch_restore(const dasc_plan_s *plan, const float *pool, int64_t pool_stride, int64_t n_slots,
                        const int32_t *src_slot, float *state, int64_t layer_stride, int64_t req_stride,
                        const int32_t *dst_req, int32_t n_pairs, int layout, const DascTpPlacement *placement,
                        void *stream) {
  const uint32_t vpr = static_cast<uint32_t>(plan->info.d_v / 4);
  const uint64_t layer_vecs = static_cast<uint64_t>(plan->rows_per_layer) * vpr;
  if (n_pairs == 0) return cudaSuccess;
  const int64_t rows_per_unit = plan->info.unit_floats / plan->info.d_v;
  const int64_t entry_stride4 = plan->info.r_max * rows_per_unit * vpr;
  const dim3 grid = copy_grid(layer_vecs, plan, n_pairs);
  const TpPools tp = make_tp(placement, plan->info.unit_floats);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const uint4 *pl = reinterpret_cast<const uint4 *>(pool);
  uint4 *st = reinterpret_cast<uint4 *>(state);
  const uint32_t lv = static_cast<uint32_t>(layer_vecs), rpl = static_cast<uint32_t>(plan->rows_per_layer);
  if (layout == 0)
    restore_kernel<Layout::Ragged><<<grid, kThreads, 0, s>>>(pl, pool_stride / 4, 0, src_slot, st, layer_stride / 4,
                                                             req_stride / 4, dst_req, plan->d_row_pos,
                                                             plan->d_layer_row_off, lv, rpl, vpr, n_pairs, tp);
  else if (layout == 1)
    restore_kernel<Layout::Padded><<<grid, kThreads, 0, s>>>(pl, entry_stride4, n_slots, src_slot, st, layer_stride / 4,
                                                             req_stride / 4, dst_req, plan->d_row_pos,
                                                             plan->d_layer_row_off, lv, rpl, vpr, n_pairs, tp);
  else
    restore_kernel<Layout::TpBalanced><<<grid, kThreads, 0, s>>>(nullptr, pool_stride / 4, 0, src_slot, st, layer_stride / 4,
                                                                 req_stride / 4, dst_req, plan->d_row_pos,
                                                                 plan->d_layer_row_off, lv, rpl, vpr, n_pairs, tp);
  return static_cast<int>(cudaGetLastError());
}

int dasc_launch_blob_copy(const void *src, int64_t src_stride_bytes, const int32_t *src_idx, void *dst,
                          int64_t dst_stride_bytes, const int32_t *dst_idx, int64_t blob_bytes, int32_t n_pairs,
                          void *stream) {
  if (n_pairs == 0 || blob_bytes == 0) return cudaSuccess;
  const uint64_t vecs = static_cast<uint64_t>(blob_bytes / 16);
  const uint32_t per_block = kThreads * kUnroll;
  dim3 grid(static_cast<uint32_t>((vecs + per_block - 1) / per_block), static_cast<uint32_t>(n_pairs < 65535 ? n_pairs : 65535));
  blob_copy_kernel<<<grid, kThreads, 0, static_cast<cudaStream_t>(stream)>>>(
      reinterpret_cast<const uint4 *>(src), src_stride_bytes / 16, src_idx, reinterpret_cast<uint4 *>(dst),
      dst_stride_bytes / 16, dst_idx, static_cast<uint32_t>(vecs), n_pairs);
  return static_cast<int>(cudaGetLastError());
}
