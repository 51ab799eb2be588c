// C ABI of libdasc: argument validation and marshalling only; all work happens
// in plan_host.cpp (host plan) and in the CUDA kernels.
#include <cuda_runtime.h>
#include <nvtx3/nvToolsExt.h>

#include <algorithm>
#include <climits>
#include <cstdint>
#include <cstring>
#include <new>

#include "dasc_internal.h"

namespace {

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// A named range around each device call of the ABI, visible in a timeline when a profiler is attached (header-only
// NVTX: without a tool the calls do nothing).
struct TraceRange {
  explicit TraceRange(const char *name) { nvtxRangePushA(name); }
  ~TraceRange() { nvtxRangePop(); }
  TraceRange(const TraceRange &) = delete;
  TraceRange &operator=(const TraceRange &) = delete;
};

struct DeviceGuard {
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
    if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
  }
  ~DeviceGuard() {
    if (prev >= 0) cudaSetDevice(prev);
  }
};

template <typename T>
cudaError_t upload(T **dst, const T *src, size_t n) {
  *dst = nullptr;
  const size_t bytes = (n ? n : 1) * sizeof(T);
  cudaError_t e = cudaMalloc(reinterpret_cast<void **>(dst), bytes);
  if (e != cudaSuccess) return e;
  if (n) e = cudaMemcpy(*dst, src, n * sizeof(T), cudaMemcpyHostToDevice);
  return e;
}

void free_device_tables(dasc_plan_s *p) {
  if (p->info.device < 0) return;
  DeviceGuard guard(p->info.device);
  cudaFree(p->d_row_src);
  cudaFree(p->d_row_pos);
  cudaFree(p->d_row_keep);
  cudaFree(p->d_layer_row_off);
  p->d_layer_row_off = nullptr;
  p->d_row_src = nullptr;
  p->d_row_pos = nullptr;
  p->d_row_keep = nullptr;
}

// The plan's index tables live on plan->info.device; a launch from another current device would hand the kernel
// pointers of a GPU it may not be able to reach.
// Upload the index tables of a host plan to `device` (the only device allocation this library makes).
dasc_status_t attach_device(dasc_plan_s *p, int device) {
  DeviceGuard guard(device);
  if (!guard.ok) return DASC_ERR_CUDA;
  p->info.device = device;
  std::vector<uint8_t> keep(p->row_pos.size());
  for (size_t i = 0; i < keep.size(); ++i) keep[i] = p->row_pos[i] >= 0 ? 1 : 0;
  cudaError_t e = upload(&p->d_row_src, p->row_src.data(), p->row_src.size());
  if (e == cudaSuccess) e = upload(&p->d_row_pos, p->row_pos.data(), p->row_pos.size());
  if (e == cudaSuccess) e = upload(&p->d_row_keep, keep.data(), keep.size());
  // packed row at which each layer starts: o_l in rows (a GDN unit is d_k rows)
  const int64_t rows_per_unit = p->info.unit_floats / p->info.d_v;
  std::vector<int32_t> row_off(p->layer_offset.size());
  for (size_t l = 0; l < row_off.size(); ++l) row_off[l] = static_cast<int32_t>(p->layer_offset[l] * rows_per_unit);
  if (e == cudaSuccess) e = upload(&p->d_layer_row_off, row_off.data(), row_off.size());
  if (e != cudaSuccess) {
    free_device_tables(p);
    p->info.device = -1;
    return e == cudaErrorMemoryAllocation ? DASC_ERR_ALLOC : DASC_ERR_CUDA;
  }
  return DASC_OK;
}

dasc_status_t check_device(const dasc_plan_t *plan) {
  if (!plan || plan->info.device < 0) return DASC_ERR_INVALID_ARG;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return DASC_ERR_CUDA;
  return dev == plan->info.device ? DASC_OK : DASC_ERR_INVALID_ARG;
}

dasc_status_t check_copy_args(const dasc_plan_t *plan, const void *state, int64_t layer_stride, int64_t req_stride,
                              const void *idx_a, const void *pool, int64_t *slot_stride, const void *idx_b,
                              int32_t n_pairs, int64_t min_slot_floats = -1) {
  if (!plan) return DASC_ERR_INVALID_ARG;
  if (plan->info.device < 0) return DASC_ERR_INVALID_ARG;
  if (n_pairs < 0) return DASC_ERR_INVALID_ARG;
  if (n_pairs == 0) return DASC_OK;
  if (!state || !pool || !idx_a || !idx_b) return DASC_ERR_INVALID_ARG;
  if (!aligned16(state) || !aligned16(pool)) return DASC_ERR_INVALID_ARG;
  if (min_slot_floats < 0) min_slot_floats = plan->info.slot_floats;
  if (*slot_stride == 0) *slot_stride = min_slot_floats;
  if (layer_stride < 0 || req_stride < 0 || *slot_stride < min_slot_floats) return DASC_ERR_INVALID_ARG;
  if (plan->info.n_layers > 65535) return DASC_ERR_SHAPE;  // one block row of the copy grids per layer
  if (const dasc_status_t ds = check_device(plan); ds != DASC_OK) return ds;
  if (layer_stride % 4 || req_stride % 4 || *slot_stride % 4) return DASC_ERR_INVALID_ARG;
  if (plan->info.n_layers > 1 && layer_stride < plan->info.dense_floats_per_layer &&
      req_stride < plan->info.dense_floats_per_layer)
    return DASC_ERR_INVALID_ARG;  // layers of one request would overlap
  // 32-bit vector indices inside the kernels
  const int64_t vpr = plan->info.d_v / 4;
  if (plan->packed_rows * vpr >= (int64_t{1} << 31) || plan->rows_per_layer * vpr >= (int64_t{1} << 31))
    return DASC_ERR_SHAPE;
  return DASC_OK;
}

// first replayed token of each request: max(cu[r], cu[r+1] - window)
__global__ void window_begin_kernel(const int32_t *__restrict__ cu, int32_t n_req, int64_t window,
                                    int32_t *__restrict__ out) {
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r < n_req) {
    const int64_t lo = cu[r], hi = cu[r + 1];
    const int64_t b = hi - window;
    out[r] = static_cast<int32_t>(b > lo ? b : lo);
  }
}

}  // namespace

extern "C" {

dasc_status_t dasc_plan(const dasc_plan_desc_t *desc, int32_t device, dasc_plan_t **out) {
  if (!out) return DASC_ERR_INVALID_ARG;
  *out = nullptr;
  if (!desc) return DASC_ERR_INVALID_ARG;
  dasc_plan_s *p = new (std::nothrow) dasc_plan_s();
  if (!p) return DASC_ERR_ALLOC;
  dasc_status_t st;
  try {
    st = dasc_build_plan_host(desc, p);
  } catch (const std::bad_alloc &) {
    st = DASC_ERR_ALLOC;
  } catch (...) {
    st = DASC_ERR_INVALID_ARG;
  }
  if (st != DASC_OK) {
    delete p;
    return st;
  }
  if (device >= 0) {
    st = attach_device(p, device);
    if (st != DASC_OK) {
      delete p;
      return st;
    }
  }
  *out = p;
  return DASC_OK;
}

// Saved plan: a flat little-endian blob { magic, version, sizeof(info), info, horizon[n], window[n], mask[n] };
// everything else (layer counts, offsets, row tables) is re-derived from the mask when the blob is loaded.
static constexpr uint64_t kPlanMagic = 0x314E4C5043534144ull;  // "DASCPLN1"
struct PlanBlobHeader {
  uint64_t magic;
  uint32_t version, info_bytes;
  int64_t n_units;
};

dasc_status_t dasc_plan_save_bytes(const dasc_plan_t *plan, size_t *out) {
  if (!plan || !out) return DASC_ERR_INVALID_ARG;
  const size_t n = plan->mask.size();
  *out = sizeof(PlanBlobHeader) + sizeof(dasc_plan_info_t) + n * (sizeof(double) + sizeof(int64_t) + 1);
  return DASC_OK;
}

dasc_status_t dasc_plan_save(const dasc_plan_t *plan, void *buf, size_t buf_bytes) {
  size_t need = 0;
  if (dasc_plan_save_bytes(plan, &need) != DASC_OK || !buf || buf_bytes < need) return DASC_ERR_INVALID_ARG;
  const size_t n = plan->mask.size();
  unsigned char *w = static_cast<unsigned char *>(buf);
  const PlanBlobHeader h{kPlanMagic, 1u, static_cast<uint32_t>(sizeof(dasc_plan_info_t)), static_cast<int64_t>(n)};
  dasc_plan_info_t info = plan->info;
  info.device = -1;  // a saved plan belongs to no device
  std::memcpy(w, &h, sizeof h); w += sizeof h;
  std::memcpy(w, &info, sizeof info); w += sizeof info;
  std::memcpy(w, plan->horizon.data(), n * sizeof(double)); w += n * sizeof(double);
  std::memcpy(w, plan->window.data(), n * sizeof(int64_t)); w += n * sizeof(int64_t);
  std::memcpy(w, plan->mask.data(), n);
  return DASC_OK;
}

dasc_status_t dasc_plan_load(const void *buf, size_t bytes, int32_t device, dasc_plan_t **out) {
  if (!out) return DASC_ERR_INVALID_ARG;
  *out = nullptr;
  if (!buf || bytes < sizeof(PlanBlobHeader) + sizeof(dasc_plan_info_t)) return DASC_ERR_INVALID_ARG;
  const unsigned char *r = static_cast<const unsigned char *>(buf);
  PlanBlobHeader h;
  std::memcpy(&h, r, sizeof h); r += sizeof h;
  if (h.magic != kPlanMagic || h.version != 1u || h.info_bytes != sizeof(dasc_plan_info_t) || h.n_units < 0)
    return DASC_ERR_INVALID_ARG;
  dasc_plan_info_t info;
  std::memcpy(&info, r, sizeof info); r += sizeof info;
  // the shape fields must be sane and agree with one another and with the blob's length before anything is sized by them
  if (info.n_layers <= 0 || info.n_v_heads <= 0 || info.n_k_heads <= 0 || info.d_k <= 0 || info.d_v <= 0 || info.d_v % 4 ||
      (info.kind != DASC_KDA && info.kind != DASC_GDN) || info.n_v_heads % info.n_k_heads)
    return DASC_ERR_INVALID_ARG;
  const int64_t n_l = static_cast<int64_t>(info.n_v_heads) * (info.kind == DASC_KDA ? info.d_k : 1);
  const int64_t unit_floats = info.kind == DASC_KDA ? info.d_v : static_cast<int64_t>(info.d_k) * info.d_v;
  const int64_t n = n_l * info.n_layers;
  if (info.units_per_layer != n_l || info.unit_floats != unit_floats || info.units_total != n || h.n_units != n ||
      static_cast<int64_t>(info.n_v_heads) * info.d_k * info.n_layers >= INT32_MAX)
    return DASC_ERR_INVALID_ARG;
  const size_t need = sizeof(PlanBlobHeader) + sizeof(dasc_plan_info_t) + static_cast<size_t>(n) * (sizeof(double) + sizeof(int64_t) + 1);
  if (bytes < need) return DASC_ERR_INVALID_ARG;
  dasc_plan_s *p = new (std::nothrow) dasc_plan_s();
  if (!p) return DASC_ERR_ALLOC;
  try {
    p->info = info;
    p->info.device = -1;
    p->horizon.resize(n);
    p->window.resize(n);
    p->mask.resize(n);
    std::memcpy(p->horizon.data(), r, n * sizeof(double)); r += n * sizeof(double);
    std::memcpy(p->window.data(), r, n * sizeof(int64_t)); r += n * sizeof(int64_t);
    std::memcpy(p->mask.data(), r, n);
    p->layer_count.assign(info.n_layers, 0);
    p->layer_offset.assign(info.n_layers + 1, 0);
    int64_t r_max = 0;
    for (int64_t l = 0; l < info.n_layers; ++l) {
      int64_t c = 0;
      for (int64_t u = 0; u < n_l; ++u) {
        if (p->mask[l * n_l + u] > 1) throw 1;
        c += p->mask[l * n_l + u];
      }
      p->layer_count[l] = c;
      p->layer_offset[l + 1] = p->layer_offset[l] + c;
      r_max = std::max(r_max, c);
    }
    // the counts the blob claims must be those of its mask
    if (p->layer_offset[info.n_layers] != info.units_retained || r_max != info.r_max ||
        info.slot_floats != info.units_retained * unit_floats ||
        info.dense_floats_per_layer != static_cast<int64_t>(info.n_v_heads) * info.d_k * info.d_v)
      throw 1;
    dasc_plan_row_tables(p);
  } catch (const std::bad_alloc &) {
    delete p;
    return DASC_ERR_ALLOC;
  } catch (...) {
    delete p;
    return DASC_ERR_INVALID_ARG;
  }
  if (device >= 0) {
    const dasc_status_t st = attach_device(p, device);
    if (st != DASC_OK) {
      delete p;
      return st;
    }
  }
  *out = p;
  return DASC_OK;
}

void dasc_plan_destroy(dasc_plan_t *plan) {
  if (!plan) return;
  free_device_tables(plan);
  delete plan;
}

dasc_status_t dasc_plan_info(const dasc_plan_t *plan, dasc_plan_info_t *out) {
  if (!plan || !out) return DASC_ERR_INVALID_ARG;
  *out = plan->info;
  return DASC_OK;
}

#define DASC_COPY_OUT(field)                                                        \
  if (!plan || !out) return DASC_ERR_INVALID_ARG;                                   \
  std::memcpy(out, plan->field.data(), plan->field.size() * sizeof(plan->field[0])); \
  return DASC_OK;

dasc_status_t dasc_plan_horizon(const dasc_plan_t *plan, double *out) { DASC_COPY_OUT(horizon) }
dasc_status_t dasc_plan_mask(const dasc_plan_t *plan, uint8_t *out) { DASC_COPY_OUT(mask) }
dasc_status_t dasc_plan_window(const dasc_plan_t *plan, int64_t *out) { DASC_COPY_OUT(window) }
dasc_status_t dasc_plan_layer_counts(const dasc_plan_t *plan, int64_t *out) { DASC_COPY_OUT(layer_count) }
dasc_status_t dasc_plan_layer_offsets(const dasc_plan_t *plan, int64_t *out) { DASC_COPY_OUT(layer_offset) }
#undef DASC_COPY_OUT

dasc_status_t dasc_pack(const dasc_plan_t *plan, const float *state_base, int64_t layer_stride, int64_t req_stride,
                        const int32_t *src_req, float *pool_base, int64_t slot_stride, const int32_t *dst_slot,
                        int32_t n_pairs, void *cuda_stream) {
  TraceRange trace("dasc_pack");
  dasc_status_t st = check_copy_args(plan, state_base, layer_stride, req_stride, src_req, pool_base, &slot_stride,
                                     dst_slot, n_pairs);
  if (st != DASC_OK || n_pairs == 0) return st;
  const int e = dasc_launch_pack(plan, state_base, layer_stride, req_stride, src_req, pool_base, slot_stride, 0,
                                 dst_slot, n_pairs, 0, nullptr, cuda_stream);
  return e == 0 ? DASC_OK : DASC_ERR_CUDA;
}

dasc_status_t dasc_restore(const dasc_plan_t *plan, const float *pool_base, int64_t slot_stride,
                           const int32_t *src_slot, float *state_base, int64_t layer_stride, int64_t req_stride,
                           const int32_t *dst_req, int32_t n_pairs, void *cuda_stream) {
  TraceRange trace("dasc_restore");
  dasc_status_t st = check_copy_args(plan, state_base, layer_stride, req_stride, dst_req, pool_base, &slot_stride,
                                     src_slot, n_pairs);
  if (st != DASC_OK || n_pairs == 0) return st;
  const int e = dasc_launch_restore(plan, pool_base, slot_stride, 0, src_slot, state_base, layer_stride, req_stride,
                                    dst_req, n_pairs, 0, nullptr, cuda_stream);
  return e == 0 ? DASC_OK : DASC_ERR_CUDA;
}

dasc_status_t dasc_padded_pool_floats(const dasc_plan_t *plan, int64_t n_slots, int64_t *out) {
  if (!plan || !out || n_slots < 0) return DASC_ERR_INVALID_ARG;
  *out = static_cast<int64_t>(plan->info.n_layers) * n_slots * plan->info.r_max * plan->info.unit_floats;
  return DASC_OK;
}

dasc_status_t dasc_pack_padded(const dasc_plan_t *plan, const float *state_base, int64_t layer_stride,
                               int64_t req_stride, const int32_t *src_req, float *pool_base, int64_t n_slots,
                               const int32_t *dst_slot, int32_t n_pairs, void *cuda_stream) {
  TraceRange trace("dasc_pack_padded");
  int64_t unused = 0;
  dasc_status_t st = check_copy_args(plan, state_base, layer_stride, req_stride, src_req, pool_base, &unused, dst_slot,
                                     n_pairs);
  if (st != DASC_OK || n_pairs == 0) return st;
  if (n_slots <= 0) return DASC_ERR_INVALID_ARG;
  const int e = dasc_launch_pack(plan, state_base, layer_stride, req_stride, src_req, pool_base, 0, n_slots, dst_slot,
                                 n_pairs, 1, nullptr, cuda_stream);
  return e == 0 ? DASC_OK : DASC_ERR_CUDA;
}

dasc_status_t dasc_restore_padded(const dasc_plan_t *plan, const float *pool_base, int64_t n_slots,
                                  const int32_t *src_slot, float *state_base, int64_t layer_stride,
                                  int64_t req_stride, const int32_t *dst_req, int32_t n_pairs, void *cuda_stream) {
  TraceRange trace("dasc_restore_padded");
  int64_t unused = 0;
  dasc_status_t st = check_copy_args(plan, state_base, layer_stride, req_stride, dst_req, pool_base, &unused, src_slot,
                                     n_pairs);
  if (st != DASC_OK || n_pairs == 0) return st;
  if (n_slots <= 0) return DASC_ERR_INVALID_ARG;
  const int e = dasc_launch_restore(plan, pool_base, 0, n_slots, src_slot, state_base, layer_stride, req_stride,
                                    dst_req, n_pairs, 1, nullptr, cuda_stream);
  return e == 0 ? DASC_OK : DASC_ERR_CUDA;
}

dasc_status_t dasc_checkpoint_bytes(const dasc_plan_t *plan, int32_t layout, int64_t conv_bytes, int64_t *out) {
  if (!plan || !out || conv_bytes < 0) return DASC_ERR_INVALID_ARG;
  int64_t units;
  switch (layout) {
    case DASC_LAYOUT_RAGGED: units = plan->info.units_retained; break;
    case DASC_LAYOUT_PADDED: units = static_cast<int64_t>(plan->info.n_layers) * plan->info.r_max; break;
    case DASC_LAYOUT_DENSE: units = plan->info.units_total; break;
    default: return DASC_ERR_INVALID_ARG;
  }
  *out = units * plan->info.unit_floats * 4 + conv_bytes;
  return DASC_OK;
}

dasc_status_t dasc_slot_budget(int64_t budget_bytes, const int64_t *temporal_bytes_per_rank, int32_t n_ranks,
                               int64_t conv_bytes, int64_t *out) {
  if (!temporal_bytes_per_rank || !out || n_ranks <= 0 || budget_bytes < 0 || conv_bytes < 0)
    return DASC_ERR_INVALID_ARG;
  int64_t bottleneck = 0;
  for (int32_t r = 0; r < n_ranks; ++r) {
    if (temporal_bytes_per_rank[r] < 0) return DASC_ERR_INVALID_ARG;
    const int64_t b = temporal_bytes_per_rank[r] + conv_bytes;
    if (b > bottleneck) bottleneck = b;
  }
  if (bottleneck == 0) return DASC_ERR_INVALID_ARG;
  *out = budget_bytes / bottleneck - 1;  // slot 0 is reserved by the allocator
  return DASC_OK;
}

dasc_status_t dasc_tp_balance(const int64_t *units_per_rank, int32_t n_ranks, int64_t *slot_width,
                              int64_t *send_counts) {
  if (!units_per_rank || !slot_width || !send_counts || n_ranks <= 0) return DASC_ERR_INVALID_ARG;
  int64_t total = 0;
  for (int32_t r = 0; r < n_ranks; ++r) {
    if (units_per_rank[r] < 0) return DASC_ERR_INVALID_ARG;
    total += units_per_rank[r];
  }
  const int64_t width = (total + n_ranks - 1) / n_ranks;
  *slot_width = width;
  // rank r's units occupy global positions [begin, begin + U_r); rank s stores positions [s*width, (s+1)*width)
  int64_t begin = 0;
  for (int32_t r = 0; r < n_ranks; ++r) {
    const int64_t end = begin + units_per_rank[r];
    for (int32_t s = 0; s < n_ranks; ++s) {
      const int64_t lo = begin > s * width ? begin : s * width;
      const int64_t hi = end < (s + 1) * width ? end : (s + 1) * width;
      send_counts[static_cast<int64_t>(r) * n_ranks + s] = hi > lo ? hi - lo : 0;
    }
    begin = end;
  }
  return DASC_OK;
}

dasc_status_t dasc_tp_head_permutation(const dasc_plan_t *plan, int32_t n_ranks, int32_t heads_per_bundle,
                                       int32_t *perm, int64_t *units_per_rank) {
  if (!plan || !perm || !units_per_rank || n_ranks <= 0 || heads_per_bundle <= 0) return DASC_ERR_INVALID_ARG;
  const int32_t H = plan->info.n_v_heads, L = plan->info.n_layers;
  if (H % heads_per_bundle) return DASC_ERR_INVALID_ARG;
  const int32_t B = H / heads_per_bundle;
  if (B % n_ranks) return DASC_ERR_INVALID_ARG;
  const int32_t per_rank = B / n_ranks;
  const int64_t units_per_head = plan->info.units_per_layer / H;
  std::vector<int64_t> load(n_ranks, 0), weight(B);
  std::vector<int32_t> order(B), room(n_ranks), owner(B);
  for (int32_t l = 0; l < L; ++l) {
    const uint8_t *m = plan->mask.data() + static_cast<int64_t>(l) * plan->info.units_per_layer;
    for (int32_t b = 0; b < B; ++b) {
      int64_t w = 0;
      for (int64_t u = b * heads_per_bundle * units_per_head; u < (b + 1) * heads_per_bundle * units_per_head; ++u) w += m[u];
      weight[b] = w;
      order[b] = b;
    }
    // heaviest bundle first, lower index first among equals
    std::stable_sort(order.begin(), order.end(), [&](int32_t x, int32_t y) { return weight[x] > weight[y]; });
    std::fill(room.begin(), room.end(), per_rank);
    for (int32_t b : order) {
      int32_t best = -1;
      for (int32_t r = 0; r < n_ranks; ++r)
        if (room[r] > 0 && (best < 0 || load[r] < load[best])) best = r;
      owner[b] = best;
      --room[best];
      load[best] += weight[b];
    }
    // rank r holds positions [r * per_rank, (r + 1) * per_rank) of the permuted layer, its bundles in ascending index
    std::vector<int32_t> fill(n_ranks, 0);
    for (int32_t b = 0; b < B; ++b) {
      const int32_t r = owner[b];
      perm[static_cast<int64_t>(l) * B + r * per_rank + fill[r]++] = b;
    }
  }
  for (int32_t r = 0; r < n_ranks; ++r) units_per_rank[r] = load[r];
  return DASC_OK;
}

// Shared validation of the TP-balanced copies; fills `pl` and the slot stride.
static dasc_status_t check_tp_args(const dasc_plan_t *plan, float *const *pool_bases, const int64_t *units_per_rank,
                                   int32_t n_ranks, int32_t rank, int64_t *slot_stride, DascTpPlacement *pl) {
  if (!plan || !pool_bases || !units_per_rank) return DASC_ERR_INVALID_ARG;
  if (n_ranks <= 0 || n_ranks > DASC_TP_MAX_RANKS || rank < 0 || rank >= n_ranks) return DASC_ERR_INVALID_ARG;
  int64_t total = 0, begin = 0;
  for (int32_t r = 0; r < n_ranks; ++r) {
    if (units_per_rank[r] < 0) return DASC_ERR_INVALID_ARG;
    if (r < rank) begin += units_per_rank[r];
    total += units_per_rank[r];
    if (!pool_bases[r] || !aligned16(pool_bases[r])) return DASC_ERR_INVALID_ARG;
    pl->pool_base[r] = pool_bases[r];
  }
  if (units_per_rank[rank] != plan->info.units_retained) return DASC_ERR_INVALID_ARG;  // U_r is this plan's payload
  if (total >= (int64_t{1} << 31)) return DASC_ERR_SHAPE;
  pl->n_ranks = n_ranks;
  pl->unit_begin = begin;
  pl->width = total > 0 ? (total + n_ranks - 1) / n_ranks : 1;
  const int64_t min_stride = pl->width * plan->info.unit_floats;
  if (*slot_stride == 0) *slot_stride = min_stride;
  if (*slot_stride < min_stride || *slot_stride % 4) return DASC_ERR_INVALID_ARG;
  return DASC_OK;
}

dasc_status_t dasc_pack_tp(const dasc_plan_t *plan, const float *state_base, int64_t layer_stride, int64_t req_stride,
                           const int32_t *src_req, float *const *pool_bases, const int64_t *units_per_rank,
                           int32_t n_ranks, int32_t rank, int64_t slot_stride, const int32_t *dst_slot,
                           int32_t n_pairs, void *cuda_stream) {
  TraceRange trace("dasc_pack_tp");
  DascTpPlacement pl{};
  dasc_status_t st = check_tp_args(plan, pool_bases, units_per_rank, n_ranks, rank, &slot_stride, &pl);
  if (st != DASC_OK) return st;
  int64_t stride_ok = slot_stride;  // the per-rank slot rule was checked above; the common rules follow
  st = check_copy_args(plan, state_base, layer_stride, req_stride, src_req, pool_bases[0], &stride_ok, dst_slot, n_pairs, 0);
  if (st != DASC_OK || n_pairs == 0) return st;
  const int e = dasc_launch_pack(plan, state_base, layer_stride, req_stride, src_req, nullptr, slot_stride, 0, dst_slot,
                                 n_pairs, 2, &pl, cuda_stream);
  return e == 0 ? DASC_OK : DASC_ERR_CUDA;
}

dasc_status_t dasc_restore_tp(const dasc_plan_t *plan, float *const *pool_bases, const int64_t *units_per_rank,
                              int32_t n_ranks, int32_t rank, int64_t slot_stride, const int32_t *src_slot,
                              float *state_base, int64_t layer_stride, int64_t req_stride, const int32_t *dst_req,
                              int32_t n_pairs, void *cuda_stream) {
  TraceRange trace("dasc_restore_tp");
  DascTpPlacement pl{};
  dasc_status_t st = check_tp_args(plan, pool_bases, units_per_rank, n_ranks, rank, &slot_stride, &pl);
  if (st != DASC_OK) return st;
  int64_t stride_ok = slot_stride;
  st = check_copy_args(plan, state_base, layer_stride, req_stride, dst_req, pool_bases[0], &stride_ok, src_slot, n_pairs, 0);
  if (st != DASC_OK || n_pairs == 0) return st;
  const int e = dasc_launch_restore(plan, nullptr, slot_stride, 0, src_slot, state_base, layer_stride, req_stride,
                                    dst_req, n_pairs, 2, &pl, cuda_stream);
  return e == 0 ? DASC_OK : DASC_ERR_CUDA;
}

static dasc_status_t conv_copy(const void *src, int64_t src_stride, const int32_t *src_idx, void *dst, int64_t dst_stride,
                               const int32_t *dst_idx, int64_t conv_bytes, int32_t n_pairs, void *cuda_stream) {
  if (n_pairs < 0 || conv_bytes < 0) return DASC_ERR_INVALID_ARG;
  if (n_pairs == 0 || conv_bytes == 0) return DASC_OK;
  if (!src || !dst || !src_idx || !dst_idx || !aligned16(src) || !aligned16(dst)) return DASC_ERR_INVALID_ARG;
  if (conv_bytes % 16 || src_stride % 16 || dst_stride % 16 || src_stride < conv_bytes || dst_stride < conv_bytes)
    return DASC_ERR_INVALID_ARG;
  if (conv_bytes / 16 >= (int64_t{1} << 31)) return DASC_ERR_SHAPE;
  const int e = dasc_launch_blob_copy(src, src_stride, src_idx, dst, dst_stride, dst_idx, conv_bytes, n_pairs, cuda_stream);
  return e == 0 ? DASC_OK : DASC_ERR_CUDA;
}

dasc_status_t dasc_conv_store(const void *conv_base, int64_t req_stride_bytes, const int32_t *src_req, void *pool_base,
                              int64_t slot_stride_bytes, const int32_t *dst_slot, int64_t conv_bytes, int32_t n_pairs,
                              void *cuda_stream) {
  return conv_copy(conv_base, req_stride_bytes, src_req, pool_base, slot_stride_bytes, dst_slot, conv_bytes, n_pairs,
                   cuda_stream);
}

dasc_status_t dasc_conv_load(const void *pool_base, int64_t slot_stride_bytes, const int32_t *src_slot, void *conv_base,
                             int64_t req_stride_bytes, const int32_t *dst_req, int64_t conv_bytes, int32_t n_pairs,
                             void *cuda_stream) {
  return conv_copy(pool_base, slot_stride_bytes, src_slot, conv_base, req_stride_bytes, dst_req, conv_bytes, n_pairs,
                   cuda_stream);
}

static int64_t int8_slot_bytes(const dasc_plan_t *plan) {
  const int64_t raw = plan->packed_rows * (plan->info.d_v + 4);
  return (raw + 15) / 16 * 16;
}

static dasc_status_t check_int8_args(const dasc_plan_t *plan, const void *state, int64_t layer_stride,
                                     int64_t req_stride, const void *idx_a, const void *pool,
                                     int64_t *slot_stride_bytes, const void *idx_b, int32_t n_pairs) {
  int64_t fp32_stride = 0;  // the fp32 slot rule does not apply; everything else does
  dasc_status_t st = check_copy_args(plan, state, layer_stride, req_stride, idx_a, pool, &fp32_stride, idx_b, n_pairs);
  if (st != DASC_OK || n_pairs == 0) return st;
  const int64_t d_v = plan->info.d_v;
  if (d_v < 4 || d_v > 128 || (d_v & (d_v - 1))) return DASC_ERR_SHAPE;
  if (*slot_stride_bytes == 0) *slot_stride_bytes = int8_slot_bytes(plan);
  if (*slot_stride_bytes < int8_slot_bytes(plan) || *slot_stride_bytes % 16) return DASC_ERR_INVALID_ARG;
  return DASC_OK;
}

dasc_status_t dasc_int8_slot_bytes(const dasc_plan_t *plan, size_t *out) {
  if (!plan || !out) return DASC_ERR_INVALID_ARG;
  *out = static_cast<size_t>(int8_slot_bytes(plan));
  return DASC_OK;
}

dasc_status_t dasc_pack_int8(const dasc_plan_t *plan, const float *state_base, int64_t layer_stride,
                             int64_t req_stride, const int32_t *src_req, void *pool_base, int64_t slot_stride_bytes,
                             const int32_t *dst_slot, int32_t n_pairs, void *cuda_stream) {
  TraceRange trace("dasc_pack_int8");
  dasc_status_t st = check_int8_args(plan, state_base, layer_stride, req_stride, src_req, pool_base,
                                     &slot_stride_bytes, dst_slot, n_pairs);
  if (st != DASC_OK || n_pairs == 0) return st;
  const int e = dasc_launch_pack_int8(plan, state_base, layer_stride, req_stride, src_req, pool_base,
                                      slot_stride_bytes, dst_slot, n_pairs, cuda_stream);
  return e == 0 ? DASC_OK : DASC_ERR_CUDA;
}

dasc_status_t dasc_restore_int8(const dasc_plan_t *plan, const void *pool_base, int64_t slot_stride_bytes,
                                const int32_t *src_slot, float *state_base, int64_t layer_stride, int64_t req_stride,
                                const int32_t *dst_req, int32_t n_pairs, void *cuda_stream) {
  TraceRange trace("dasc_restore_int8");
  dasc_status_t st = check_int8_args(plan, state_base, layer_stride, req_stride, dst_req, pool_base,
                                     &slot_stride_bytes, src_slot, n_pairs);
  if (st != DASC_OK || n_pairs == 0) return st;
  const int e = dasc_launch_restore_int8(plan, pool_base, slot_stride_bytes, src_slot, state_base, layer_stride,
                                         req_stride, dst_req, n_pairs, cuda_stream);
  return e == 0 ? DASC_OK : DASC_ERR_CUDA;
}

static bool chunked_shape_ok(const dasc_plan_t *plan) { return plan->info.d_k == 128 && plan->info.d_v == 128; }

dasc_status_t dasc_refresh_workspace_bytes(const dasc_plan_t *plan, int32_t n_req, int32_t n_layers_in_call,
                                           int32_t algo, size_t *out) {
  if (!plan || !out || n_req < 0 || n_layers_in_call < 0) return DASC_ERR_INVALID_ARG;
  if (algo != DASC_ALGO_AUTO && algo != DASC_ALGO_SEQUENTIAL && algo != DASC_ALGO_CHUNKED) return DASC_ERR_INVALID_ARG;
  const bool chunked = algo == DASC_ALGO_CHUNKED || (algo == DASC_ALGO_AUTO && chunked_shape_ok(plan));
  *out = chunked ? dasc_refresh_chunked_workspace_bytes(n_req, n_layers_in_call, plan->info.n_v_heads) : 0;
  return DASC_OK;
}

namespace {

// What a validated refresh request boils down to.
struct RefreshRequest {
  DascRefreshArgs args{};
  bool nothing_to_do = false;
  bool chunked = false;  // the tensor-core kernel takes part
  int32_t algo = DASC_ALGO_AUTO;
};

// Every argument check of dasc_refresh / dasc_refresh_window, before anything is launched.
// tok_begin: device array of first tokens (null = cu_seqlens[r]).  q may be null when o is null.
dasc_status_t refresh_validate(const dasc_plan_t *plan, float *state_base, int64_t layer_stride, int64_t req_stride,
                               const int32_t *req_idx, const void *q, const void *k, const void *v, int32_t io_dtype,
                               const float *g, const float *beta, const int32_t *cu_seqlens, const int32_t *tok_begin,
                               int32_t n_req, int64_t total_tokens, int32_t max_seqlen, int32_t layer_begin,
                               int32_t layer_end, float q_scale, void *o, int32_t o_dtype, int32_t mode, int32_t algo,
                               void *workspace, size_t workspace_bytes, RefreshRequest *out) {
  if (!plan || plan->info.device < 0) return DASC_ERR_INVALID_ARG;
  if (!q && !o) q = k;  // never read for its values: the kernels skip or discard the output side
  if (n_req < 0 || total_tokens < 0 || max_seqlen < 0) return DASC_ERR_INVALID_ARG;
  if (layer_begin < 0 || layer_end < layer_begin || layer_end > plan->info.n_layers) return DASC_ERR_INVALID_ARG;
  if (io_dtype != DASC_IO_BF16 && io_dtype != DASC_IO_FP32) return DASC_ERR_INVALID_ARG;
  if (o && o_dtype != DASC_IO_BF16 && o_dtype != DASC_IO_FP32) return DASC_ERR_INVALID_ARG;
  if (mode != DASC_REFRESH_CONTINUE && mode != DASC_REFRESH_SCRATCH_MERGE_LOCAL) return DASC_ERR_INVALID_ARG;
  if (algo != DASC_ALGO_AUTO && algo != DASC_ALGO_SEQUENTIAL && algo != DASC_ALGO_CHUNKED) return DASC_ERR_INVALID_ARG;
  if (n_req == 0 || layer_end == layer_begin || total_tokens == 0) {
    out->nothing_to_do = true;
    return DASC_OK;
  }
  if (!state_base || !req_idx || !q || !k || !v || !g || !beta || !cu_seqlens) return DASC_ERR_INVALID_ARG;
  if (!aligned16(state_base) || !aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(g) ||
      (o && !aligned16(o)))
    return DASC_ERR_INVALID_ARG;
  if (layer_stride < 0 || req_stride < 0 || layer_stride % 4 || req_stride % 4) return DASC_ERR_INVALID_ARG;
  const size_t esz = io_dtype == DASC_IO_BF16 ? 2 : 4;
  if ((plan->info.d_k * esz) % 16 || (plan->info.d_v * esz) % 16) return DASC_ERR_SHAPE;
  if (const dasc_status_t ds = check_device(plan); ds != DASC_OK) return ds;

  // the chunked kernel takes d_k = d_v = 128 and bf16 token streams
  const bool chunked_ok = chunked_shape_ok(plan) && io_dtype == DASC_IO_BF16;
  if (algo == DASC_ALGO_CHUNKED && !chunked_ok) return DASC_ERR_SHAPE;
  out->chunked = algo == DASC_ALGO_CHUNKED || (algo == DASC_ALGO_AUTO && chunked_ok);
  out->algo = algo;

  DascRefreshArgs &a = out->args;
  a.kind = plan->info.kind;
  a.H_v = plan->info.n_v_heads;
  a.H_k = plan->info.n_k_heads;
  a.d_k = plan->info.d_k;
  a.d_v = plan->info.d_v;
  a.state = state_base;
  a.layer_stride = layer_stride;
  a.req_stride = req_stride;
  a.req_idx = req_idx;
  a.q = q;
  a.k = k;
  a.v = v;
  a.io_bf16 = io_dtype == DASC_IO_BF16;
  a.g = g;
  a.beta = beta;
  a.cu_seqlens = cu_seqlens;
  a.tok_begin = tok_begin;
  a.n_req = n_req;
  a.total_tokens = total_tokens;
  a.max_seqlen = max_seqlen;
  a.layer_begin = layer_begin;
  a.n_layers_in_call = layer_end - layer_begin;
  a.q_scale = q_scale;
  a.o = o;
  a.o_bf16 = o_dtype == DASC_IO_BF16;
  a.mode = mode;
  a.row_keep = plan->d_row_keep;
  a.rows_per_layer = plan->rows_per_layer;
  a.workspace = workspace;
  a.workspace_bytes = workspace_bytes;
  a.short_thr = -1;
  if (out->chunked) {
    const size_t need = dasc_refresh_chunked_workspace_bytes(n_req, a.n_layers_in_call, a.H_v);
    if (!workspace || workspace_bytes < need || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return DASC_ERR_WORKSPACE;
    a.unit_list = reinterpret_cast<int32_t *>(static_cast<unsigned char *>(workspace) + kRefreshWsHeader);
    a.unit_list_cap = static_cast<int32_t>((need - kRefreshWsHeader) / sizeof(int32_t));
  }
  return DASC_OK;
}

// AUTO with a shape the tensor-core kernel takes: that kernel replays every unit inside its range and at least
// kShortSuffix + 1 tokens long and lists the others; the exact kernel then walks the list on the same stream, from
// stored states the first kernel has not touched.  CHUNKED runs the tensor-core kernel alone (a unit outside its
// range is left unwritten, listed and reported); SEQUENTIAL the exact kernel alone.
dasc_status_t refresh_launch(const RefreshRequest &rq, void *cuda_stream) {
  if (rq.nothing_to_do) return DASC_OK;
  DascRefreshArgs a = rq.args;
  int e;
  if (!rq.chunked) {
    e = dasc_launch_refresh_seq(a, cuda_stream);
  } else if (rq.algo == DASC_ALGO_CHUNKED) {
    a.domain_is_error = 1;
    e = dasc_launch_refresh_chunked(a, cuda_stream);
    if (e == -1) return DASC_ERR_UNSUPPORTED;
  } else {
    a.short_thr = kShortSuffix;
    e = dasc_launch_refresh_chunked(a, cuda_stream);
    if (e == 0) {
      a.from_list = 1;
      e = dasc_launch_refresh_seq(a, cuda_stream);
    }
  }
  if (e == -1) return DASC_ERR_SHAPE;
  return e == 0 ? DASC_OK : DASC_ERR_CUDA;
}

}  // namespace

dasc_status_t dasc_refresh(const dasc_plan_t *plan, float *state_base, int64_t layer_stride, int64_t req_stride,
                           const int32_t *req_idx, const void *q, const void *k, const void *v, int32_t io_dtype,
                           const float *g, const float *beta, const int32_t *cu_seqlens, int32_t n_req,
                           int64_t total_tokens, int32_t max_seqlen, int32_t layer_begin, int32_t layer_end,
                           float q_scale, void *o, int32_t o_dtype, int32_t mode, int32_t algo, void *workspace,
                           size_t workspace_bytes, void *cuda_stream) {
  TraceRange trace("dasc_refresh");
  if (!q) return n_req == 0 || total_tokens == 0 || layer_end == layer_begin ? DASC_OK : DASC_ERR_INVALID_ARG;
  RefreshRequest rq;
  const dasc_status_t st = refresh_validate(plan, state_base, layer_stride, req_stride, req_idx, q, k, v, io_dtype, g,
                                            beta, cu_seqlens, nullptr, n_req, total_tokens, max_seqlen, layer_begin,
                                            layer_end, q_scale, o, o_dtype, mode, algo, workspace, workspace_bytes, &rq);
  if (st != DASC_OK) return st;
  return refresh_launch(rq, cuda_stream);
}

dasc_status_t dasc_refresh_window(const dasc_plan_t *plan, float *state_base, int64_t layer_stride,
                                  int64_t req_stride, const int32_t *req_idx, const void *q, const void *k,
                                  const void *v, int32_t io_dtype, const float *g, const float *beta,
                                  const int32_t *cu_seqlens, int32_t n_req, int64_t total_tokens, int64_t window,
                                  int32_t layer_begin, int32_t layer_end, float q_scale, void *o, int32_t o_dtype,
                                  int32_t algo, int32_t *window_begin, void *workspace, size_t workspace_bytes,
                                  void *cuda_stream) {
  TraceRange trace("dasc_refresh_window");
  if (!plan || plan->info.device < 0 || n_req < 0) return DASC_ERR_INVALID_ARG;
  if (o && !q) return DASC_ERR_INVALID_ARG;
  if (window <= 0) window = plan->info.w_replay;
  if (n_req == 0) return DASC_OK;
  if (!cu_seqlens || !window_begin) return DASC_ERR_INVALID_ARG;
  if (window > INT32_MAX) window = INT32_MAX;
  // every check comes before the first launch: an argument error leaves window_begin untouched as well
  RefreshRequest rq;
  const dasc_status_t st =
      refresh_validate(plan, state_base, layer_stride, req_stride, req_idx, q, k, v, io_dtype, g, beta, cu_seqlens,
                       window_begin, n_req, total_tokens, static_cast<int32_t>(window), layer_begin, layer_end, q_scale, o,
                       o_dtype, DASC_REFRESH_SCRATCH_MERGE_LOCAL, algo, workspace, workspace_bytes, &rq);
  if (st != DASC_OK) return st;
  if (const dasc_status_t ds = check_device(plan); ds != DASC_OK) return ds;
  window_begin_kernel<<<(n_req + 255) / 256, 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(cu_seqlens, n_req, window,
                                                                                               window_begin);
  if (cudaGetLastError() != cudaSuccess) return DASC_ERR_CUDA;
  if (window == 0) return DASC_OK;  // nothing is omitted, so nothing needs a refresh
  return refresh_launch(rq, cuda_stream);
}

dasc_status_t dasc_refresh_status(const void *workspace, size_t workspace_bytes) {
  if (!workspace || workspace_bytes < 4) return DASC_OK;  // nothing was recorded
  uint32_t flag[2] = {0, 0};  // [0] a wait timed out, [1] log-decay out of range and not replayed
  if (cudaMemcpy(flag, workspace, workspace_bytes < 8 ? 4 : 8, cudaMemcpyDeviceToHost) != cudaSuccess) return DASC_ERR_CUDA;
  if (flag[0] != 0) return DASC_ERR_TIMEOUT;
  return flag[1] == 0 ? DASC_OK : DASC_ERR_DOMAIN;
}

dasc_status_t dasc_refresh_counters(const void *workspace, size_t workspace_bytes, int32_t *handed_over,
                                    int32_t *replayed_exactly) {
  if (!workspace || workspace_bytes < 16 || !handed_over || !replayed_exactly) return DASC_ERR_INVALID_ARG;
  uint32_t w[4] = {0, 0, 0, 0};
  if (cudaMemcpy(w, workspace, 16, cudaMemcpyDeviceToHost) != cudaSuccess) return DASC_ERR_CUDA;
  *handed_over = static_cast<int32_t>(w[2]);
  *replayed_exactly = static_cast<int32_t>(w[3]);
  return DASC_OK;
}

void dasc_debug_set_refresh_poll_limit(uint32_t polls) { __atomic_store_n(&g_dasc_debug_poll_limit, polls, __ATOMIC_RELAXED); }

const char *dasc_status_string(dasc_status_t s) {
  switch (s) {
    case DASC_OK: return "ok";
    case DASC_ERR_INVALID_ARG: return "invalid argument";
    case DASC_ERR_SHAPE: return "unsupported shape";
    case DASC_ERR_UNSUPPORTED: return "not implemented";
    case DASC_ERR_ALLOC: return "allocation failed";
    case DASC_ERR_CUDA: return "CUDA error";
    case DASC_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case DASC_ERR_TIMEOUT: return "device-side wait timed out";
    case DASC_ERR_DOMAIN: return "log-decay outside the chunked kernel's range";
  }
  return "unknown status";
}

const char *dasc_version(void) { return "0.1.0"; }

}  // extern "C"
