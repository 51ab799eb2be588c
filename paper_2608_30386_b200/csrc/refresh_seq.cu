// Suffix refresh, sequential form: the gated delta rule (Eq. 1, transposed
// orientation) replayed token by token in fp32 on the CUDA cores.  Exact for any
// log-decay g <= 0; it is the reference point for the chunked tensor-core kernel
// and the path for shapes that kernel does not take.
//
// One CTA per (request, layer, value head).  The d_k x d_v state lives in
// registers: thread (s, v) owns column v of row slice s (DK/RS rows).  Per token
//   S   <- Diag(alpha_t) S                       (decay on the key-channel index)
//   r   <- S^T k_t                               (reduced over the row slices via shared memory)
//   u   <- beta_t (v_t - r)
//   S   <- S + k_t u^T
//   o_t <- q_scale * S^T q_t
// Token inputs are staged TB tokens at a time: raw rows by cp.async into a double
// buffer, then converted once (bf16 -> fp32, alpha = exp(g)) for all threads.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "dasc_internal.h"

namespace {

constexpr int TB = 16;  // tokens staged per group

__device__ __forceinline__ void cp_async16(void *smem, const void *gmem) {
  const uint32_t s = static_cast<uint32_t>(__cvta_generic_to_shared(smem));
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(s), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async4(void *smem, const void *gmem) {
  const uint32_t s = static_cast<uint32_t>(__cvta_generic_to_shared(smem));
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(s), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

template <typename IO>
__device__ __forceinline__ float io_to_float(IO x);
template <>
__device__ __forceinline__ float io_to_float<float>(float x) { return x; }
template <>
__device__ __forceinline__ float io_to_float<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }

template <typename IO>
__device__ __forceinline__ IO float_to_io(float x);
template <>
__device__ __forceinline__ float float_to_io<float>(float x) { return x; }
template <>
__device__ __forceinline__ __nv_bfloat16 float_to_io<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

template <int DK, int DV, typename IO, bool KDA>
struct SeqSmem {
  // raw staging, double buffered
  alignas(16) IO q[2][TB][DK];
  alignas(16) IO k[2][TB][DK];
  alignas(16) IO v[2][TB][DV];
  alignas(16) float g[2][TB][KDA ? DK : 4];
  alignas(16) float beta[2][TB];
  // converted, current group
  alignas(16) float kf[TB][DK];
  alignas(16) float qf[TB][DK];
  alignas(16) float af[TB][DK];
  alignas(16) float vf[TB][DV];
  float bf[TB];
};

// One (request, layer, value head) unit, replayed by the whole CTA.
template <int DK, int DV, int RS, typename IO, typename OT, bool KDA>
__device__ __forceinline__ void seq_unit(const DascRefreshArgs &a, int unit, unsigned char *smem_raw) {
  constexpr int NT = DV * RS;
  constexpr int ROWS = DK / RS;  // rows of the state held by one thread
  using Smem = SeqSmem<DK, DV, IO, KDA>;
  Smem &sm = *reinterpret_cast<Smem *>(smem_raw);
  // partial sums across row slices, double buffered by token parity
  float(*red_r)[RS][DV] = reinterpret_cast<float(*)[RS][DV]>(smem_raw + sizeof(Smem));
  float(*red_o)[RS][DV] = red_r + 2;

  const int tid = threadIdx.x;
  const int v_col = tid % DV;
  const int slice = tid / DV;
  const int row0 = slice * ROWS;

  const int h = unit % a.H_v;
  const int lc = (unit / a.H_v) % a.n_layers_in_call;
  const int r = unit / (a.H_v * a.n_layers_in_call);
  const int hk = h / (a.H_v / a.H_k);
  const int layer = a.layer_begin + lc;
  const int64_t t_begin = a.tok_begin ? a.tok_begin[r] : a.cu_seqlens[r];
  const int n_tok = static_cast<int>(a.cu_seqlens[r + 1] - t_begin);
  // An empty suffix continues nothing; in the scratch mode it still replaces the omitted
  // units by the (all-zero) scratch state, as the definition says.
  if (n_tok <= 0 && a.mode == DASC_REFRESH_CONTINUE) return;

  float *st = a.state + static_cast<int64_t>(a.req_idx[r]) * a.req_stride + static_cast<int64_t>(layer) * a.layer_stride +
              static_cast<int64_t>(h) * DK * DV;
  float S[ROWS];
  if (a.mode == DASC_REFRESH_CONTINUE) {
#pragma unroll
    for (int i = 0; i < ROWS; ++i) S[i] = st[(row0 + i) * DV + v_col];
  } else {
#pragma unroll
    for (int i = 0; i < ROWS; ++i) S[i] = 0.f;
  }

  const int64_t tok0 = static_cast<int64_t>(lc) * a.total_tokens + t_begin;
  const IO *gq = static_cast<const IO *>(a.q) + (tok0 * a.H_k + hk) * DK;
  const IO *gk = static_cast<const IO *>(a.k) + (tok0 * a.H_k + hk) * DK;
  const IO *gv = static_cast<const IO *>(a.v) + (tok0 * a.H_v + h) * DV;
  const float *gg = a.g + (tok0 * a.H_v + h) * (KDA ? DK : 1);
  const float *gb = a.beta + tok0 * a.H_v + h;
  OT *go = a.o ? static_cast<OT *>(a.o) + (tok0 * a.H_v + h) * DV : nullptr;
  const int64_t qk_stride = static_cast<int64_t>(a.H_k) * DK, v_stride = static_cast<int64_t>(a.H_v) * DV;
  const int64_t g_stride = static_cast<int64_t>(a.H_v) * (KDA ? DK : 1), b_stride = a.H_v;

  auto stage = [&](int grp, int buf) {
    const int t_lo = grp * TB;
    const int cnt = min(TB, n_tok - t_lo);
    constexpr int QV = DK * sizeof(IO) / 16, VV = DV * sizeof(IO) / 16, GV = KDA ? DK * 4 / 16 : 1;
    for (int i = tid; i < cnt * QV; i += NT) {
      const int t = i / QV, j = i % QV;
      cp_async16(reinterpret_cast<char *>(&sm.q[buf][t][0]) + j * 16,
                 reinterpret_cast<const char *>(gq + (t_lo + t) * qk_stride) + j * 16);
      cp_async16(reinterpret_cast<char *>(&sm.k[buf][t][0]) + j * 16,
                 reinterpret_cast<const char *>(gk + (t_lo + t) * qk_stride) + j * 16);
    }
    for (int i = tid; i < cnt * VV; i += NT) {
      const int t = i / VV, j = i % VV;
      cp_async16(reinterpret_cast<char *>(&sm.v[buf][t][0]) + j * 16,
                 reinterpret_cast<const char *>(gv + (t_lo + t) * v_stride) + j * 16);
    }
    if constexpr (KDA) {
      for (int i = tid; i < cnt * GV; i += NT) {
        const int t = i / GV, j = i % GV;
        cp_async16(reinterpret_cast<char *>(&sm.g[buf][t][0]) + j * 16,
                   reinterpret_cast<const char *>(gg + (t_lo + t) * g_stride) + j * 16);
      }
    } else {
      for (int t = tid; t < cnt; t += NT) cp_async4(&sm.g[buf][t][0], gg + (t_lo + t) * g_stride);
    }
    for (int t = tid; t < cnt; t += NT) cp_async4(&sm.beta[buf][t], gb + (t_lo + t) * b_stride);
    cp_async_commit();
  };

  const int n_grp = n_tok > 0 ? (n_tok + TB - 1) / TB : 0;
  if (n_grp > 0) stage(0, 0);
  int parity = 0;  // token parity for the reduction buffers
  bool have_prev_o = false;
  int prev_t = 0;
  for (int grp = 0; grp < n_grp; ++grp) {
    const int buf = grp & 1;
    const int t_lo = grp * TB;
    const int cnt = min(TB, n_tok - t_lo);
    cp_async_wait_all();
    __syncthreads();  // raw[buf] landed; everyone is past the previous group's converted buffers
    if (grp + 1 < n_grp) stage(grp + 1, buf ^ 1);
    for (int i = tid; i < cnt * DK; i += NT) {
      const int t = i / DK, c = i % DK;
      sm.kf[t][c] = io_to_float<IO>(sm.k[buf][t][c]);
      sm.qf[t][c] = io_to_float<IO>(sm.q[buf][t][c]) * a.q_scale;
      sm.af[t][c] = expf(sm.g[buf][t][KDA ? c : 0]);
    }
    for (int i = tid; i < cnt * DV; i += NT) sm.vf[i / DV][i % DV] = io_to_float<IO>(sm.v[buf][i / DV][i % DV]);
    for (int t = tid; t < cnt; t += NT) sm.bf[t] = sm.beta[buf][t];
    __syncthreads();

    for (int t = 0; t < cnt; ++t) {
      // decay and the partial of r = S^T k over this thread's rows
      float racc = 0.f;
#pragma unroll
      for (int i = 0; i < ROWS; i += 4) {
        const float4 al = *reinterpret_cast<const float4 *>(&sm.af[t][row0 + i]);
        const float4 kk = *reinterpret_cast<const float4 *>(&sm.kf[t][row0 + i]);
        S[i + 0] *= al.x; racc = fmaf(kk.x, S[i + 0], racc);
        S[i + 1] *= al.y; racc = fmaf(kk.y, S[i + 1], racc);
        S[i + 2] *= al.z; racc = fmaf(kk.z, S[i + 2], racc);
        S[i + 3] *= al.w; racc = fmaf(kk.w, S[i + 3], racc);
      }
      if (RS > 1) red_r[parity][slice][v_col] = racc;
      __syncthreads();
      // the previous token's read-out partials are complete now as well
      if (RS > 1 && have_prev_o && slice == 0 && go) {
        float o = 0.f;
#pragma unroll
        for (int s = 0; s < RS; ++s) o += red_o[parity ^ 1][s][v_col];
        go[prev_t * v_stride + v_col] = float_to_io<OT>(o);
      }
      float rsum = racc;
      if (RS > 1) {
        rsum = 0.f;
#pragma unroll
        for (int s = 0; s < RS; ++s) rsum += red_r[parity][s][v_col];
      }
      const float u = sm.bf[t] * (sm.vf[t][v_col] - rsum);
      float oacc = 0.f;
#pragma unroll
      for (int i = 0; i < ROWS; i += 4) {
        const float4 kk = *reinterpret_cast<const float4 *>(&sm.kf[t][row0 + i]);
        const float4 qq = *reinterpret_cast<const float4 *>(&sm.qf[t][row0 + i]);
        S[i + 0] = fmaf(kk.x, u, S[i + 0]); oacc = fmaf(qq.x, S[i + 0], oacc);
        S[i + 1] = fmaf(kk.y, u, S[i + 1]); oacc = fmaf(qq.y, S[i + 1], oacc);
        S[i + 2] = fmaf(kk.z, u, S[i + 2]); oacc = fmaf(qq.z, S[i + 2], oacc);
        S[i + 3] = fmaf(kk.w, u, S[i + 3]); oacc = fmaf(qq.w, S[i + 3], oacc);
      }
      if (RS > 1) {
        red_o[parity][slice][v_col] = oacc;
        have_prev_o = true;
        prev_t = t_lo + t;
      } else if (go) {
        go[(t_lo + t) * v_stride + v_col] = float_to_io<OT>(oacc);
      }
      parity ^= 1;
    }
  }
  if (RS > 1) {
    __syncthreads();
    if (have_prev_o && slice == 0 && go) {
      float o = 0.f;
#pragma unroll
      for (int s = 0; s < RS; ++s) o += red_o[parity ^ 1][s][v_col];
      go[prev_t * v_stride + v_col] = float_to_io<OT>(o);
    }
  }

  if (a.mode == DASC_REFRESH_CONTINUE) {
#pragma unroll
    for (int i = 0; i < ROWS; ++i) st[(row0 + i) * DV + v_col] = S[i];
  } else {
    const uint8_t *keep = a.row_keep + static_cast<int64_t>(layer) * a.rows_per_layer + static_cast<int64_t>(h) * DK;
#pragma unroll
    for (int i = 0; i < ROWS; ++i)
      if (!keep[row0 + i]) st[(row0 + i) * DV + v_col] = S[i];
  }
}

// grid = one CTA per unit (from_list == 0), or a fixed grid whose CTAs walk the list of units that the chunked kernel
// handed over (from_list == 1; the list and its length are in the workspace, written earlier on the same stream).
template <int DK, int DV, int RS, typename IO, typename OT, bool KDA>
__global__ void __launch_bounds__(DV *RS) refresh_seq_kernel(DascRefreshArgs a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  if (!a.from_list) {
    seq_unit<DK, DV, RS, IO, OT, KDA>(a, static_cast<int>(blockIdx.x), smem_raw);
    return;
  }
  uint32_t *ws = static_cast<uint32_t *>(a.workspace);
  const uint32_t listed = ws[2];
  const int n_list = static_cast<int>(listed < static_cast<uint32_t>(a.unit_list_cap) ? listed : a.unit_list_cap);
  for (int i = blockIdx.x; i < n_list; i += gridDim.x) {
    seq_unit<DK, DV, RS, IO, OT, KDA>(a, a.unit_list[i], smem_raw);
    if (threadIdx.x == 0) atomicAdd(ws + 3, 1u);
    __syncthreads();  // the next unit reuses the staging buffers
  }
}

template <int DK, int DV, int RS, typename IO, typename OT, bool KDA>
int launch(const DascRefreshArgs &a, void *stream) {
  const size_t smem = sizeof(SeqSmem<DK, DV, IO, KDA>) + sizeof(float) * 4 * RS * DV;
  auto kern = refresh_seq_kernel<DK, DV, RS, IO, OT, KDA>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (e != cudaSuccess) return static_cast<int>(e);
  const int64_t n_units = static_cast<int64_t>(a.n_req) * a.n_layers_in_call * a.H_v;
  if (n_units == 0) return cudaSuccess;
  if (n_units > 2147483647LL) return static_cast<int>(cudaErrorInvalidConfiguration);
  // a handed-over list is short (units outside the chunked kernel's range or below its length threshold): a grid
  // of a few CTAs per SM walks it, and costs next to nothing when the list is empty
  const int64_t grid = a.from_list ? (n_units < 444 ? n_units : 444) : n_units;
  kern<<<static_cast<unsigned>(grid), DV * RS, smem, static_cast<cudaStream_t>(stream)>>>(a);
  return static_cast<int>(cudaGetLastError());
}

template <int DK, int DV, int RS, typename IO, typename OT>
int dispatch_kind(const DascRefreshArgs &a, void *stream) {
  return a.kind == DASC_KDA ? launch<DK, DV, RS, IO, OT, true>(a, stream) : launch<DK, DV, RS, IO, OT, false>(a, stream);
}

template <int DK, int DV, int RS>
int dispatch(const DascRefreshArgs &a, void *stream) {
  const bool o_bf16 = a.o ? a.o_bf16 != 0 : a.io_bf16 != 0;  // no output: any instantiation will do
  if (a.io_bf16)
    return o_bf16 ? dispatch_kind<DK, DV, RS, __nv_bfloat16, __nv_bfloat16>(a, stream)
                  : dispatch_kind<DK, DV, RS, __nv_bfloat16, float>(a, stream);
  return o_bf16 ? dispatch_kind<DK, DV, RS, float, __nv_bfloat16>(a, stream)
                : dispatch_kind<DK, DV, RS, float, float>(a, stream);
}

}  // namespace

// Returns a cudaError_t as int, or -1 if the shape has no instantiation.
int dasc_launch_refresh_seq(const DascRefreshArgs &a, void *stream) {
  if (a.d_k == 128 && a.d_v == 128) return dispatch<128, 128, 2>(a, stream);
  if (a.d_k == 64 && a.d_v == 64) return dispatch<64, 64, 2>(a, stream);
  if (a.d_k == 32 && a.d_v == 32) return dispatch<32, 32, 1>(a, stream);
  return -1;
}
