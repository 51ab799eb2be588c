// Suffix refresh, chunked form, on the Blackwell tensor cores (tcgen05 + TMEM).
//
// Eq. 1 (transposed orientation) over a chunk of C = 64 tokens starting from S_0, with
// G_t the running sum of the log-decay inside the chunk and m the chunk midpoint:
//   Kt_t = k_t * exp(G_t - G_m),  Kh_t = k_t * exp(G_m - G_t),  Qt_t = q_t * exp(G_t - G_m)
//   S'   = Diag(exp(G_m)) S_0                                   (state decayed to the midpoint)
//   A    = strict_lower(Kt Kh^T) * beta,   P = lower_incl_diag(Qt Kh^T)
//   U    = (I + A)^-1 * beta * (V - Kt S')                      (the deltas written at each token)
//   O    = Qt S' + P U
//   S_C  = Diag(exp(G_C - G_m)) (S' + Kh^T U)
// Referencing the decay to the midpoint keeps every exponent within half a chunk's decay.
//
// Mapping.  One CTA (128 threads) per (request, layer, value head); the state lives in TMEM
// transposed, S'^T: lane = value column v, column = key channel c, fp32, for the whole suffix.
// All five products run as M = 128 tcgen05.mma (kind::tf32, fp32 accumulate) with the value
// index on the TMEM lanes, so that each accumulator is directly the A operand of the next:
//   MMA1  [Kt;Qt] Kh^T            -> A (lanes 0-63) and P (lanes 64-127)        smem x smem
//   MMA2  S'^T [Kt;Qt]^T          -> R^T | (Qt S')^T                            tmem x smem
//   MMA3  RHS^T T^T               -> U^T                                         tmem x smem
//   MMA4  (Qt S')^T += U^T P^T    -> O^T                                         tmem x smem
//   MMA5  S'^T      += U^T Kh     -> state                                       tmem x smem
// Operands built on the CUDA cores are rounded to tf32 (round-to-nearest) before use; the
// state master copy stays fp32.  The unit-lower-triangular inverse T = (I + A)^-1 is computed
// in fp32 on the CUDA cores (16x16 diagonal blocks by substitution, the rest blockwise).
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "dasc_internal.h"
#include "tcgen05_util.cuh"

namespace {

using namespace tc5;

constexpr int C = 64;     // chunk length
constexpr int D = 128;    // d_k = d_v
constexpr int NT = 128;   // threads per CTA
constexpr int LDX = 68;   // row pitch (floats) of the fp32 triangular work matrices

// TMEM columns
constexpr uint32_t COL_S = 0, COL_SOP = 128, COL_RO = 256, COL_AP = 384, COL_U = 448;

// shared memory map (bytes)
constexpr uint32_t OFF_KQ = 0;                       // [4][128 rows][128 B]  rows 0-63 Kt, 64-127 Qt
constexpr uint32_t OFF_KH = OFF_KQ + 4 * 128 * 128;  // [4][64 rows][128 B]   Kh[t][c]
constexpr uint32_t OFF_KHT = OFF_KH + 4 * 64 * 128;  // [2][128 rows][128 B]  Kh^T[c][t]
constexpr uint32_t OFF_TM = OFF_KHT + 2 * 128 * 128; // [2][64 rows][128 B]   T[t][i]
constexpr uint32_t OFF_PM = OFF_TM + 2 * 64 * 128;   // [2][64 rows][128 B]   P[t][i]
constexpr uint32_t OFF_V = OFF_PM + 2 * 64 * 128;    // [64][128] bf16
constexpr uint32_t OFF_L = OFF_V + C * D * 2;        // [64][LDX] fp32
constexpr uint32_t OFF_X = OFF_L + C * LDX * 4;      // [64][LDX] fp32
constexpr uint32_t OFF_FAC = OFF_X + C * LDX * 4;    // [128] fp32 state factor per channel
constexpr uint32_t OFF_BETA = OFF_FAC + D * 4;       // [64] fp32
constexpr uint32_t OFF_MISC = OFF_BETA + C * 4;      // barriers, tmem base, abort flag
constexpr uint32_t SMEM_BYTES = OFF_MISC + 64;
constexpr uint32_t SMEM_ALLOC = SMEM_BYTES + 1024;   // slack to align the base to 1024 bytes

constexpr uint32_t kMaxPolls = 1u << 22;

struct Misc {
  uint64_t bar_ap, bar_ro, bar_u, bar_os;
  uint32_t tmem_base;
  volatile uint32_t abort_flag;
};

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ void cp_async16_zfill(uint32_t smem, const void *gmem, bool valid) {
  const uint32_t n = valid ? 16u : 0u;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem), "l"(gmem), "r"(n) : "memory");
}

// Bounded wait on an MMA-completion barrier; after one time-out every later wait returns at once.
__device__ __forceinline__ void wait_bar(uint64_t *bar, uint32_t parity, Misc *misc, uint32_t *err) {
  if (misc->abort_flag) return;
  if (!mbar_wait_bounded(bar, parity, kMaxPolls)) {
    misc->abort_flag = 1;
    if (err) atomicExch(err, 1u);
  }
}

// C (16x16, at c) = sign * sum_p A_p B_p over `np` block pairs; 64 threads, thread (i, jq) -> C[i][4jq..4jq+3].
__device__ __forceinline__ void block_mm(float *c, const float *const *a, const float *const *b, int np, float sign,
                                         int id) {
  const int i = id >> 2, j0 = (id & 3) << 2;
  float acc0 = 0.f, acc1 = 0.f, acc2 = 0.f, acc3 = 0.f;
  for (int p = 0; p < np; ++p) {
    const float *ap = a[p] + i * LDX;
    const float *bp = b[p] + j0;
#pragma unroll
    for (int k = 0; k < 16; ++k) {
      const float av = ap[k];
      const float4 bv = *reinterpret_cast<const float4 *>(bp + k * LDX);
      acc0 = fmaf(av, bv.x, acc0);
      acc1 = fmaf(av, bv.y, acc1);
      acc2 = fmaf(av, bv.z, acc2);
      acc3 = fmaf(av, bv.w, acc3);
    }
  }
  *reinterpret_cast<float4 *>(c + i * LDX + j0) = make_float4(sign * acc0, sign * acc1, sign * acc2, sign * acc3);
}

template <bool KDA, typename OT>
__global__ void __launch_bounds__(NT, 1) refresh_chunked_kernel(DascRefreshArgs a) {
  extern __shared__ unsigned char smem_dyn[];
  unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t{1023});
  const uint32_t sbase = smem_u32(smem);
  float *Lm = reinterpret_cast<float *>(smem + OFF_L);
  float *Xm = reinterpret_cast<float *>(smem + OFF_X);
  float *fac_s = reinterpret_cast<float *>(smem + OFF_FAC);
  float *beta_s = reinterpret_cast<float *>(smem + OFF_BETA);
  const __nv_bfloat16 *Vs = reinterpret_cast<const __nv_bfloat16 *>(smem + OFF_V);
  Misc *misc = reinterpret_cast<Misc *>(smem + OFF_MISC);
  uint32_t *err = static_cast<uint32_t *>(a.workspace);

  const int tid = threadIdx.x, warp = tid >> 5;
  const int h = blockIdx.x % a.H_v;
  const int lc = (blockIdx.x / a.H_v) % a.n_layers_in_call;
  const int r = blockIdx.x / (a.H_v * a.n_layers_in_call);
  const int hk = h / (a.H_v / a.H_k);
  const int layer = a.layer_begin + lc;
  const int64_t t_begin = a.cu_seqlens[r];
  const int n_tok = static_cast<int>(a.cu_seqlens[r + 1] - t_begin);
  if (n_tok <= 0 && a.mode == DASC_REFRESH_CONTINUE) return;

  float *st = a.state + static_cast<int64_t>(a.req_idx[r]) * a.req_stride + static_cast<int64_t>(layer) * a.layer_stride +
              static_cast<int64_t>(h) * D * D;
  const int64_t tok0 = static_cast<int64_t>(lc) * a.total_tokens + t_begin;
  const __nv_bfloat16 *gq = static_cast<const __nv_bfloat16 *>(a.q) + (tok0 * a.H_k + hk) * D;
  const __nv_bfloat16 *gk = static_cast<const __nv_bfloat16 *>(a.k) + (tok0 * a.H_k + hk) * D;
  const __nv_bfloat16 *gv = static_cast<const __nv_bfloat16 *>(a.v) + (tok0 * a.H_v + h) * D;
  const float *gg = a.g + (tok0 * a.H_v + h) * (KDA ? D : 1);
  const float *gb = a.beta + tok0 * a.H_v + h;
  OT *go = a.o ? static_cast<OT *>(a.o) + (tok0 * a.H_v + h) * D : nullptr;
  const int64_t qk_stride = static_cast<int64_t>(a.H_k) * D, v_stride = static_cast<int64_t>(a.H_v) * D;
  const int64_t g_stride = static_cast<int64_t>(a.H_v) * (KDA ? D : 1), b_stride = a.H_v;

  // ---- set-up: barriers and tensor memory ----
  if (tid == 0) {
    mbar_init(&misc->bar_ap, 1);
    mbar_init(&misc->bar_ro, 1);
    mbar_init(&misc->bar_u, 1);
    mbar_init(&misc->bar_os, 1);
    misc->abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 0) {
    tmem_alloc(&misc->tmem_base, 512);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tm = misc->tmem_base;
  const uint32_t tlane = tm + (static_cast<uint32_t>(warp * 32) << 16);  // this warp's lane quadrant

  constexpr uint32_t ID_M128_N64 = idesc_tf32(128, 64, false, false);
  constexpr uint32_t ID_M128_N128 = idesc_tf32(128, 128, false, false);
  constexpr float LOG2E = 1.4426950408889634f;

  float prev_post = 0.f;  // thread c: log of the factor still owed to channel c of the state
  const int n_chunks = (n_tok + C - 1) / C;

  for (int ch = 0; ch < n_chunks; ++ch) {
    const uint32_t par = ch & 1;
    const int t0 = ch * C;
    const int ntok = min(C, n_tok - t0);

    // ---- (1) V tile and beta for this chunk (used in step 7) ----
    for (int i = tid; i < C * (D * 2 / 16); i += NT) {
      const int t = i >> 4, j = i & 15;
      const bool valid = t < ntok;
      cp_async16_zfill(sbase + OFF_V + t * (D * 2) + j * 16,
                       reinterpret_cast<const char *>(gv + (t0 + (valid ? t : 0)) * v_stride) + j * 16, valid);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
    if (tid < C) beta_s[tid] = tid < ntok ? gb[(t0 + tid) * b_stride] : 0.f;

    // ---- (2) prep: thread = key channel c ----
    {
      const int c = tid;
      float G[C];
#pragma unroll
      for (int t = 0; t < C; ++t) G[t] = t < ntok ? gg[(t0 + t) * g_stride + (KDA ? c : 0)] : 0.f;
#pragma unroll
      for (int t = 1; t < C; ++t) G[t] += G[t - 1];
      const float Gm = G[C / 2 - 1], Gc = G[C - 1];
      fac_s[c] = ex2f((prev_post + Gm) * LOG2E);
      prev_post = Gc - Gm;
#pragma unroll
      for (int t4 = 0; t4 < C; t4 += 4) {
        uint32_t kht[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int t = t4 + u;
          float kf = 0.f, qf = 0.f;
          if (t < ntok) {
            kf = __bfloat162float(gk[(t0 + t) * qk_stride + c]);
            qf = __bfloat162float(gq[(t0 + t) * qk_stride + c]) * a.q_scale;
          }
          const float d = (G[t] - Gm) * LOG2E;
          const float e1 = ex2f(d), e2 = ex2f(-d);
          *reinterpret_cast<uint32_t *>(smem + OFF_KQ + sw128_offset(128, t, c)) = to_tf32(kf * e1);
          *reinterpret_cast<uint32_t *>(smem + OFF_KQ + sw128_offset(128, 64 + t, c)) = to_tf32(qf * e1);
          kht[u] = to_tf32(kf * e2);
          *reinterpret_cast<uint32_t *>(smem + OFF_KH + sw128_offset(64, t, c)) = kht[u];
        }
        *reinterpret_cast<uint4 *>(smem + OFF_KHT + sw128_offset(128, c, t4)) = make_uint4(kht[0], kht[1], kht[2], kht[3]);
      }
    }
    fence_smem_to_async();
    __syncthreads();

    // ---- (3) MMA1: [Kt;Qt] Kh^T ----
    if (tid == 0) {
      tc_fence_after_sync();
#pragma unroll
      for (int kb = 0; kb < 4; ++kb)
#pragma unroll
        for (int j = 0; j < 4; ++j)
          mma_ss(tm + COL_AP, desc_kmajor(sbase + OFF_KQ + kb * (128 * 128) + j * 32),
                 desc_kmajor(sbase + OFF_KH + kb * (64 * 128) + j * 32), ID_M128_N64, (kb | j) != 0);
      mma_commit(&misc->bar_ap);
    }

    // ---- (4) state pass: thread = value column v; scale to this chunk's midpoint, refresh the tf32 copy ----
    {
      const int v = tid;
#pragma unroll 1
      for (int c0 = 0; c0 < D; c0 += 32) {
        uint32_t s[32];
        if (ch == 0) {
          if (a.mode == DASC_REFRESH_CONTINUE) {
#pragma unroll
            for (int j = 0; j < 32; ++j) s[j] = __float_as_uint(st[(c0 + j) * D + v]);
          } else {
#pragma unroll
            for (int j = 0; j < 32; ++j) s[j] = 0u;
          }
        } else {
          tmem_ld32(tlane + COL_S + c0, s);
          tmem_ld_wait();
        }
        uint32_t sop[32];
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const float x = __uint_as_float(s[j]) * fac_s[c0 + j];
          s[j] = __float_as_uint(x);
          sop[j] = to_tf32(x);
        }
        tmem_st32(tlane + COL_S + c0, s);
        tmem_st32(tlane + COL_SOP + c0, sop);
      }
      tmem_st_wait();
    }
    tc_fence_before_sync();
    __syncthreads();

    // ---- (5) MMA2: S'^T [Kt;Qt]^T ----
    if (tid == 0) {
      tc_fence_after_sync();
#pragma unroll
      for (int kb = 0; kb < 4; ++kb)
#pragma unroll
        for (int j = 0; j < 4; ++j)
          mma_ts(tm + COL_RO, tm + COL_SOP + kb * 32 + j * 8, desc_kmajor(sbase + OFF_KQ + kb * (128 * 128) + j * 32),
                 ID_M128_N128, (kb | j) != 0);
      mma_commit(&misc->bar_ro);
    }

    // ---- (6) A and P out of TMEM; T = (I + A)^-1 ----
    wait_bar(&misc->bar_ap, par, misc, err);
    tc_fence_after_sync();
    if (tid < C) {
      // lanes 0-63: row t of A = strict_lower(Kt Kh^T) * beta_t, kept in fp32 for the inverse
      const int t = tid;
      const float bt = beta_s[t];
#pragma unroll 1
      for (int c0 = 0; c0 < C; c0 += 32) {
        uint32_t x[32];
        tmem_ld32(tlane + COL_AP + c0, x);
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 32; j += 4) {
          float4 o;
          o.x = (c0 + j + 0 < t) ? bt * __uint_as_float(x[j + 0]) : 0.f;
          o.y = (c0 + j + 1 < t) ? bt * __uint_as_float(x[j + 1]) : 0.f;
          o.z = (c0 + j + 2 < t) ? bt * __uint_as_float(x[j + 2]) : 0.f;
          o.w = (c0 + j + 3 < t) ? bt * __uint_as_float(x[j + 3]) : 0.f;
          *reinterpret_cast<float4 *>(Lm + t * LDX + c0 + j) = o;
        }
      }
    } else {
      // lanes 64-127: row t of P = lower_incl_diag(Qt Kh^T), straight to its operand tile
      const int t = tid - C;
#pragma unroll 1
      for (int c0 = 0; c0 < C; c0 += 32) {
        uint32_t x[32];
        tmem_ld32(tlane + COL_AP + c0, x);
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 32; j += 4) {
          uint4 o;
          o.x = (c0 + j + 0 <= t) ? to_tf32(__uint_as_float(x[j + 0])) : 0u;
          o.y = (c0 + j + 1 <= t) ? to_tf32(__uint_as_float(x[j + 1])) : 0u;
          o.z = (c0 + j + 2 <= t) ? to_tf32(__uint_as_float(x[j + 2])) : 0u;
          o.w = (c0 + j + 3 <= t) ? to_tf32(__uint_as_float(x[j + 3])) : 0u;
          *reinterpret_cast<uint4 *>(smem + OFF_PM + sw128_offset(64, t, c0 + j)) = o;
        }
      }
    }
    __syncthreads();
    // diagonal 16x16 blocks: thread (block b, column cc) solves (I + L_bb) x = e_cc by forward substitution
    if (tid < C) {
      const int b = tid >> 4, cc = tid & 15;
      const float *Lb = Lm + (b * 16) * LDX + b * 16;
      float x[16];
#pragma unroll
      for (int rr = 0; rr < 16; ++rr) {
        float acc = (rr == cc) ? 1.f : 0.f;
#pragma unroll
        for (int j = 0; j < rr; ++j) acc = fmaf(-Lb[rr * LDX + j], x[j], acc);
        x[rr] = acc;
      }
#pragma unroll
      for (int rr = 0; rr < 16; ++rr) Xm[(b * 16 + rr) * LDX + b * 16 + cc] = x[rr];
    }
    __syncthreads();
    {
      // off-diagonal blocks; Y_IJ = sum_K L_IK X_KJ is parked in the (unused) upper block (J, I) of X
      const int grp = tid >> 6, id = tid & 63;
      auto Lb = [&](int I, int J) { return Lm + (I * 16) * LDX + J * 16; };
      auto Xb = [&](int I, int J) { return Xm + (I * 16) * LDX + J * 16; };
      const float *pa[3];
      const float *pb[3];
      // first sub-diagonal
      if (grp == 0) {
        pa[0] = Lb(1, 0); pb[0] = Xb(0, 0); block_mm(Xb(0, 1), pa, pb, 1, 1.f, id);
        pa[0] = Lb(3, 2); pb[0] = Xb(2, 2); block_mm(Xb(2, 3), pa, pb, 1, 1.f, id);
      } else {
        pa[0] = Lb(2, 1); pb[0] = Xb(1, 1); block_mm(Xb(1, 2), pa, pb, 1, 1.f, id);
      }
      __syncthreads();
      if (grp == 0) {
        pa[0] = Xb(1, 1); pb[0] = Xb(0, 1); block_mm(Xb(1, 0), pa, pb, 1, -1.f, id);
        pa[0] = Xb(3, 3); pb[0] = Xb(2, 3); block_mm(Xb(3, 2), pa, pb, 1, -1.f, id);
      } else {
        pa[0] = Xb(2, 2); pb[0] = Xb(1, 2); block_mm(Xb(2, 1), pa, pb, 1, -1.f, id);
      }
      __syncthreads();
      // second sub-diagonal
      if (grp == 0) {
        pa[0] = Lb(2, 0); pb[0] = Xb(0, 0); pa[1] = Lb(2, 1); pb[1] = Xb(1, 0); block_mm(Xb(0, 2), pa, pb, 2, 1.f, id);
      } else {
        pa[0] = Lb(3, 1); pb[0] = Xb(1, 1); pa[1] = Lb(3, 2); pb[1] = Xb(2, 1); block_mm(Xb(1, 3), pa, pb, 2, 1.f, id);
      }
      __syncthreads();
      if (grp == 0) {
        pa[0] = Xb(2, 2); pb[0] = Xb(0, 2); block_mm(Xb(2, 0), pa, pb, 1, -1.f, id);
      } else {
        pa[0] = Xb(3, 3); pb[0] = Xb(1, 3); block_mm(Xb(3, 1), pa, pb, 1, -1.f, id);
      }
      __syncthreads();
      // corner block
      if (grp == 0) {
        pa[0] = Lb(3, 0); pb[0] = Xb(0, 0); pa[1] = Lb(3, 1); pb[1] = Xb(1, 0); pa[2] = Lb(3, 2); pb[2] = Xb(2, 0);
        block_mm(Xb(0, 3), pa, pb, 3, 1.f, id);
      }
      __syncthreads();
      if (grp == 0) {
        pa[0] = Xb(3, 3); pb[0] = Xb(0, 3); block_mm(Xb(3, 0), pa, pb, 1, -1.f, id);
      }
      __syncthreads();
      // T (lower triangle of X, unit diagonal) -> tf32 operand tile
      const int t = tid >> 1, i0 = (tid & 1) * 32;
#pragma unroll
      for (int j = 0; j < 32; j += 4) {
        const float4 xv = *reinterpret_cast<const float4 *>(Xm + t * LDX + i0 + j);
        uint4 o;
        o.x = (i0 + j + 0 <= t) ? to_tf32(xv.x) : 0u;
        o.y = (i0 + j + 1 <= t) ? to_tf32(xv.y) : 0u;
        o.z = (i0 + j + 2 <= t) ? to_tf32(xv.z) : 0u;
        o.w = (i0 + j + 3 <= t) ? to_tf32(xv.w) : 0u;
        *reinterpret_cast<uint4 *>(smem + OFF_TM + sw128_offset(64, t, i0 + j)) = o;
      }
    }
    fence_smem_to_async();

    // ---- (7) RHS^T = beta (V - R)^T, written over R^T as the tf32 A operand of MMA3 ----
    wait_bar(&misc->bar_ro, par, misc, err);
    tc_fence_after_sync();
    asm volatile("cp.async.wait_all;" ::: "memory");
    __syncthreads();  // V tile visible to everyone
    {
      const int v = tid;
#pragma unroll 1
      for (int c0 = 0; c0 < C; c0 += 32) {
        uint32_t x[32];
        tmem_ld32(tlane + COL_RO + c0, x);
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const float vv = __bfloat162float(Vs[(c0 + j) * D + v]);
          x[j] = to_tf32(beta_s[c0 + j] * (vv - __uint_as_float(x[j])));
        }
        tmem_st32(tlane + COL_RO + c0, x);
      }
      tmem_st_wait();
    }
    tc_fence_before_sync();
    __syncthreads();

    // ---- (8) MMA3: U^T = RHS^T T^T ----
    if (tid == 0) {
      tc_fence_after_sync();
#pragma unroll
      for (int kb = 0; kb < 2; ++kb)
#pragma unroll
        for (int j = 0; j < 4; ++j)
          mma_ts(tm + COL_U, tm + COL_RO + kb * 32 + j * 8, desc_kmajor(sbase + OFF_TM + kb * (64 * 128) + j * 32),
                 ID_M128_N64, (kb | j) != 0);
      mma_commit(&misc->bar_u);
    }

    // ---- (9) U^T rounded to tf32 in place ----
    wait_bar(&misc->bar_u, par, misc, err);
    tc_fence_after_sync();
#pragma unroll 1
    for (int c0 = 0; c0 < C; c0 += 32) {
      uint32_t x[32];
      tmem_ld32(tlane + COL_U + c0, x);
      tmem_ld_wait();
#pragma unroll
      for (int j = 0; j < 32; ++j) x[j] = to_tf32(__uint_as_float(x[j]));
      tmem_st32(tlane + COL_U + c0, x);
    }
    tmem_st_wait();
    tc_fence_before_sync();
    __syncthreads();

    // ---- (10) MMA4: O^T += U^T P^T;  MMA5: S'^T += U^T Kh ----
    if (tid == 0) {
      tc_fence_after_sync();
      if (go) {
#pragma unroll
        for (int kb = 0; kb < 2; ++kb)
#pragma unroll
          for (int j = 0; j < 4; ++j)
            mma_ts(tm + COL_RO + 64, tm + COL_U + kb * 32 + j * 8, desc_kmajor(sbase + OFF_PM + kb * (64 * 128) + j * 32),
                   ID_M128_N64, true);
      }
#pragma unroll
      for (int kb = 0; kb < 2; ++kb)
#pragma unroll
        for (int j = 0; j < 4; ++j)
          mma_ts(tm + COL_S, tm + COL_U + kb * 32 + j * 8, desc_kmajor(sbase + OFF_KHT + kb * (128 * 128) + j * 32),
                 ID_M128_N128, true);
      mma_commit(&misc->bar_os);
    }

    // ---- (11) outputs of this chunk ----
    wait_bar(&misc->bar_os, par, misc, err);
    tc_fence_after_sync();
    if (go) {
      const int v = tid;
#pragma unroll 1
      for (int c0 = 0; c0 < C; c0 += 32) {
        uint32_t x[32];
        tmem_ld32(tlane + COL_RO + 64 + c0, x);
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          const int t = c0 + j;
          if (t < ntok) {
            if constexpr (sizeof(OT) == 2) go[(t0 + t) * v_stride + v] = __float2bfloat16_rn(__uint_as_float(x[j]));
            else go[(t0 + t) * v_stride + v] = __uint_as_float(x[j]);
          }
        }
      }
    }
    tc_fence_before_sync();
    __syncthreads();
  }

  // ---- final state: the factor still owed, then write back ----
  fac_s[tid] = ex2f(prev_post * LOG2E);
  __syncthreads();
  tc_fence_after_sync();
  {
    const int v = tid;
    const uint8_t *keep = a.row_keep + static_cast<int64_t>(layer) * a.rows_per_layer + static_cast<int64_t>(h) * D;
    const bool merge = a.mode != DASC_REFRESH_CONTINUE;
#pragma unroll 1
    for (int c0 = 0; c0 < D; c0 += 32) {
      uint32_t s[32];
      if (n_chunks > 0) {
        tmem_ld32(tlane + COL_S + c0, s);
        tmem_ld_wait();
      } else {
#pragma unroll
        for (int j = 0; j < 32; ++j) s[j] = 0u;  // scratch mode with an empty suffix
      }
#pragma unroll
      for (int j = 0; j < 32; ++j) {
        const int c = c0 + j;
        if (!merge || !keep[c]) st[c * D + v] = __uint_as_float(s[j]) * fac_s[c];
      }
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tm, 512);
}

template <bool KDA, typename OT>
int launch(const DascRefreshArgs &a, void *stream) {
  auto kern = refresh_chunked_kernel<KDA, OT>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(SMEM_ALLOC));
  if (e != cudaSuccess) return static_cast<int>(e);
  const int64_t n_units = static_cast<int64_t>(a.n_req) * a.n_layers_in_call * a.H_v;
  if (n_units == 0) return cudaSuccess;
  if (n_units > 2147483647LL) return static_cast<int>(cudaErrorInvalidConfiguration);
  e = cudaMemsetAsync(a.workspace, 0, 4, static_cast<cudaStream_t>(stream));  // clear the time-out flag
  if (e != cudaSuccess) return static_cast<int>(e);
  kern<<<static_cast<unsigned>(n_units), NT, SMEM_ALLOC, static_cast<cudaStream_t>(stream)>>>(a);
  return static_cast<int>(cudaGetLastError());
}

}  // namespace

// Scratch the chunked kernel needs: one 32-bit time-out flag (first word), padded to 256 bytes.
size_t dasc_refresh_chunked_workspace_bytes(int32_t, int32_t, int32_t) { return 256; }

// Returns a cudaError_t as int, or -1 if this kernel does not take the request
// (it needs d_k = d_v = 128 and bf16 token streams).
int dasc_launch_refresh_chunked(const DascRefreshArgs &a, void *stream) {
  if (a.d_k != D || a.d_v != D || !a.io_bf16) return -1;
  const bool kda = a.kind == DASC_KDA;
  const bool o_bf16 = a.o ? a.o_bf16 != 0 : true;
  if (o_bf16) return kda ? launch<true, __nv_bfloat16>(a, stream) : launch<false, __nv_bfloat16>(a, stream);
  return kda ? launch<true, float>(a, stream) : launch<false, float>(a, stream);
}
