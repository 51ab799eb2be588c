// Suffix refresh, chunked form, on the Blackwell tensor cores (tcgen05 + TMEM):
// 32-token chunks, two CTAs resident per SM.
//
// Eq. 1 (transposed orientation) over a chunk of C = 32 tokens starting from S_0, with
// G_t the running sum of the log-decay inside the chunk and m the chunk midpoint:
//   Kt_t = k_t * exp(G_t - G_m),  Kh_t = k_t * exp(G_m - G_t),  Qt_t = q_t * exp(G_t - G_m)
//   S'   = Diag(exp(G_m)) S_0                                   (state decayed to the midpoint)
//   A    = strict_lower(Kt Kh^T) * beta,   P = lower_incl_diag(Qt Kh^T)
//   U    = (I + A)^-1 * beta * (V - Kt S')                      (the deltas written at each token)
//   O    = Qt S' + P U
//   S_C  = Diag(exp(G_C - G_m)) (S' + Kh^T U)
// Referencing the decay to the midpoint keeps every exponent within half a chunk's decay.
//
// Mapping.  One CTA per (request, layer, value head): eight compute warps (two per TMEM lane quadrant,
// each taking half of the columns) and one warp that only issues tensor-core work; 256 TMEM columns and about 108 KB of shared memory per CTA, so two
// CTAs share an SM and one fills the other's latency gaps (every phase of a chunk depends on the
// one before it).  The state lives in TMEM transposed, S'^T: lane = value column v, column = key
// channel c, fp32, for the whole suffix; the tensor core reads it as a tf32 operand directly.
// All products are M = 128 tcgen05.mma (kind::tf32, fp32 accumulate) with the value index on the
// TMEM lanes, so that each accumulator is the A operand of the next product:
//   MMA1  [Kt;Qt] Kh^T            -> A (lanes 0-31) and P (lanes 32-63)         smem x smem
//   MMA2  S'^T [Kt;Qt]^T          -> R^T | (Qt S')^T                            tmem x smem
//   MMA3  RHS^T T^T               -> U^T      (RHS as a tf32 high/low pair)     tmem x smem
//   MMA4  (Qt S')^T += U^T P^T    -> O^T                                         tmem x smem
//   MMA5  S'^T      += U^T Kh     -> state    (U as a tf32 high/low pair)       tmem x smem
// Operands built on the CUDA cores are rounded to tf32 (round-to-nearest).  T = (I + A)^-1 is
// formed by one warp: 16x16 diagonal blocks by fp32 substitution, the off-diagonal block by
// mma.sync (tf32) products.  Token inputs of chunk n+1 are fetched with cp.async while chunk n
// computes.  Kh[t][c] (needed by MMA1 only) shares its storage with the T and P tiles; the raw
// log-decay tile shares its storage with the V tile.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "dasc_internal.h"
#include "tcgen05_util.cuh"

namespace {

using namespace tc5;

constexpr int C = 32;        // chunk length
constexpr int D = 128;       // d_k = d_v
constexpr int NC = 256;      // compute threads
constexpr int NT = NC + 32;  // + the MMA-issuing warp
constexpr int LDX = 36;      // row pitch (floats) of the fp32 triangular work matrices
constexpr uint32_t TMEM_COLS = 256;

// TMEM columns
constexpr uint32_t COL_S = 0, COL_AP = 128, COL_RO = 160, COL_U = 224;  // RO: R^T 160-191 | (Qt S')^T 192-223

// shared memory map (bytes)
constexpr uint32_t OFF_KQ = 0;                         // [4][64 rows][128 B]  rows 0-31 Kt, 32-63 Qt; later the O tile
constexpr uint32_t OFF_KHT = OFF_KQ + 4 * 64 * 128;    // [1][128 rows][128 B] Kh^T[c][t]
constexpr uint32_t OFF_KH = OFF_KHT + 128 * 128;       // [4][32 rows][128 B]  Kh[t][c], until MMA1 is done; then:
constexpr uint32_t OFF_TM = OFF_KH;                    // [1][32 rows][128 B]  T[t][i]
constexpr uint32_t OFF_PM = OFF_TM + 32 * 128;         // [1][32 rows][128 B]  P[t][i]
constexpr uint32_t OFF_RAWQ = OFF_KH + 4 * 32 * 128;   // [32][128] bf16 raw q of the next chunk
constexpr uint32_t OFF_RAWK = OFF_RAWQ + C * D * 2;    // [32][128] bf16 raw k of the next chunk
constexpr uint32_t OFF_G = OFF_RAWK + C * D * 2;       // [32][128] fp32 raw g (until prep), then
constexpr uint32_t OFF_V = OFF_G;                      // [32][128] bf16 v (until the right-hand side is formed)
constexpr uint32_t OFF_L = OFF_G + C * D * 4;          // [32][LDX] fp32
constexpr uint32_t OFF_X = OFF_L + C * LDX * 4;        // [32][LDX] fp32
constexpr uint32_t OFF_FAC = OFF_X + C * LDX * 4;      // [128] fp32 state factor per channel
constexpr uint32_t OFF_POST = OFF_FAC + D * 4;         // [2][128] fp32 log-factor owed after a chunk, by chunk parity
constexpr uint32_t OFF_BETA = OFF_POST + 2 * D * 4;    // [2][32] fp32, by chunk parity
constexpr uint32_t OFF_GSC = OFF_BETA + 2 * C * 4;     // [2][32] fp32 scalar log-decay (GDN), by chunk parity
constexpr uint32_t OFF_MISC = OFF_GSC + 2 * C * 4;     // barriers, tmem base, abort flag
constexpr uint32_t SMEM_BYTES = OFF_MISC + 128;
constexpr uint32_t SMEM_ALLOC = SMEM_BYTES + 1024;     // slack to align the base to 1024 bytes
static_assert(SMEM_ALLOC <= 113 * 1024, "two CTAs per SM");

constexpr uint32_t kMaxPolls = 1u << 22;

// The tensor core reads the fp32 state as tf32 by dropping its low 13 mantissa bits, i.e. rounding
// towards zero: on average the operand is 2^-11 * E[1/m] = 3.52e-4 too small in magnitude (m the
// significand, log-uniform in [1, 2)).  The rows of Kt and Qt, the only partners of that operand,
// are scaled up by this factor to cancel the bias; A and P, which also come from those rows, are
// scaled back down when they are taken out of TMEM.
constexpr float kTruncComp = 1.000352f;
constexpr float kInvTruncComp = 1.0f / kTruncComp;
constexpr float kLog2TruncComp = 5.0774e-4f;  // log2(kTruncComp)

#ifdef DASC_PHASE_TIMING
#define PT_DECL long long pt_acc[16] = {0}; long long pt_last = clock64();
#define PT(i) do { long long pt_now = clock64(); pt_acc[i] += pt_now - pt_last; pt_last = pt_now; } while (0)
#define PT_DUMP do { if (blockIdx.x == gridDim.x / 2 && tid == 0) { long long *d = reinterpret_cast<long long *>(static_cast<char *>(a.workspace) + 64); for (int i = 0; i < 16; ++i) d[i] = pt_acc[i]; } } while (0)
#else
#define PT_DECL
#define PT(i)
#define PT_DUMP
#endif

struct Misc {
  // tensor core -> compute warps (one tcgen05.commit each per chunk)
  uint64_t bar_ap, bar_ro, bar_u, bar_o, bar_s;
  // compute warps -> issuing warp (256 arrivals each per chunk)
  uint64_t rdy_prep, rdy_state, rdy_rhs, rdy_u;
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

__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// barrier among the 256 compute threads only
__device__ __forceinline__ void sync_compute() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

// Bounded wait; after one time-out every later wait of this CTA returns at once.
__device__ __forceinline__ void wait_bar(uint64_t *bar, uint32_t parity, Misc *misc, uint32_t *err) {
  if (misc->abort_flag) return;
  if (!mbar_wait_bounded(bar, parity, kMaxPolls)) {
    misc->abort_flag = 1;
    if (err) atomicExch(err, 1u);
  }
}

__device__ __forceinline__ void mma_tf32_16x8x8(float (&d)[4], const uint32_t (&a)[4], const uint32_t (&b)[2]) {
  asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}

// One warp: acc (16x16) += A (16x16) * B (16x16), blocks in shared memory with pitch LDX.
__device__ __forceinline__ void warp_mm_acc(float (&acc)[2][4], const float *A, const float *B, int lane) {
  const int g = lane >> 2, tig = lane & 3;
#pragma unroll
  for (int kh = 0; kh < 2; ++kh) {
    uint32_t af[4];
    af[0] = tf32_pre(A[g * LDX + 8 * kh + tig]);
    af[1] = tf32_pre(A[(g + 8) * LDX + 8 * kh + tig]);
    af[2] = tf32_pre(A[g * LDX + 8 * kh + tig + 4]);
    af[3] = tf32_pre(A[(g + 8) * LDX + 8 * kh + tig + 4]);
#pragma unroll
    for (int nh = 0; nh < 2; ++nh) {
      uint32_t bf[2];
      bf[0] = tf32_pre(B[(8 * kh + tig) * LDX + 8 * nh + g]);
      bf[1] = tf32_pre(B[(8 * kh + tig + 4) * LDX + 8 * nh + g]);
      mma_tf32_16x8x8(acc[nh], af, bf);
    }
  }
}
__device__ __forceinline__ void warp_mm_store(float *Cb, const float (&acc)[2][4], float sign, int lane) {
  const int g = lane >> 2, tig = lane & 3;
#pragma unroll
  for (int nh = 0; nh < 2; ++nh) {
    *reinterpret_cast<float2 *>(Cb + g * LDX + 8 * nh + 2 * tig) = make_float2(sign * acc[nh][0], sign * acc[nh][1]);
    *reinterpret_cast<float2 *>(Cb + (g + 8) * LDX + 8 * nh + 2 * tig) = make_float2(sign * acc[nh][2], sign * acc[nh][3]);
  }
}

__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

// WITH_O = false is the state-only variant (no outputs wanted): q is never read, the Qt rows, P and the
// output product are left out.
template <bool KDA, typename OT, bool WITH_O>
__global__ void __launch_bounds__(NT, 2) refresh_chunked_kernel(DascRefreshArgs a) {
  extern __shared__ unsigned char smem_dyn[];
  unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t{1023});
  const uint32_t sbase = smem_u32(smem);
  float *Lm = reinterpret_cast<float *>(smem + OFF_L);
  float *Xm = reinterpret_cast<float *>(smem + OFF_X);
  float *fac_s = reinterpret_cast<float *>(smem + OFF_FAC);
  float *post_s = reinterpret_cast<float *>(smem + OFF_POST);
  float *beta_s = reinterpret_cast<float *>(smem + OFF_BETA);
  float *gsc_s = reinterpret_cast<float *>(smem + OFF_GSC);
  const __nv_bfloat16 *Vs = reinterpret_cast<const __nv_bfloat16 *>(smem + OFF_V);
  Misc *misc = reinterpret_cast<Misc *>(smem + OFF_MISC);
  uint32_t *err = static_cast<uint32_t *>(a.workspace);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int h = blockIdx.x % a.H_v;
  const int lc = (blockIdx.x / a.H_v) % a.n_layers_in_call;
  const int r = blockIdx.x / (a.H_v * a.n_layers_in_call);
  const int hk = h / (a.H_v / a.H_k);
  const int layer = a.layer_begin + lc;
  const int64_t t_begin = a.tok_begin ? a.tok_begin[r] : a.cu_seqlens[r];
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
  OT *const go = WITH_O ? static_cast<OT *>(a.o) + (tok0 * a.H_v + h) * D : nullptr;
  const int64_t qk_stride = static_cast<int64_t>(a.H_k) * D, v_stride = static_cast<int64_t>(a.H_v) * D;
  const int64_t g_stride = static_cast<int64_t>(a.H_v) * (KDA ? D : 1), b_stride = a.H_v;

  // ---- set-up: barriers and tensor memory ----
  if (tid == 0) {
    mbar_init(&misc->bar_ap, 1);
    mbar_init(&misc->bar_ro, 1);
    mbar_init(&misc->bar_u, 1);
    mbar_init(&misc->bar_o, 1);
    mbar_init(&misc->bar_s, 1);
    mbar_init(&misc->rdy_prep, NC);
    mbar_init(&misc->rdy_state, NC);
    mbar_init(&misc->rdy_rhs, NC);
    mbar_init(&misc->rdy_u, NC);
    misc->abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 8) {
    tmem_alloc(&misc->tmem_base, TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tm = misc->tmem_base;
  const int n_chunks = (n_tok + C - 1) / C;

  constexpr uint32_t ID_N32 = idesc_tf32(128, 32, false, false);
  constexpr uint32_t ID_N64 = idesc_tf32(128, 64, false, false);
  constexpr uint32_t ID_N128 = idesc_tf32(128, 128, false, false);

  if (warp == 8) {
    // =========================== tensor-core issue warp ===========================
    for (int ch = 0; ch < n_chunks; ++ch) {
      const uint32_t par = ch & 1;
      // MMA1: [Kt;Qt] Kh^T.  M is padded to 128: rows 64-127 of the A tile are whatever follows it in
      // shared memory, and land in TMEM lanes 64-127 that nobody reads.
      if (lane == 0) wait_bar(&misc->rdy_prep, par, misc, err);
      __syncwarp();
      if (lane == 0) {
        tc_fence_after_sync();
#pragma unroll 1
        for (int kk = 0; kk < 16; ++kk)  // K = 128 in slices of 8: block kk / 4, 32 bytes per slice inside a block
          mma_ss(tm + COL_AP, desc_kmajor(sbase + OFF_KQ + (kk >> 2) * (64 * 128) + (kk & 3) * 32),
                 desc_kmajor(sbase + OFF_KH + (kk >> 2) * (32 * 128) + (kk & 3) * 32), ID_N32, kk != 0);
        mma_commit(&misc->bar_ap);
      }
      // MMA2: S'^T [Kt;Qt]^T, the fp32 state read as a tf32 operand
      if (lane == 0) wait_bar(&misc->rdy_state, par, misc, err);
      __syncwarp();
      if (lane == 0) {
        tc_fence_after_sync();
#pragma unroll 1
        for (int kk = 0; kk < 16; ++kk)
          mma_ts(tm + COL_RO, tm + COL_S + kk * 8, desc_kmajor(sbase + OFF_KQ + (kk >> 2) * (64 * 128) + (kk & 3) * 32),
                 go ? ID_N64 : ID_N32, kk != 0);  // without outputs only the Kt rows are needed
        mma_commit(&misc->bar_ro);
      }
      // MMA3: U^T = RHS^T T^T; RHS^T is a tf32 pair (high part over R^T, low part in the A|P columns)
      if (lane == 0) wait_bar(&misc->rdy_rhs, par, misc, err);
      __syncwarp();
      if (lane == 0) {
        tc_fence_after_sync();
#pragma unroll 1
        for (int kk = 0; kk < 8; ++kk)
          mma_ts(tm + COL_U, tm + (kk < 4 ? COL_RO : COL_AP) + (kk & 3) * 8, desc_kmajor(sbase + OFF_TM + (kk & 3) * 32),
                 ID_N32, kk != 0);
        mma_commit(&misc->bar_u);
      }
      // MMA4: O^T += U^T P^T (high part of U);  MMA5: S'^T += U^T Kh (U as a pair: high in place, low over RHS^T)
      if (lane == 0) wait_bar(&misc->rdy_u, par, misc, err);
      __syncwarp();
      if (lane == 0) {
        tc_fence_after_sync();
        if (go) {
#pragma unroll 1
          for (int kk = 0; kk < 4; ++kk)
            mma_ts(tm + COL_RO + 32, tm + COL_U + kk * 8, desc_kmajor(sbase + OFF_PM + kk * 32), ID_N32, true);
        }
        mma_commit(&misc->bar_o);
#pragma unroll 1
        for (int kk = 0; kk < 8; ++kk)
          mma_ts(tm + COL_S, tm + (kk < 4 ? COL_U : COL_RO) + (kk & 3) * 8, desc_kmajor(sbase + OFF_KHT + (kk & 3) * 32),
                 ID_N128, true);
        mma_commit(&misc->bar_s);
      }
      __syncwarp();
    }
  } else {
    // =============================== compute warps ===============================
    const int quad = warp & 3, colh = warp >> 2;                           // TMEM lane quadrant, column half
    const uint32_t tlane = tm + (static_cast<uint32_t>(quad * 32) << 16);  // this warp's TMEM lanes
    const int vrow = quad * 32 + lane;                                     // the TMEM lane this thread owns
    constexpr float LOG2E = 1.4426950408889634f;
    PT_DECL

    // cp.async stages of one chunk's inputs
    auto stage_qk = [&](int ch) {
      const int t0 = ch * C, ntok = min(C, n_tok - t0);
      for (int i = tid; i < C * 16; i += NC) {
        const int t = i >> 4, j = i & 15;
        const bool valid = t < ntok;
        const int64_t tt = t0 + (valid ? t : 0);
        if (go)  // no outputs wanted: q is never read
          cp_async16_zfill(sbase + OFF_RAWQ + t * 256 + j * 16, reinterpret_cast<const char *>(gq + tt * qk_stride) + j * 16, valid);
        cp_async16_zfill(sbase + OFF_RAWK + t * 256 + j * 16, reinterpret_cast<const char *>(gk + tt * qk_stride) + j * 16, valid);
      }
    };
    auto stage_g = [&](int ch) {
      const int t0 = ch * C, ntok = min(C, n_tok - t0);
      if constexpr (KDA) {
        for (int i = tid; i < C * 32; i += NC) {
          const int t = i >> 5, j = i & 31;
          const bool valid = t < ntok;
          cp_async16_zfill(sbase + OFF_G + t * 512 + j * 16,
                           reinterpret_cast<const char *>(gg + (t0 + (valid ? t : 0)) * g_stride) + j * 16, valid);
        }
      }
    };
    auto stage_v = [&](int ch) {
      const int t0 = ch * C, ntok = min(C, n_tok - t0);
      for (int i = tid; i < C * 16; i += NC) {
        const int t = i >> 4, j = i & 15;
        const bool valid = t < ntok;
        cp_async16_zfill(sbase + OFF_V + t * 256 + j * 16,
                         reinterpret_cast<const char *>(gv + (t0 + (valid ? t : 0)) * v_stride) + j * 16, valid);
      }
    };
    // per-token scalars of a chunk (beta, and the scalar log-decay of GDN): threads 0-31 / 32-63
    auto load_scalar = [&](int ch) -> float {
      const int t0 = ch * C, ntok = min(C, n_tok - t0);
      if (tid < C) return tid < ntok ? gb[(t0 + tid) * b_stride] : 0.f;
      if (!KDA && tid < 2 * C) return (tid - C) < ntok ? gg[(t0 + tid - C) * g_stride] : 0.f;
      return 0.f;
    };
    auto store_scalar = [&](int ch, float x) {
      if (tid < C) beta_s[(ch & 1) * C + tid] = x;
      else if (!KDA && tid < 2 * C) gsc_s[(ch & 1) * C + tid - C] = x;
    };

    if (n_chunks > 0) {
      stage_qk(0);
      stage_g(0);
      asm volatile("cp.async.commit_group;" ::: "memory");
      store_scalar(0, load_scalar(0));
    }
    post_s[tid] = 0.f;  // [2][128]: nothing owed before the first chunk
    // the start state goes into TMEM as it is; the first chunk's state pass scales it like any other
    if (n_chunks > 0) {
#pragma unroll 1
      for (int c0 = colh * 64; c0 < colh * 64 + 64; c0 += 32) {
        uint32_t s[32];
        if (a.mode == DASC_REFRESH_CONTINUE) {
#pragma unroll
          for (int j = 0; j < 32; ++j) s[j] = __float_as_uint(st[(c0 + j) * D + vrow]);
        } else {
#pragma unroll
          for (int j = 0; j < 32; ++j) s[j] = 0u;
        }
        tmem_st32(tlane + COL_S + c0, s);
      }
      tmem_st_wait();
    }

    for (int ch = 0; ch < n_chunks; ++ch) {
      const uint32_t par = ch & 1;
      const int t0 = ch * C;
      const int ntok = min(C, n_tok - t0);
      const bool more = ch + 1 < n_chunks;
      const float *beta_c = beta_s + par * C;

      // ---- (1) this chunk's inputs have landed; the previous chunk's state update is complete ----
      if (ch > 0) wait_bar(&misc->bar_s, par ^ 1, misc, err);
      tc_fence_after_sync();
      asm volatile("cp.async.wait_all;" ::: "memory");
      sync_compute();
      const float scalar_next = more ? load_scalar(ch + 1) : 0.f;  // in flight during the chunk
      PT(0);

      // ---- (2) prep: warp = (block of 32 channels, half of the tokens); lane = (4 adjacent channels, 4 consecutive
      //          tokens), a 4 x 4 tile, so that Kh can also be stored transposed.  The midpoint is the end of the
      //          first half: first-half exponents are (local sum - the half's total), second-half exponents the
      //          local sums themselves. ----
      {
        const int cq = lane & 7, tg = lane >> 3, half = warp >> 2;
        const int c0 = (warp & 3) * 32 + cq * 4, t4 = half * 16 + tg * 4;
        // all shared-memory reads of the tile before its first write
        uint2 kraw[4], qraw[4];
        float gl[4][4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          kraw[j] = *reinterpret_cast<const uint2 *>(smem + OFF_RAWK + (t4 + j) * 256 + c0 * 2);
          qraw[j] = go ? *reinterpret_cast<const uint2 *>(smem + OFF_RAWQ + (t4 + j) * 256 + c0 * 2) : make_uint2(0u, 0u);
          if constexpr (KDA) {
            const float4 g4 = *reinterpret_cast<const float4 *>(smem + OFF_G + (t4 + j) * 512 + c0 * 4);
            gl[j][0] = g4.x; gl[j][1] = g4.y; gl[j][2] = g4.z; gl[j][3] = g4.w;
          } else {
            const float gs = gsc_s[par * C + t4 + j];
            gl[j][0] = gs; gl[j][1] = gs; gl[j][2] = gs; gl[j][3] = gs;
          }
        }
        const float4 post_prev = *reinterpret_cast<const float4 *>(post_s + (par ^ 1) * D + c0);
        // this lane's total, the prefix over the four token groups of the warp (lanes 8 apart), the half's total
        float run[4], refL[4], tot[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          float incl = gl[0][i] + gl[1][i] + gl[2][i] + gl[3][i];
          const float own = incl;
          float x = __shfl_up_sync(0xffffffffu, incl, 8);
          if (tg >= 1) incl += x;
          x = __shfl_up_sync(0xffffffffu, incl, 16);
          if (tg >= 2) incl += x;
          run[i] = incl - own;                               // accumulated before this lane's first token
          tot[i] = __shfl_sync(0xffffffffu, incl, cq + 24);   // the half's total
          refL[i] = half == 0 ? tot[i] * LOG2E : 0.f;
        }
        if (tg == 0) {
          if (half == 0)
            *reinterpret_cast<float4 *>(fac_s + c0) =
                make_float4(ex2f((post_prev.x + tot[0]) * LOG2E), ex2f((post_prev.y + tot[1]) * LOG2E),
                            ex2f((post_prev.z + tot[2]) * LOG2E), ex2f((post_prev.w + tot[3]) * LOG2E));
          else
            *reinterpret_cast<float4 *>(post_s + par * D + c0) = make_float4(tot[0], tot[1], tot[2], tot[3]);  // G_C - G_m
        }
        uint32_t kht[4][4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int t = t4 + j;
          const uint2 kw = kraw[j], qw = qraw[j];
          const float kf[4] = {bf16lo(kw.x), bf16hi(kw.x), bf16lo(kw.y), bf16hi(kw.y)};
          const float qf[4] = {bf16lo(qw.x), bf16hi(qw.x), bf16lo(qw.y), bf16hi(qw.y)};
          uint32_t kt[4], qt[4], kh[4];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            run[i] += gl[j][i];
            const float d = fmaf(run[i], LOG2E, -refL[i]);      // (G_t - G_m) log2(e)
            const float e1 = ex2f(d + kLog2TruncComp), e2 = ex2f(-d);
            kt[i] = tf32_pre(kf[i] * e1);
            qt[i] = tf32_pre(qf[i] * a.q_scale * e1);
            kh[i] = tf32_pre(kf[i] * e2);
            kht[i][j] = kh[i];
          }
          *reinterpret_cast<uint4 *>(smem + OFF_KQ + sw128_offset(64, t, c0)) = make_uint4(kt[0], kt[1], kt[2], kt[3]);
          if (go) *reinterpret_cast<uint4 *>(smem + OFF_KQ + sw128_offset(64, 32 + t, c0)) = make_uint4(qt[0], qt[1], qt[2], qt[3]);
          *reinterpret_cast<uint4 *>(smem + OFF_KH + sw128_offset(32, t, c0)) = make_uint4(kh[0], kh[1], kh[2], kh[3]);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i)
          *reinterpret_cast<uint4 *>(smem + OFF_KHT + sw128_offset(128, c0 + i, t4)) =
              make_uint4(kht[i][0], kht[i][1], kht[i][2], kht[i][3]);
      }
      fence_smem_to_async();
      tc_fence_before_sync();
      mbar_arrive(&misc->rdy_prep);  // -> MMA1
      sync_compute();                // fac_s visible; raw q/k/g consumed by everyone
      stage_v(ch);                   // V of this chunk takes the place of the raw log-decay tile
      asm volatile("cp.async.commit_group;" ::: "memory");
      if (more) stage_qk(ch + 1);
      asm volatile("cp.async.commit_group;" ::: "memory");
      PT(1);

      // ---- (3) state pass: thread = (value column v, half of the channels); scale the state to this chunk's midpoint ----
      {
        // kept as a real loop (and every other per-chunk phase as compact as possible): the chunk loop is
        // executed once per 32 tokens by every warp, so its code size decides the instruction-fetch cost
#pragma unroll 1
        for (int c0 = colh * 64; c0 < colh * 64 + 64; c0 += 32) {
          uint32_t s[32];
          tmem_ld32(tlane + COL_S + c0, s);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 32; j += 4) {
            const float4 f = *reinterpret_cast<const float4 *>(fac_s + c0 + j);
            s[j + 0] = __float_as_uint(__uint_as_float(s[j + 0]) * f.x);
            s[j + 1] = __float_as_uint(__uint_as_float(s[j + 1]) * f.y);
            s[j + 2] = __float_as_uint(__uint_as_float(s[j + 2]) * f.z);
            s[j + 3] = __float_as_uint(__uint_as_float(s[j + 3]) * f.w);
          }
          tmem_st32(tlane + COL_S + c0, s);
        }
        tmem_st_wait();
      }
      tc_fence_before_sync();
      mbar_arrive(&misc->rdy_state);  // -> MMA2
      PT(2);

      // ---- (4) A and P out of TMEM; T = (I + A)^-1, by warp 0 (A) and warp 1 (P) ----
      wait_bar(&misc->bar_ap, par, misc, err);
      tc_fence_after_sync();
      PT(3);
      if (warp < 2) {
        uint32_t x[32];
        tmem_ld32(tlane + COL_AP, x);
        tmem_ld_wait();
        const int t = lane;
        if (warp == 0) {
          // lanes 0-31: row t of A = strict_lower(Kt Kh^T) * beta_t, kept in fp32 for the inverse
          const float bt = beta_c[t] * kInvTruncComp;
#pragma unroll
          for (int j = 0; j < 32; j += 4) {
            float4 o;
            o.x = (j + 0 < t) ? bt * __uint_as_float(x[j + 0]) : 0.f;
            o.y = (j + 1 < t) ? bt * __uint_as_float(x[j + 1]) : 0.f;
            o.z = (j + 2 < t) ? bt * __uint_as_float(x[j + 2]) : 0.f;
            o.w = (j + 3 < t) ? bt * __uint_as_float(x[j + 3]) : 0.f;
            *reinterpret_cast<float4 *>(Lm + t * LDX + j) = o;
          }
          __syncwarp();
          // diagonal 16x16 blocks: lane (block b, column cc) solves (I + L_bb) x = e_cc by forward substitution
          {
            const int b = lane >> 4, cc = lane & 15;
            const float *Lb = Lm + (b * 16) * LDX + b * 16;
            float xs[16];
#pragma unroll
            for (int rr = 0; rr < 16; ++rr) {
              float acc0 = (rr == cc) ? 1.f : 0.f, acc1 = 0.f;
#pragma unroll
              for (int j = 0; j + 1 < rr; j += 2) {
                acc0 = fmaf(-Lb[rr * LDX + j], xs[j], acc0);
                acc1 = fmaf(-Lb[rr * LDX + j + 1], xs[j + 1], acc1);
              }
              if (rr & 1) acc0 = fmaf(-Lb[rr * LDX + rr - 1], xs[rr - 1], acc0);
              xs[rr] = acc0 + acc1;
            }
#pragma unroll
            for (int rr = 0; rr < 16; ++rr) Xm[(b * 16 + rr) * LDX + b * 16 + cc] = xs[rr];
          }
          __syncwarp();
          // off-diagonal block: X_10 = -X_11 (L_10 X_00); the product L_10 X_00 is parked in the unused block (0,1)
          {
            float acc[2][4] = {};
            warp_mm_acc(acc, Lm + 16 * LDX, Xm, lane);
            warp_mm_store(Xm + 16, acc, 1.f, lane);
            __syncwarp();
            float acc2[2][4] = {};
            warp_mm_acc(acc2, Xm + 16 * LDX + 16, Xm + 16, lane);
            warp_mm_store(Xm + 16 * LDX, acc2, -1.f, lane);
          }
        } else if (go) {
          // lanes 32-63: row t of P = lower_incl_diag(Qt Kh^T), straight to its operand tile
#pragma unroll
          for (int j = 0; j < 32; j += 4) {
            uint4 o;
            o.x = (j + 0 <= t) ? tf32_pre(__uint_as_float(x[j + 0]) * kInvTruncComp) : 0u;
            o.y = (j + 1 <= t) ? tf32_pre(__uint_as_float(x[j + 1]) * kInvTruncComp) : 0u;
            o.z = (j + 2 <= t) ? tf32_pre(__uint_as_float(x[j + 2]) * kInvTruncComp) : 0u;
            o.w = (j + 3 <= t) ? tf32_pre(__uint_as_float(x[j + 3]) * kInvTruncComp) : 0u;
            *reinterpret_cast<uint4 *>(smem + OFF_PM + sw128_offset(32, t, j)) = o;
          }
        }
      }
      sync_compute();
      PT(4);
      {
        // T (lower triangle of X, unit diagonal) -> tf32 operand tile; 4 elements per thread
        const int t = tid >> 3, i0 = (tid & 7) * 4;
#pragma unroll
        for (int j = 0; j < 4; j += 4) {
          const float4 xv = *reinterpret_cast<const float4 *>(Xm + t * LDX + i0 + j);
          uint4 o;
          o.x = (i0 + j + 0 <= t) ? tf32_pre(xv.x) : 0u;
          o.y = (i0 + j + 1 <= t) ? tf32_pre(xv.y) : 0u;
          o.z = (i0 + j + 2 <= t) ? tf32_pre(xv.z) : 0u;
          o.w = (i0 + j + 3 <= t) ? tf32_pre(xv.w) : 0u;
          *reinterpret_cast<uint4 *>(smem + OFF_TM + sw128_offset(32, t, i0 + j)) = o;
        }
      }
      fence_smem_to_async();
      PT(5);

      // ---- (5) RHS^T = beta (V - R)^T as a tf32 pair: high over R^T, low in the consumed A|P columns ----
      wait_bar(&misc->bar_ro, par, misc, err);
      tc_fence_after_sync();
      asm volatile("cp.async.wait_group 1;" ::: "memory");  // V of this chunk (the newer group is the next q, k)
      sync_compute();
      PT(6);
      {
        const int tb = colh * 16;
        uint32_t x[16], lo[16];
        tmem_ld16(tlane + COL_RO + tb, x);
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const float vv = __bfloat162float(Vs[(tb + j) * D + vrow]);
          const float rhs = beta_c[tb + j] * (vv - __uint_as_float(x[j]));
          x[j] = to_tf32(rhs);
          lo[j] = tf32_pre(rhs - __uint_as_float(x[j]));
        }
        tmem_st16(tlane + COL_RO + tb, x);
        tmem_st16(tlane + COL_AP + tb, lo);
        tmem_st_wait();
      }
      tc_fence_before_sync();
      mbar_arrive(&misc->rdy_rhs);  // -> MMA3 (T tile and RHS^T are ready)
      sync_compute();               // everyone is done with V: the next chunk's log-decay tile may land
      if (more) stage_g(ch + 1);
      asm volatile("cp.async.commit_group;" ::: "memory");
      PT(7);

      // ---- (6) U^T as a tf32 pair: high in place, low over the consumed RHS^T ----
      wait_bar(&misc->bar_u, par, misc, err);
      tc_fence_after_sync();
      PT(8);
      {
        const int tb = colh * 16;
        uint32_t x[16], lo[16];
        tmem_ld16(tlane + COL_U + tb, x);
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const float u = __uint_as_float(x[j]);
          x[j] = to_tf32(u);
          lo[j] = tf32_pre(u - __uint_as_float(x[j]));
        }
        tmem_st16(tlane + COL_U + tb, x);
        tmem_st16(tlane + COL_RO + tb, lo);
        tmem_st_wait();
      }
      tc_fence_before_sync();
      mbar_arrive(&misc->rdy_u);  // -> MMA4, MMA5
      PT(9);

      // ---- (7) outputs of this chunk ----
      wait_bar(&misc->bar_o, par, misc, err);
      tc_fence_after_sync();
      PT(10);
      if (go) {
        const int tb = colh * 16;
        uint32_t x[16];
        tmem_ld16(tlane + COL_RO + 32 + tb, x);
        tmem_ld_wait();
        if constexpr (sizeof(OT) == 2) {
          // through shared memory (the Kt/Qt tile is free now) so that global stores are 16 bytes wide
          __nv_bfloat16 *Os = reinterpret_cast<__nv_bfloat16 *>(smem + OFF_KQ);
#pragma unroll
          for (int j = 0; j < 16; ++j) Os[(tb + j) * D + vrow] = __float2bfloat16_rn(__uint_as_float(x[j]));
          sync_compute();
          for (int i = tid; i < ntok * 16; i += NC) {
            const int t = i >> 4, j = i & 15;
            *reinterpret_cast<uint4 *>(reinterpret_cast<char *>(go + (t0 + t) * v_stride) + j * 16) =
                *reinterpret_cast<const uint4 *>(smem + OFF_KQ + t * 256 + j * 16);
          }
        } else {
#pragma unroll
          for (int j = 0; j < 16; ++j)
            if (tb + j < ntok) go[(t0 + tb + j) * v_stride + vrow] = __uint_as_float(x[j]);
        }
      }
      store_scalar(ch + 1, scalar_next);
      tc_fence_before_sync();
      sync_compute();  // every thread is done with this chunk's tiles before they are rewritten
      PT(11);
    }

    // ---- final state: the factor still owed, then write back ----
    if (n_chunks > 0) wait_bar(&misc->bar_s, (n_chunks - 1) & 1, misc, err);
    if (tid < D) fac_s[tid] = ex2f(post_s[((n_chunks + 1) & 1) * D + tid] * LOG2E);
    sync_compute();
    tc_fence_after_sync();
    {
      const uint8_t *keep = a.row_keep + static_cast<int64_t>(layer) * a.rows_per_layer + static_cast<int64_t>(h) * D;
      const bool merge = a.mode != DASC_REFRESH_CONTINUE;
#pragma unroll 1
      for (int c0 = colh * 64; c0 < colh * 64 + 64; c0 += 32) {
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
          if (!merge || !keep[c]) st[c * D + vrow] = __uint_as_float(s[j]) * fac_s[c];
        }
      }
    }
    PT(12);
    PT_DUMP;
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 8) tmem_dealloc(tm, TMEM_COLS);
}

template <bool KDA, typename OT, bool WITH_O>
int launch(const DascRefreshArgs &a, void *stream) {
  auto kern = refresh_chunked_kernel<KDA, OT, WITH_O>;
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
  if (!a.o) return kda ? launch<true, __nv_bfloat16, false>(a, stream) : launch<false, __nv_bfloat16, false>(a, stream);
  if (a.o_bf16) return kda ? launch<true, __nv_bfloat16, true>(a, stream) : launch<false, __nv_bfloat16, true>(a, stream);
  return kda ? launch<true, float, true>(a, stream) : launch<false, float, true>(a, stream);
}

// ---------------------------------------------------------------------------------------------
// dasc_refresh_static: the chunked refresh without any caller-provided workspace.
// ---------------------------------------------------------------------------------------------
namespace {

// Scratch of the static variant.  It lives in the library image: every GPU that loads libdasc
// holds these bytes until the process exits.  In host code the name below is only a handle; the
// device address is obtained once per device with cudaGetSymbolAddress.
constexpr size_t kStaticScratchBytes = 4096;
static __device__ __align__(256) unsigned char g_refresh_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
void *g_static_scratch_addr[kMaxDevices] = {};  // device address per CUDA device, filled on first use

// Device address of the static scratch on the CURRENT device; resolves it on the first call.
cudaError_t static_scratch_address(void **out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  void *p = __atomic_load_n(&g_static_scratch_addr[dev], __ATOMIC_ACQUIRE);
  if (!p) {
    e = cudaGetSymbolAddress(&p, g_refresh_static_scratch);
    if (e != cudaSuccess) return e;
    __atomic_store_n(&g_static_scratch_addr[dev], p, __ATOMIC_RELEASE);  // racing first calls store the same value
  }
  *out = p;
  return cudaSuccess;
}

}  // namespace

extern "C" dasc_status_t dasc_refresh_static(const dasc_plan_t *plan, float *state_base, int64_t layer_stride,
                                             int64_t req_stride, const int32_t *req_idx, const void *q, const void *k,
                                             const void *v, const float *g, const float *beta,
                                             const int32_t *cu_seqlens, int32_t n_req, int64_t total_tokens,
                                             int32_t max_seqlen, int32_t layer_begin, int32_t layer_end, float q_scale,
                                             void *o, int32_t o_dtype, int32_t mode, void **scratch_out,
                                             void *cuda_stream) {
  if (scratch_out) *scratch_out = nullptr;
  if (!plan || plan->info.device < 0) return DASC_ERR_INVALID_ARG;
  if (n_req < 0 || total_tokens < 0 || max_seqlen < 0) return DASC_ERR_INVALID_ARG;
  if (layer_begin < 0 || layer_end < layer_begin || layer_end > plan->info.n_layers) return DASC_ERR_INVALID_ARG;
  if (o && o_dtype != DASC_IO_BF16 && o_dtype != DASC_IO_FP32) return DASC_ERR_INVALID_ARG;
  if (mode != DASC_REFRESH_CONTINUE && mode != DASC_REFRESH_SCRATCH_MERGE_LOCAL) return DASC_ERR_INVALID_ARG;
  if (plan->info.d_k != D || plan->info.d_v != D) return DASC_ERR_SHAPE;  // the chunked kernel's shape
  // The scratch this request would need from a caller must fit the static array.
  const size_t need = dasc_refresh_chunked_workspace_bytes(n_req, layer_end - layer_begin, plan->info.n_v_heads);
  if (need > kStaticScratchBytes) return DASC_ERR_WORKSPACE;
  void *scratch = nullptr;
  if (static_scratch_address(&scratch) != cudaSuccess) return DASC_ERR_CUDA;
  if (scratch_out) *scratch_out = scratch;
  if (n_req == 0 || layer_end == layer_begin || total_tokens == 0) return DASC_OK;
  if (!state_base || !req_idx || !q || !k || !v || !g || !beta || !cu_seqlens) return DASC_ERR_INVALID_ARG;
  auto misaligned = [](const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; };
  if (misaligned(state_base) || misaligned(q) || misaligned(k) || misaligned(v) || misaligned(g) || (o && misaligned(o)))
    return DASC_ERR_INVALID_ARG;
  if (layer_stride < 0 || req_stride < 0 || layer_stride % 4 || req_stride % 4) return DASC_ERR_INVALID_ARG;

  DascRefreshArgs a{};
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
  a.io_bf16 = 1;
  a.g = g;
  a.beta = beta;
  a.cu_seqlens = cu_seqlens;
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
  a.workspace = scratch;  // the launcher clears the time-out flag (first word) on the stream
  a.workspace_bytes = kStaticScratchBytes;
  const int e = dasc_launch_refresh_chunked(a, cuda_stream);
  if (e == -1) return DASC_ERR_SHAPE;
  return e == 0 ? DASC_OK : DASC_ERR_CUDA;
}
