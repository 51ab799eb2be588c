// Suffix refresh, chunked form, on the Blackwell tensor cores (tcgen05 + TMEM), warp-specialised:
// 32-token chunks, two CTAs resident per SM, four roles per CTA.
//
// Eq. 1 (transposed orientation) over a chunk of C = 32 tokens starting from S_0, with
// G_t the running sum of the log-decay inside the chunk and m the chunk midpoint:
//   Kt_t = k_t * exp(G_t - G_m),  Kh_t = k_t * exp(G_m - G_t),  Qt_t = q_t * exp(G_t - G_m)
//   S'   = Diag(exp(G_m)) S_0                                   (state decayed to the midpoint)
//   A    = strict_lower(Kt Kh^T) * beta,   P = lower_incl_diag(Qt Kh^T)
//   U    = (I + A)^-1 * beta * (V - Kt S')                      (the deltas written at each token)
//   O    = Qt S' + P U
//   S_C  = Diag(exp(G_C - G_m)) (S' + Kh^T U)
//
// Roles.  The operand tiles Kt, Qt, Kh depend on the token inputs only, not on the state, so they
// are built one chunk ahead by four PRODUCER warps; their inputs land in the tiles they become (the
// KDA log-decay by TMA, k and q by cp.async), off the critical path.  One TRIANGULAR warp forms
// T = (I + A)^-1, also state-independent.  Eight CHAIN warps carry the state-dependent sequence:
// state rescale -> right-hand side -> deltas -> outputs.  One warp issues all tensor-core work.
// The groups meet only at mbarriers.  GDN (one scalar log-decay per token) keeps the decay out of
// the products: MMA1 and MMA2 run on the raw k, q and the per-token factors are applied where A, P,
// k S' and the outputs leave tensor memory.
//   MMA1  [Kt;Qt] Kh^T            -> A (lanes 0-31) and P (lanes 32-63)         smem x smem
//   MMA2  S'^T [Kt;Qt]^T          -> R^T | (Qt S')^T                            tmem x smem
//   MMA3  RHS^T T^T               -> U^T      (RHS as a tf32 high/low pair)     tmem x smem
//   MMA4  (Qt S')^T += U^T P^T    -> O^T                                         tmem x smem
//   MMA5  S'^T      += U^T Kh     -> state    (U as a tf32 high/low pair)       tmem x smem
// Buffers: the Kt/Qt and Kh tiles of chunk n+1 may be written once MMA2 of chunk n has completed
// (MMA1 and MMA2 are their only readers); MMA5 contracts over the tokens and reads Kh as an MN-major
// operand from a second tile (tf32 MN-major operands have a swizzle of their own), which, read last,
// is double-buffered by chunk parity.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "dasc_internal.h"
#include "tcgen05_util.cuh"

namespace {

using namespace tc5;

constexpr int C = 32;          // chunk length
constexpr int D = 128;         // d_k = d_v
constexpr int NCH = 256;       // chain threads (warps 0-7)
constexpr int NP = 128;        // producer threads (warps 8-11)
constexpr int WARP_T = 12;     // the warp that inverts the triangular system
constexpr int WARP_MMA = 13;   // the warp that issues tensor-core work
constexpr int NT = NCH + NP + 64;
constexpr int LDX = 36;        // row pitch (floats) of the fp32 triangular work matrices
constexpr uint32_t TMEM_COLS = 256;

// TMEM columns
constexpr uint32_t COL_S = 0, COL_AP = 128, COL_RO = 160, COL_U = 224;  // RO: R^T 160-191 | (Qt S')^T 192-223

// shared memory map (bytes)
constexpr uint32_t OFF_KQ = 0;                          // [4][64 rows][128 B]  rows 0-31 Kt, 32-63 Qt
constexpr uint32_t OFF_KHT = OFF_KQ + 4 * 64 * 128;     // [2][4][32 rows][128 B] Kh[t][c] once more, as the MN-major operand of MMA5, by chunk parity
constexpr uint32_t OFF_KH = OFF_KHT + 2 * 128 * 128;    // [4][32 rows][128 B]  Kh[t][c]
constexpr uint32_t OFF_TM = OFF_KH + 4 * 32 * 128;      // [1][32 rows][128 B]  T[t][i]; TM|PM later the bf16 O tile
constexpr uint32_t OFF_PM = OFF_TM + 32 * 128;          // [1][32 rows][128 B]  P[t][i]
constexpr uint32_t OFF_V = OFF_PM + 32 * 128;           // [32][128] bf16 v
constexpr uint32_t OFF_L = OFF_V + C * D * 2;           // [32][LDX] fp32
constexpr uint32_t OFF_X = OFF_L + C * LDX * 4;         // [32][LDX] fp32
constexpr uint32_t OFF_FAC = OFF_X + C * LDX * 4;       // [2][128] fp32 state factor per channel, by chunk parity
constexpr uint32_t OFF_POST = OFF_FAC + 2 * D * 4;      // [2][128] fp32 log-factor owed after a chunk, by chunk parity
constexpr uint32_t OFF_BETA = OFF_POST + 2 * D * 4;     // [4][32] fp32, by chunk index mod 4 (written well ahead)
// GDN only, same ring as beta: per-token factors of the scalar decay, e1 = exp(G_t - G_m), e2 = exp(G_m - G_t)
constexpr uint32_t OFF_E1C = OFF_BETA + 4 * C * 4;      // [4][32] fp32 e1 * (truncation compensation)
constexpr uint32_t OFF_E2 = OFF_E1C + 4 * C * 4;        // [4][32] fp32 e2
constexpr uint32_t OFF_BTE1 = OFF_E2 + 4 * C * 4;       // [4][32] fp32 beta * e1
constexpr uint32_t OFF_MISC = OFF_BTE1 + 4 * C * 4;     // barriers, tmem base, abort flag
// GDN only: raw k (rows 0-31) and q (rows 32-63) as bf16, [2][64 rows][128 B], in the place of the K-major Kh tile
constexpr uint32_t OFF_KQ16 = OFF_KH;
constexpr uint32_t SMEM_BYTES = OFF_MISC + 192;
constexpr uint32_t SMEM_ALLOC = SMEM_BYTES + 1024;      // slack to align the base to 1024 bytes
static_assert(SMEM_ALLOC <= 113 * 1024, "two CTAs per SM");

constexpr uint32_t kMaxPolls = 1u << 22;

// The tensor core reads the fp32 state as tf32 by dropping its low 13 mantissa bits, i.e. rounding
// towards zero: on average the operand is 2^-11 * E[1/m] = 3.52e-4 too small in magnitude (m the
// significand, log-uniform in [1, 2)).  The rows of Kt and Qt, the only partners of that operand,
// are scaled up by this factor to cancel the bias; A and P, which also come from those rows, are
// scaled back down when they are taken out of TMEM.
// Largest |sum of the log-decay over half a chunk| per channel for which every factor formed relative to the chunk
// midpoint stays a normal fp32 number with room for the products that follow.
constexpr float kMaxHalfDecay = 80.f;

constexpr float kTruncComp = 1.000352f;
constexpr float kInvTruncComp = 1.0f / kTruncComp;
constexpr float kLog2TruncComp = 5.0774e-4f;  // log2(kTruncComp)

struct Misc {
  // tensor core -> chain warps (one tcgen05.commit each per chunk); bar_ro also releases the producer
  uint64_t bar_ap, bar_ro, bar_u, bar_o, bar_s;
  // producer -> issuing warp and chain warps (128 arrivals per chunk)
  uint64_t rdy_prep;
  // producer -> chain warps: the state factors of a chunk are ready (128 arrivals per chunk)
  // One barrier per chunk parity: the producer may hand over the factors of chunk n+1 before the chain warps
  // have waited for those of chunk n, and a single barrier cannot tell phases two apart.
  uint64_t rdy_fac[2];
  // chain warps -> issuing warp (256 arrivals each per chunk)
  uint64_t rdy_state, rdy_rhs, rdy_u;
  // triangular warp -> chain warps (A has left TMEM: 32 arrivals) and -> issuing warp (T tile ready: 32 arrivals)
  uint64_t a_taken, rdy_t;
  // chain warps -> triangular warp: the T|P tile region is free again (256 arrivals per chunk)
  uint64_t tp_free;
  // issuing thread, only after a wait has run out: arrives once every tensor-core product issued so far has completed
  uint64_t drain;
  // TMA -> producer warps: the log-decay tile of a chunk has landed in the Kh tile (KDA)
  uint64_t g_full;
  uint32_t tmem_base;
  volatile uint32_t abort_flag;   // a bounded wait ran out: every later wait of this CTA returns at once
  volatile uint32_t domain_flag;  // a half-chunk decay sum left the range the midpoint factors can carry
};
static_assert(sizeof(Misc) <= 192, "Misc outgrew its shared-memory slot");

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ void cp_async16_zfill(uint32_t smem, const void *gmem, bool valid) {
  const uint32_t n = valid ? 16u : 0u;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem), "l"(gmem), "r"(n) : "memory");
}

__device__ __forceinline__ void cp_async8_zfill(uint32_t smem, const void *gmem, bool valid) {
  const uint32_t n = valid ? 8u : 0u;
  asm volatile("cp.async.ca.shared.global [%0], [%1], 8, %2;" ::"r"(smem), "l"(gmem), "r"(n) : "memory");
}

__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// barrier among the 256 chain threads only
__device__ __forceinline__ void sync_chain() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

// Bounded wait; after one time-out every later wait of this CTA returns at once.
__device__ __forceinline__ void wait_bar(uint64_t *bar, uint32_t parity, Misc *misc, uint32_t *err) {
  if (misc->abort_flag) return;
  if (!mbar_wait_bounded(bar, parity, kMaxPolls)) {
    misc->abort_flag = 1;
    if (err) atomicExch(err, 1u);
  }
}

// The test hook's wait (one call site): `max_polls` non-blocking looks at the barrier, so that a short limit runs out
// whatever the time slice of a blocking poll is.
__device__ __forceinline__ void wait_bar_short(uint64_t *bar, uint32_t parity, Misc *misc, uint32_t *err, uint32_t max_polls) {
  bool done = false;
  for (uint32_t i = 0; i < max_polls && !done; ++i) done = mbar_test_wait(bar, parity);
  if (!done) {
    misc->abort_flag = 1;
    if (err) atomicExch(err, 1u);
  }
}

// This CTA does not (or could not) replay its unit: put the unit on the list that the token-by-token kernel walks
// next on the same stream.  Without a list, or when it is full, or when the caller asked for this kernel alone, an
// out-of-range unit is an error (word 1).
__device__ __forceinline__ void hand_over(const DascRefreshArgs &a, bool out_of_range) {
  uint32_t *ws = static_cast<uint32_t *>(a.workspace);
  const uint32_t idx = atomicAdd(ws + 2, 1u);
  const bool listed = a.unit_list && idx < static_cast<uint32_t>(a.unit_list_cap);
  if (listed) a.unit_list[idx] = static_cast<int32_t>(blockIdx.x);
  if (!listed || (out_of_range && a.domain_is_error)) atomicExch(ws + 1, 1u);
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

// packed pairs of fp32 (one instruction per pair)
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float &lo, float &hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}

// WITH_O = false is the state-only variant (no outputs wanted): q is never read, the Qt rows, P and the
// output product are left out.
template <bool KDA, typename OT, bool WITH_O>
__global__ void __launch_bounds__(NT, 2) refresh_chunked_kernel(DascRefreshArgs a, const __grid_constant__ CUtensorMap tmap_g) {
  extern __shared__ unsigned char smem_dyn[];
  unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~uintptr_t{1023});
  const uint32_t sbase = smem_u32(smem);
  float *Lm = reinterpret_cast<float *>(smem + OFF_L);
  float *Xm = reinterpret_cast<float *>(smem + OFF_X);
  float *fac_s = reinterpret_cast<float *>(smem + OFF_FAC);
  float *post_s = reinterpret_cast<float *>(smem + OFF_POST);
  float *beta_s = reinterpret_cast<float *>(smem + OFF_BETA);
  float *e1c_s = reinterpret_cast<float *>(smem + OFF_E1C);
  float *e2_s = reinterpret_cast<float *>(smem + OFF_E2);
  float *bte1_s = reinterpret_cast<float *>(smem + OFF_BTE1);
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
  if (n_tok <= a.short_thr) {  // left to the exact kernel (short_thr = -1: never)
    if (tid == 0) hand_over(a, false);
    return;
  }

  float *st = a.state + static_cast<int64_t>(a.req_idx[r]) * a.req_stride + static_cast<int64_t>(layer) * a.layer_stride +
              static_cast<int64_t>(h) * D * D;
  const int64_t tok0 = static_cast<int64_t>(lc) * a.total_tokens + t_begin;
  const __nv_bfloat16 *gq = static_cast<const __nv_bfloat16 *>(a.q) + (tok0 * a.H_k + hk) * D;
  const __nv_bfloat16 *gk = static_cast<const __nv_bfloat16 *>(a.k) + (tok0 * a.H_k + hk) * D;
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
    mbar_init(&misc->rdy_prep, NP);
    mbar_init(&misc->rdy_fac[0], NP);
    mbar_init(&misc->rdy_fac[1], NP);
    mbar_init(&misc->rdy_state, NCH);
    mbar_init(&misc->rdy_rhs, NCH);
    mbar_init(&misc->rdy_u, NCH);
    mbar_init(&misc->a_taken, 32);
    mbar_init(&misc->rdy_t, 32);
    mbar_init(&misc->tp_free, NCH);
    mbar_init(&misc->drain, 1);
    mbar_init(&misc->g_full, 1);
    misc->abort_flag = 0;
    misc->domain_flag = 0;
    fence_mbar_init();
  }
  if (warp == WARP_MMA) {
    tmem_alloc(&misc->tmem_base, TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tm = misc->tmem_base;
  const int n_chunks = (n_tok + C - 1) / C;
  constexpr float LOG2E = 1.4426950408889634f;

  constexpr uint32_t ID_N32 = idesc_tf32(128, 32, false, false);
  constexpr uint32_t ID_BF16_N32 = idesc_bf16(128, 32);
  constexpr uint32_t ID_N64 = idesc_tf32(128, 64, false, false);
  constexpr uint32_t ID_N128_MN = idesc_tf32(128, 128, false, true);  // B = Kh[t][c]: the channel index N is the contiguous one

  if (warp == WARP_MMA) {
    // =========================== tensor-core issue warp ===========================
    for (int ch = 0; ch < n_chunks; ++ch) {
      const uint32_t par = ch & 1;
      // MMA1: [Kt;Qt] Kh^T.  M is padded to 128: rows 64-127 of the A tile are whatever follows it in
      // shared memory, and land in TMEM lanes 64-127 that nobody reads.
      if (lane == 0) {
        if (ch == 0 && a.poll_limit_first_wait)
          wait_bar_short(&misc->rdy_prep, par, misc, err, a.poll_limit_first_wait);
        else
          wait_bar(&misc->rdy_prep, par, misc, err);
        tc_fence_after_sync();
        if constexpr (KDA) {
#pragma unroll 1
          for (int kk = 0; kk < 16; ++kk)  // K = 128 in slices of 8: block kk / 4, 32 bytes per slice inside a block
            mma_ss(tm + COL_AP, desc_kmajor(sbase + OFF_KQ + (kk >> 2) * (64 * 128) + (kk & 3) * 32),
                   desc_kmajor(sbase + OFF_KH + (kk >> 2) * (32 * 128) + (kk & 3) * 32), ID_N32, kk != 0);
        } else {
          // GDN: the decay is one scalar per token, so it is applied to A and P after the product, and the product
          // itself is [k; q] k^T on the raw bf16 inputs: exact operands, K = 16 per instruction.  A and B come from
          // the same tile (B = its first 32 rows).
#pragma unroll 1
          for (int kk = 0; kk < 8; ++kk) {
            const uint64_t d = desc_kmajor(sbase + OFF_KQ16 + (kk >> 2) * (64 * 128) + (kk & 3) * 32);
            mma_ss_bf16(tm + COL_AP, d, d, ID_BF16_N32, kk != 0);
          }
        }
        mma_commit(&misc->bar_ap);
      }
      __syncwarp();
      // MMA2: S'^T [Kt;Qt]^T, the fp32 state read as a tf32 operand
      if (lane == 0) wait_bar(&misc->rdy_state, par, misc, err);
      __syncwarp();
      if (lane == 0) {
        tc_fence_after_sync();
#pragma unroll 1
        for (int kk = 0; kk < 16; ++kk)
          mma_ts(tm + COL_RO, tm + COL_S + kk * 8, desc_kmajor(sbase + OFF_KQ + (kk >> 2) * (64 * 128) + (kk & 3) * 32),
                 WITH_O ? ID_N64 : ID_N32, kk != 0);  // without outputs only the Kt rows are needed
        mma_commit(&misc->bar_ro);
      }
      // MMA3: U^T = RHS^T T^T; RHS^T is a tf32 pair (high part over R^T, low part in the A|P columns)
      if (lane == 0) {
        wait_bar(&misc->rdy_t, par, misc, err);
        wait_bar(&misc->rdy_rhs, par, misc, err);
      }
      __syncwarp();
      if (lane == 0) {
        tc_fence_after_sync();
#pragma unroll 1
        for (int kk = 0; kk < 8; ++kk)
          mma_ts(tm + COL_U, tm + (kk < 4 ? COL_RO : COL_AP) + (kk & 3) * 8, desc_kmajor(sbase + OFF_TM + (kk & 3) * 32),
                 ID_N32, kk != 0);
        mma_commit(&misc->bar_u);
        // U^T stays where MMA3 leaves it: read as an operand, each fp32 value gives its high (truncated) part, and
        // the chain warps supply the exact remainder afterwards (U = U_hi + U_lo).  The high-part products go out at
        // once, behind MMA3 in the tensor pipe's issue order, without a round trip through the chain warps:
        // MMA4 (high): O^T += U_hi^T P^T;  MMA5 (high): S'^T += U_hi^T Kh
        if (WITH_O) {
#pragma unroll 1
          for (int kk = 0; kk < 4; ++kk)
            mma_ts(tm + COL_RO + 32, tm + COL_U + kk * 8, desc_kmajor(sbase + OFF_PM + kk * 32), ID_N32, true);
        }
#pragma unroll 1
        for (int kk = 0; kk < 4; ++kk)
          mma_ts(tm + COL_S, tm + COL_U + kk * 8, desc_mn32(sbase + OFF_KHT + par * (128 * 128) + kk * 1024, 32 * 128), ID_N128_MN, true);
      }
      // MMA4 (low), MMA5 (low): the same with U_lo^T, which the chain warps wrote over the consumed RHS^T
      if (lane == 0) wait_bar(&misc->rdy_u, par, misc, err);
      __syncwarp();
      if (lane == 0) {
        tc_fence_after_sync();
        if (WITH_O) {
#pragma unroll 1
          for (int kk = 0; kk < 4; ++kk)
            mma_ts(tm + COL_RO + 32, tm + COL_RO + kk * 8, desc_kmajor(sbase + OFF_PM + kk * 32), ID_N32, true);
        }
        mma_commit(&misc->bar_o);
#pragma unroll 1
        for (int kk = 0; kk < 4; ++kk)
          mma_ts(tm + COL_S, tm + COL_RO + kk * 8, desc_mn32(sbase + OFF_KHT + par * (128 * 128) + kk * 1024, 32 * 128), ID_N128_MN, true);
        mma_commit(&misc->bar_s);
      }
      __syncwarp();
    }
    // After a time-out the other roles no longer wait for the products: make sure none is still in flight when the
    // tensor memory is given back (a real wait, bounded like the others).
    if (lane == 0 && misc->abort_flag) {
      mma_commit(&misc->drain);
      mbar_wait_bounded(&misc->drain, 0, kMaxPolls);
    }
    __syncwarp();
  } else if (warp == WARP_T) {
    // ================================ triangular warp ================================
    // T = (I + A)^-1 depends on the token inputs only, so it is formed off the chain: A out of TMEM (lanes 0-31 are
    // this warp's quadrant), 16x16 diagonal blocks by fp32 substitution, the off-diagonal block by mma.sync products.
    const uint32_t tlane = tm;  // TMEM lanes 0-31
    for (int ch = 0; ch < n_chunks; ++ch) {
      const uint32_t par = ch & 1;
      const float *beta_c = beta_s + (ch & 3) * C;
      wait_bar(&misc->bar_ap, par, misc, err);
      tc_fence_after_sync();
      uint32_t x[32];
      tmem_ld32(tlane + COL_AP, x);
      tmem_ld_wait();
      tc_fence_before_sync();
      mbar_arrive(&misc->a_taken);  // the chain warps may reuse the A|P columns
      const int t = lane;
      // row t of A = strict_lower(Kt Kh^T) * beta_t, kept in fp32 for the inverse
      // KDA: the decay is inside the product, whose Kt rows carry the truncation compensation.  GDN: the product is
      // the raw k_t . k_j and the decay exp(G_t - G_j) = e1_t e2_j is applied here.
      const float bt = KDA ? beta_c[t] * kInvTruncComp : bte1_s[(ch & 3) * C + t];
#pragma unroll
      for (int j = 0; j < 32; j += 4) {
        float4 e2 = make_float4(1.f, 1.f, 1.f, 1.f);
        if constexpr (!KDA) e2 = *reinterpret_cast<const float4 *>(e2_s + (ch & 3) * C + j);
        float4 o;
        o.x = (j + 0 < t) ? bt * e2.x * __uint_as_float(x[j + 0]) : 0.f;
        o.y = (j + 1 < t) ? bt * e2.y * __uint_as_float(x[j + 1]) : 0.f;
        o.z = (j + 2 < t) ? bt * e2.z * __uint_as_float(x[j + 2]) : 0.f;
        o.w = (j + 3 < t) ? bt * e2.w * __uint_as_float(x[j + 3]) : 0.f;
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
      __syncwarp();
      // the T tile's storage (shared with the P tile and the chain warps' output tile) is free once the chain
      // warps have copied the previous chunk's outputs out
      if (ch > 0) wait_bar(&misc->tp_free, par ^ 1, misc, err);
      // T (lower triangle of X, unit diagonal) -> tf32 operand tile; lane = row
#pragma unroll
      for (int j = 0; j < 32; j += 4) {
        const float4 xv = *reinterpret_cast<const float4 *>(Xm + t * LDX + j);
        uint4 o;
        o.x = (j + 0 <= t) ? tf32_pre(xv.x) : 0u;
        o.y = (j + 1 <= t) ? tf32_pre(xv.y) : 0u;
        o.z = (j + 2 <= t) ? tf32_pre(xv.z) : 0u;
        o.w = (j + 3 <= t) ? tf32_pre(xv.w) : 0u;
        *reinterpret_cast<uint4 *>(smem + OFF_TM + sw128_offset(32, t, j)) = o;
      }
      fence_smem_to_async();
      mbar_arrive(&misc->rdy_t);  // -> MMA3
      __syncwarp();
    }
  } else if (warp >= 8) {
    // =============================== producer warps ===============================
    // warp = block of 32 channels; per half of the chunk, lane = (4 adjacent channels, 4 consecutive tokens), a 4 x 4
    // tile.  The midpoint is the end of the first half: first-half
    // exponents are (local sum - the half's total), second-half exponents the local sums themselves.
    const int pw = warp - 8, ptid = tid - NCH;
    const int cq = lane & 7, tg = lane >> 3;
    const int c0 = pw * 32 + cq * 4;
    // Inputs land IN the operand tiles they will be overwritten with.  The raw log-decay of a chunk comes by TMA
    // (KDA: four boxes of 32 tokens x 32 channels, 128-byte swizzle, i.e. exactly the layout of the Kh tile, so that
    // the decay of (token t, channels c0..c0+3) sits where Kh[t][c0..] goes).  Raw k and q come by cp.async, each lane
    // copying the 8-byte vectors of its own 4 x 4 tiles into the first half of the Kt / Qt vectors: a lane only ever
    // reads what it copied itself, so no barrier is needed for them, and no register holds data in flight.
    int g_issued = 0;
    float beta_next = (n_chunks > 0 && ptid < min(C, n_tok)) ? gb[ptid * b_stride] : 0.f;
    float gsc_next = (!KDA && n_chunks > 0 && ptid < min(C, n_tok)) ? gg[ptid * g_stride] : 0.f;
    float gsc_cur = 0.f, post_prev = 0.f;  // GDN, first producer warp: this chunk's log-decay, the factor owed by the previous chunk
    for (int ch = 0; ch < n_chunks; ++ch) {
      const uint32_t par = ch & 1;
      const int t0 = ch * C, ntok = min(C, n_tok - t0);
      unsigned char *kht_tile = smem + OFF_KHT + par * (128 * 128);
      // per-token scalars: this chunk's go to their ring slots (the chain warps are at most two chunks behind),
      // the next chunk's are fetched now and stored one iteration later
      if (ptid < C) {
        beta_s[(ch & 3) * C + ptid] = beta_next;
        if (!KDA) gsc_cur = gsc_next;
        const bool v1 = ch + 1 < n_chunks && ptid < min(C, n_tok - t0 - C);
        beta_next = v1 ? gb[(t0 + C + ptid) * b_stride] : 0.f;
        if (!KDA) gsc_next = v1 ? gg[(t0 + C + ptid) * g_stride] : 0.f;
      }
      // (a) raw log-decay -> Kh tile, free once MMA1 of the previous chunk has completed
      if (ch > 0) wait_bar(&misc->bar_ap, par ^ 1, misc, err);
      if constexpr (KDA) {
        if (ptid == 0 && !misc->abort_flag) {
          mbar_expect_tx(&misc->g_full, C * D * 4);
#pragma unroll
          for (int blk = 0; blk < 4; ++blk)
            tma_load_3d(sbase + OFF_KH + blk * (C * 128), &tmap_g, blk * 32, h, static_cast<int32_t>(tok0 + t0), &misc->g_full);
          ++g_issued;
        }
      } else {
        asm volatile("cp.async.commit_group;" ::: "memory");
      }
      // (b) raw k, q -> Kt/Qt tile, free once MMA2 of the previous chunk has completed; by then the chain warps
      //     have also left the chunk before that one, whose parity buffers (post, the MN-major Kh tile) are reused
      if (ch > 0) wait_bar(&misc->bar_ro, par ^ 1, misc, err);
#pragma unroll
      for (int jj = 0; jj < 8; ++jj) {
        const int t = (jj >> 2) * 16 + tg * 4 + (jj & 3);
        const bool valid = t < ntok;
        const int64_t tt = t0 + (valid ? t : 0);
        cp_async8_zfill(sbase + OFF_KQ + sw128_offset(64, t, c0), gk + tt * qk_stride + c0, valid);
        if (WITH_O) cp_async8_zfill(sbase + OFF_KQ + sw128_offset(64, 32 + t, c0), gq + tt * qk_stride + c0, valid);
      }
      asm volatile("cp.async.commit_group;" ::: "memory");
      if constexpr (KDA) {
        {
          wait_bar(&misc->g_full, par, misc, err);  // the log-decay has landed
          if (ntok < C) {
            // the box reached past the request's last token: those rows hold the decay of other tokens (or the
            // zeros past the end of the stream) and are cleared, each lane its own vectors
  #pragma unroll
            for (int jj = 0; jj < 8; ++jj) {
              const int t = (jj >> 2) * 16 + tg * 4 + (jj & 3);
              if (t >= ntok) *reinterpret_cast<float4 *>(smem + OFF_KH + sw128_offset(32, t, c0)) = make_float4(0.f, 0.f, 0.f, 0.f);
            }
          }
        }
        // sums: this lane's total, the prefix over the four token groups of the warp (lanes 8 apart), the half's total
        float run0[2][4], refL[4];
        bool out_of_range = false;
  #pragma unroll
        for (int half = 0; half < 2; ++half) {
          float own[4] = {0.f, 0.f, 0.f, 0.f};
  #pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int t = half * 16 + tg * 4 + j;
            const float4 g4 = *reinterpret_cast<const float4 *>(smem + OFF_KH + sw128_offset(32, t, c0));
            own[0] += g4.x; own[1] += g4.y; own[2] += g4.z; own[3] += g4.w;
          }
          float tot[4];
  #pragma unroll
          for (int i = 0; i < 4; ++i) {
            float incl = own[i];
            float x = __shfl_up_sync(0xffffffffu, incl, 8);
            if (tg >= 1) incl += x;
            x = __shfl_up_sync(0xffffffffu, incl, 16);
            if (tg >= 2) incl += x;
            run0[half][i] = incl - own[i];                      // accumulated before this lane's first token
            tot[i] = __shfl_sync(0xffffffffu, incl, cq + 24);    // the half's total
            if (half == 0) refL[i] = -tot[i] * LOG2E;            // minus the midpoint reference, in log2 units
            out_of_range |= !(fabsf(tot[i]) <= kMaxHalfDecay);   // also true for NaN
          }
          if (half == 0) {
            // The factor that takes the state from where the previous chunk left it to this chunk's midpoint needs
            // the first half's sums only: it is handed to the chain warps before the tiles are built.
            if (tg == 0) {
              const float4 post_prev = ch > 0 ? *reinterpret_cast<const float4 *>(post_s + (par ^ 1) * D + c0)
                                              : make_float4(0.f, 0.f, 0.f, 0.f);
              *reinterpret_cast<float4 *>(fac_s + par * D + c0) =
                  make_float4(ex2f((post_prev.x + tot[0]) * LOG2E), ex2f((post_prev.y + tot[1]) * LOG2E),
                              ex2f((post_prev.z + tot[2]) * LOG2E), ex2f((post_prev.w + tot[3]) * LOG2E));
            }
            mbar_arrive(&misc->rdy_fac[par]);
          } else if (tg == 0) {
            *reinterpret_cast<float4 *>(post_s + par * D + c0) = make_float4(tot[0], tot[1], tot[2], tot[3]);  // G_C - G_m
          }
        }
        asm volatile("cp.async.wait_group 0;" ::: "memory");  // k and q have landed
        const uint64_t l2e2 = pack2(LOG2E, LOG2E), comp2 = pack2(kLog2TruncComp, kLog2TruncComp);
        const uint64_t qs2 = pack2(a.q_scale, a.q_scale);
  #pragma unroll 1
        for (int half = 0; half < 2; ++half) {
          const int t4 = half * 16 + tg * 4;
          uint64_t run01 = half == 0 ? pack2(run0[0][0], run0[0][1]) : pack2(run0[1][0], run0[1][1]);
          uint64_t run23 = half == 0 ? pack2(run0[0][2], run0[0][3]) : pack2(run0[1][2], run0[1][3]);
          const uint64_t ref01 = half == 0 ? pack2(refL[0], refL[1]) : 0ull, ref23 = half == 0 ? pack2(refL[2], refL[3]) : 0ull;
  #pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int t = t4 + j;
            const uint32_t off_k = OFF_KQ + sw128_offset(64, t, c0), off_q = OFF_KQ + sw128_offset(64, 32 + t, c0);
            const uint32_t off_h = OFF_KH + sw128_offset(32, t, c0);
            const uint2 kw = *reinterpret_cast<const uint2 *>(smem + off_k);
            const float4 g4 = *reinterpret_cast<const float4 *>(smem + off_h);
            const uint64_t g01 = pack2(g4.x, g4.y), g23 = pack2(g4.z, g4.w);
            const uint64_t k01 = pack2(bf16lo(kw.x), bf16hi(kw.x)), k23 = pack2(bf16lo(kw.y), bf16hi(kw.y));
            run01 = add2(run01, g01);
            run23 = add2(run23, g23);
            const uint64_t d01 = fma2(run01, l2e2, ref01), d23 = fma2(run23, l2e2, ref23);  // (G_t - G_m) log2(e)
            float d[4], dc[4];
            unpack2(d01, d[0], d[1]);
            unpack2(d23, d[2], d[3]);
            unpack2(add2(d01, comp2), dc[0], dc[1]);
            unpack2(add2(d23, comp2), dc[2], dc[3]);
            const uint64_t e1_01 = pack2(ex2f(dc[0]), ex2f(dc[1])), e1_23 = pack2(ex2f(dc[2]), ex2f(dc[3]));
            const uint64_t e2_01 = pack2(ex2f(-d[0]), ex2f(-d[1])), e2_23 = pack2(ex2f(-d[2]), ex2f(-d[3]));
            float kt[4], kh[4];
            unpack2(mul2(k01, e1_01), kt[0], kt[1]);
            unpack2(mul2(k23, e1_23), kt[2], kt[3]);
            unpack2(mul2(k01, e2_01), kh[0], kh[1]);
            unpack2(mul2(k23, e2_23), kh[2], kh[3]);
            if (WITH_O) {
              const uint2 qw = *reinterpret_cast<const uint2 *>(smem + off_q);
              const uint64_t q01 = pack2(bf16lo(qw.x), bf16hi(qw.x)), q23 = pack2(bf16lo(qw.y), bf16hi(qw.y));
              float qt[4];
              unpack2(mul2(q01, mul2(e1_01, qs2)), qt[0], qt[1]);
              unpack2(mul2(q23, mul2(e1_23, qs2)), qt[2], qt[3]);
              *reinterpret_cast<uint4 *>(smem + off_q) =
                  make_uint4(tf32_pre(qt[0]), tf32_pre(qt[1]), tf32_pre(qt[2]), tf32_pre(qt[3]));
            }
            *reinterpret_cast<uint4 *>(smem + off_k) =
                make_uint4(tf32_pre(kt[0]), tf32_pre(kt[1]), tf32_pre(kt[2]), tf32_pre(kt[3]));
            // Kh goes out twice, the same four values in both places: K-major (MMA1 contracts over the channels) and
            // MN-major (MMA5 contracts over the tokens).  A tf32 MN-major operand has a swizzle of its own, so the two
            // tiles differ in where a vector lands, not in what it holds.
            const uint4 khv = make_uint4(tf32_pre(kh[0]), tf32_pre(kh[1]), tf32_pre(kh[2]), tf32_pre(kh[3]));
            *reinterpret_cast<uint4 *>(smem + off_h) = khv;
            *reinterpret_cast<uint4 *>(kht_tile + mn32_offset(32, t, c0)) = khv;
          }
        }
        // the exponents of this chunk may have overflowed: the unit will not be written back.  (Every lane of a channel
        // quad holds the same totals; having only the first token group store keeps the producer loop free of spills.)
        if (out_of_range && tg == 0) misc->domain_flag = 1;
      } else {
        // ---- GDN: one scalar log-decay per token.  The first producer warp (lane = token) forms the running sums and
        // the per-token factors; nothing per channel needs an exponential, and k, q stay exactly their bf16 values:
        //   e1_t = exp(G_t - G_m), e2_t = exp(G_m - G_t) with m the end of the first half;
        //   MMA1 works on raw k, q (bf16 tile), MMA2 on raw k, q widened to tf32 containers, MMA5 on k_t e2_t;
        //   e1_t goes onto the rows of A, R and the outputs where they leave tensor memory, e2_j onto the columns of A, P.
        bool out_of_range = false;
        if (ptid < C) {
          const int slot = (ch & 3) * C + lane;
          float incl = gsc_cur;
#pragma unroll
          for (int dlt = 1; dlt < 32; dlt <<= 1) {
            const float x = __shfl_up_sync(0xffffffffu, incl, dlt);
            if (lane >= dlt) incl += x;
          }
          const float tot0 = __shfl_sync(0xffffffffu, incl, 15);          // G_m: the first half's total
          const float tot1 = __shfl_sync(0xffffffffu, incl, 31) - tot0;   // G_C - G_m
          const float d2 = (incl - tot0) * LOG2E;
          const float e1 = ex2f(d2), e2 = ex2f(-d2);
          e1c_s[slot] = e1 * kTruncComp;
          e2_s[slot] = e2;
          bte1_s[slot] = beta_s[slot] * e1;
          out_of_range = !(fabsf(tot0) <= kMaxHalfDecay) || !(fabsf(tot1) <= kMaxHalfDecay);   // also true for NaN
          // state factor from where the previous chunk left the state to this chunk's midpoint, and the factor owed after
          // it; scalars here, written for every channel so that the chain warps read them as they do for KDA
          const float f = ex2f((post_prev + tot0) * LOG2E);
          post_prev = tot1;
          *reinterpret_cast<float4 *>(fac_s + par * D + lane * 4) = make_float4(f, f, f, f);
          *reinterpret_cast<float4 *>(post_s + par * D + lane * 4) = make_float4(tot1, tot1, tot1, tot1);
        }
        mbar_arrive(&misc->rdy_fac[par]);
        asm volatile("bar.sync 2, 128;" ::: "memory");   // the factors are visible to all producer warps
        asm volatile("cp.async.wait_group 0;" ::: "memory");  // k and q have landed
#pragma unroll 1
        for (int half = 0; half < 2; ++half) {
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int t = half * 16 + tg * 4 + j;
            const uint32_t off_k = OFF_KQ + sw128_offset(64, t, c0), off_q = OFF_KQ + sw128_offset(64, 32 + t, c0);
            const uint2 kw = *reinterpret_cast<const uint2 *>(smem + off_k);
            const uint4 kf = make_uint4(kw.x << 16, kw.x & 0xFFFF0000u, kw.y << 16, kw.y & 0xFFFF0000u);  // exact
            *reinterpret_cast<uint4 *>(smem + off_k) = kf;
            *reinterpret_cast<uint2 *>(smem + OFF_KQ16 + sw128_offset_bf16(64, t, c0)) = kw;
            if (WITH_O) {
              const uint2 qw = *reinterpret_cast<const uint2 *>(smem + off_q);
              *reinterpret_cast<uint4 *>(smem + off_q) = make_uint4(qw.x << 16, qw.x & 0xFFFF0000u, qw.y << 16, qw.y & 0xFFFF0000u);
              *reinterpret_cast<uint2 *>(smem + OFF_KQ16 + sw128_offset_bf16(64, 32 + t, c0)) = qw;
            }
            const float e2 = e2_s[(ch & 3) * C + t];
            *reinterpret_cast<uint4 *>(kht_tile + mn32_offset(32, t, c0)) =
                make_uint4(tf32_pre(__uint_as_float(kf.x) * e2), tf32_pre(__uint_as_float(kf.y) * e2),
                           tf32_pre(__uint_as_float(kf.z) * e2), tf32_pre(__uint_as_float(kf.w) * e2));
          }
        }
        if (out_of_range && lane == 0) misc->domain_flag = 1;
      }
      fence_smem_to_async();
      mbar_arrive(&misc->rdy_prep);  // -> MMA1
    }
    // after a time-out the last log-decay copy may not have been waited for: it must have landed before the CTA leaves
    if (KDA && ptid == 0 && misc->abort_flag && g_issued > 0) mbar_wait_bounded(&misc->g_full, (g_issued - 1) & 1, kMaxPolls);
  } else {
    // ================================= chain warps =================================
    const int quad = warp & 3, colh = warp >> 2;                           // TMEM lane quadrant, column half
    const uint32_t tlane = tm + (static_cast<uint32_t>(quad * 32) << 16);  // this warp's TMEM lanes
    const int vrow = quad * 32 + lane;                                     // the TMEM lane this thread owns

    // V arrives by TMA, one box of 32 tokens x 128 values per chunk, started by one thread.  A box that reaches past
    // the request's last token brings in the following tokens of the stream (zeros past its end): those columns are
    // masked where V is used.
    const __nv_bfloat16 *gv = static_cast<const __nv_bfloat16 *>(a.v) + (tok0 * a.H_v + h) * D;
    auto stage_v = [&](int ch) {
      const int t0 = ch * C, ntok = min(C, n_tok - t0);
      for (int i = tid; i < C * 16; i += NCH) {
        const int t = i >> 4, j = i & 15;
        const bool valid = t < ntok;
        cp_async16_zfill(sbase + OFF_V + t * 256 + j * 16,
                         reinterpret_cast<const char *>(gv + (t0 + (valid ? t : 0)) * v_stride) + j * 16, valid);
      }
      asm volatile("cp.async.commit_group;" ::: "memory");
    };

    if (n_chunks > 0) {
      stage_v(0);
      // the start state goes into TMEM as it is; the first chunk's state pass scales it like any other
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
      const float *beta_c = beta_s + (ch & 3) * C;
      const float *fac_c = fac_s + par * D;

      // ---- (1) the previous chunk's state update is complete; this chunk's factors and tiles are ready ----
      if (ch > 0) wait_bar(&misc->bar_s, par ^ 1, misc, err);
      wait_bar(&misc->rdy_fac[par], (ch >> 1) & 1, misc, err);
      tc_fence_after_sync();

      // ---- (2) state pass: thread = (value column v, half of the channels); scale the state to this chunk's midpoint ----
      {
#pragma unroll 1
        for (int c0 = colh * 64; c0 < colh * 64 + 64; c0 += 32) {
          uint32_t s[32];
          tmem_ld32(tlane + COL_S + c0, s);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 32; j += 4) {
            const float4 f = *reinterpret_cast<const float4 *>(fac_c + c0 + j);
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

      // ---- (3) P out of TMEM, by warp 1 (lanes 32-63 are its quadrant); A and T are the triangular warp's ----
      if (WITH_O && warp == 1) {
        wait_bar(&misc->bar_ap, par, misc, err);
        tc_fence_after_sync();
        uint32_t x[32];
        tmem_ld32(tlane + COL_AP, x);
        tmem_ld_wait();
        const int t = lane;
        // row t of P = lower_incl_diag(Qt Kh^T), straight to its operand tile
        // (GDN: the raw q_t . k_j gets its column factor e2_j here; the row factor e1_t is applied to the outputs)
#pragma unroll
        for (int j = 0; j < 32; j += 4) {
          float4 e2 = make_float4(kInvTruncComp, kInvTruncComp, kInvTruncComp, kInvTruncComp);
          if constexpr (!KDA) {
            e2 = *reinterpret_cast<const float4 *>(e2_s + (ch & 3) * C + j);
            e2.x *= kInvTruncComp; e2.y *= kInvTruncComp; e2.z *= kInvTruncComp; e2.w *= kInvTruncComp;
          }
          uint4 o;
          o.x = (j + 0 <= t) ? tf32_pre(__uint_as_float(x[j + 0]) * e2.x) : 0u;
          o.y = (j + 1 <= t) ? tf32_pre(__uint_as_float(x[j + 1]) * e2.y) : 0u;
          o.z = (j + 2 <= t) ? tf32_pre(__uint_as_float(x[j + 2]) * e2.z) : 0u;
          o.w = (j + 3 <= t) ? tf32_pre(__uint_as_float(x[j + 3]) * e2.w) : 0u;
          *reinterpret_cast<uint4 *>(smem + OFF_PM + sw128_offset(32, t, j)) = o;
        }
        fence_smem_to_async();
      }

      // ---- (4) RHS^T = beta (V - R)^T as a tf32 pair: high over R^T, low in the consumed A|P columns ----
      wait_bar(&misc->bar_ro, par, misc, err);
      tc_fence_after_sync();
      asm volatile("cp.async.wait_all;" ::: "memory");  // V of this chunk
      wait_bar(&misc->a_taken, par, misc, err);         // the A|P columns are about to be overwritten
      sync_chain();
      {
        const int tb = colh * 16;
        uint32_t x[16], lo[16];
        tmem_ld16(tlane + COL_RO + tb, x);
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const float vv = __bfloat162float(Vs[(tb + j) * D + vrow]);
          // GDN: the product is k_t S' on the raw keys; its row factor e1_t (with the truncation compensation) comes here
          const float r = KDA ? __uint_as_float(x[j]) : e1c_s[(ch & 3) * C + tb + j] * __uint_as_float(x[j]);
          const float rhs = beta_c[tb + j] * (vv - r);
          x[j] = to_tf32(rhs);
          lo[j] = tf32_pre(rhs - __uint_as_float(x[j]));
        }
        tmem_st16(tlane + COL_RO + tb, x);
        tmem_st16(tlane + COL_AP + tb, lo);
        tmem_st_wait();
      }
      tc_fence_before_sync();
      mbar_arrive(&misc->rdy_rhs);  // -> MMA3 (T tile and RHS^T are ready)
      sync_chain();                 // everyone is done with V: the next chunk's V may land
      if (more) stage_v(ch + 1);

      // ---- (5) the part of U^T the tensor core drops when it reads it (the low 13 mantissa bits), written over
      //          the consumed RHS^T: U = U_hi + U_lo exactly ----
      wait_bar(&misc->bar_u, par, misc, err);
      tc_fence_after_sync();
      {
        const int tb = colh * 16;
        uint32_t x[16];
        tmem_ld16(tlane + COL_U + tb, x);
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 16; ++j)
          x[j] = tf32_pre(__uint_as_float(x[j]) - __uint_as_float(x[j] & 0xFFFFE000u));
        tmem_st16(tlane + COL_RO + tb, x);
        tmem_st_wait();
      }
      tc_fence_before_sync();
      mbar_arrive(&misc->rdy_u);  // -> MMA4, MMA5

      // ---- (6) outputs of this chunk ----
      wait_bar(&misc->bar_o, par, misc, err);
      tc_fence_after_sync();
      if (WITH_O) {
        const int tb = colh * 16;
        uint32_t x[16];
        tmem_ld16(tlane + COL_RO + 32 + tb, x);
        tmem_ld_wait();
        if constexpr (!KDA) {
          // GDN: the accumulated q_t (S' + sum_j e2_j k_j u_j^T) still lacks its row factor e1_t, the query scale and
          // the truncation compensation
#pragma unroll
          for (int j = 0; j < 16; ++j)
            x[j] = __float_as_uint(__uint_as_float(x[j]) * (e1c_s[(ch & 3) * C + tb + j] * a.q_scale));
        }
        if constexpr (sizeof(OT) == 2) {
          // through shared memory (the T and P tiles are free now) so that global stores are 16 bytes wide
          __nv_bfloat16 *Os = reinterpret_cast<__nv_bfloat16 *>(smem + OFF_TM);
#pragma unroll
          for (int j = 0; j < 16; ++j) Os[(tb + j) * D + vrow] = __float2bfloat16_rn(__uint_as_float(x[j]));
          sync_chain();
          for (int i = tid; i < ntok * 16; i += NCH) {
            const int t = i >> 4, j = i & 15;
            *reinterpret_cast<uint4 *>(reinterpret_cast<char *>(go + (t0 + t) * v_stride) + j * 16) =
                *reinterpret_cast<const uint4 *>(smem + OFF_TM + t * 256 + j * 16);
          }
        } else {
#pragma unroll
          for (int j = 0; j < 16; ++j)
            if (tb + j < ntok) go[(t0 + tb + j) * v_stride + vrow] = __uint_as_float(x[j]);
        }
      }
      tc_fence_before_sync();
      mbar_arrive(&misc->tp_free);  // this thread is done with the T|P|O tile region
      sync_chain();  // every chain thread is done with this chunk's P and O tiles before they are rewritten
    }

    // ---- final state: the factor still owed, then write back ----
    if (n_chunks > 0) {
      wait_bar(&misc->rdy_prep, (n_chunks - 1) & 1, misc, err);  // the last chunk's post_s
      wait_bar(&misc->bar_s, (n_chunks - 1) & 1, misc, err);
    }
    // fac_s is free: the producer has finished (its last arrival was waited for above)
    if (tid < D) fac_s[tid] = n_chunks > 0 ? ex2f(post_s[((n_chunks - 1) & 1) * D + tid] * LOG2E) : 1.f;
    sync_chain();
    tc_fence_after_sync();
    // A unit whose decay left the range, or whose CTA gave up on a wait, is NOT written back: its stored state keeps
    // the bits it had before the call, so that it can be replayed by the exact kernel (or by the caller).
    const bool bad = misc->abort_flag != 0 || misc->domain_flag != 0;
    if (bad) {
      if (tid == 0 && misc->abort_flag == 0) hand_over(a, true);
    } else {
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
  }
  tc_fence_before_sync();
  __syncthreads();
  if (warp == WARP_MMA) tmem_dealloc(tm, TMEM_COLS);
}

// cuTensorMapEncodeTiled is a driver entry point.  It is looked up through the runtime at first use, so that the library
// has no link-time dependency on libcuda and still loads (plan building, accessors) on a machine without a driver.
using EncodeTiledFn = CUresult (*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                   const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = [] {
    void *p = nullptr;
    cudaDriverEntryPointQueryResult q = cudaDriverEntryPointSymbolNotFound;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      p = nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

template <bool KDA, typename OT, bool WITH_O>
int launch(const DascRefreshArgs &a, void *stream) {
  auto kern = refresh_chunked_kernel<KDA, OT, WITH_O>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(SMEM_ALLOC));
  if (e != cudaSuccess) return static_cast<int>(e);
  const int64_t n_units = static_cast<int64_t>(a.n_req) * a.n_layers_in_call * a.H_v;
  if (n_units == 0) return cudaSuccess;
  if (n_units > 2147483647LL) return static_cast<int>(cudaErrorInvalidConfiguration);
  e = cudaMemsetAsync(a.workspace, 0, 16, static_cast<cudaStream_t>(stream));  // clear the four header words
  if (e != cudaSuccess) return static_cast<int>(e);
  // tensor map of the KDA log-decay [Lc*T tokens][H_v][128] fp32: boxes of 32 tokens x one head x 32 channels with the
  // 128-byte swizzle, which is the layout of one block of the Kh operand tile (GDN has one scalar per token: no map)
  CUtensorMap tmap_g{};
  if (KDA) {
    const cuuint64_t dims[3] = {static_cast<cuuint64_t>(D), static_cast<cuuint64_t>(a.H_v),
                                static_cast<cuuint64_t>(a.n_layers_in_call) * static_cast<cuuint64_t>(a.total_tokens)};
    const cuuint64_t strides[2] = {static_cast<cuuint64_t>(D) * 4, static_cast<cuuint64_t>(a.H_v) * D * 4};
    const cuuint32_t box[3] = {32, 1, static_cast<cuuint32_t>(C)};
    const cuuint32_t ones[3] = {1, 1, 1};
    const EncodeTiledFn encode = encode_tiled_fn();
    if (!encode) return static_cast<int>(cudaErrorNotSupported);
    if (encode(&tmap_g, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<float *>(a.g), dims, strides, box, ones,
                               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return static_cast<int>(cudaErrorInvalidValue);
  }
  kern<<<static_cast<unsigned>(n_units), NT, SMEM_ALLOC, static_cast<cudaStream_t>(stream)>>>(a, tmap_g);
  return static_cast<int>(cudaGetLastError());
}

}  // namespace

// Scratch the chunked kernel needs: the 256-byte header (flags and counters) and one list entry per unit of the call.
size_t dasc_refresh_chunked_workspace_bytes(int32_t n_req, int32_t n_layers_in_call, int32_t H_v) {
  const size_t units = static_cast<size_t>(n_req) * static_cast<size_t>(n_layers_in_call) * static_cast<size_t>(H_v);
  return kRefreshWsHeader + (units * sizeof(int32_t) + 255) / 256 * 256;
}

uint32_t g_dasc_debug_poll_limit = 0;

// Returns a cudaError_t as int, or -1 if this kernel does not take the request
// (it needs d_k = d_v = 128 and bf16 token streams).
int dasc_launch_refresh_chunked(const DascRefreshArgs &a_in, void *stream) {
  if (a_in.d_k != D || a_in.d_v != D || !a_in.io_bf16) return -1;
  DascRefreshArgs a = a_in;
  a.poll_limit_first_wait = __atomic_load_n(&g_dasc_debug_poll_limit, __ATOMIC_RELAXED);
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

// Device address of the static scratch on device `dev`, which must be the CURRENT device; resolves it on the
// first call.
cudaError_t static_scratch_address(int dev, void **out) {
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  void *p = __atomic_load_n(&g_static_scratch_addr[dev], __ATOMIC_ACQUIRE);
  if (!p) {
    const cudaError_t e = cudaGetSymbolAddress(&p, g_refresh_static_scratch);
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
  // The plan's tables, the caller's buffers and the scratch all have to be on the device the kernel runs on.
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return DASC_ERR_CUDA;
  if (dev != plan->info.device) return DASC_ERR_INVALID_ARG;
  // The scratch this kernel cannot do without (the header words) must fit the static array; the list of units left
  // unwritten is as long as the rest of the array allows (a longer list is cut, the error word is set all the same).
  const size_t need = kRefreshWsHeader;
  if (need > kStaticScratchBytes) return DASC_ERR_WORKSPACE;
  void *scratch = nullptr;
  if (static_scratch_address(dev, &scratch) != cudaSuccess) return DASC_ERR_CUDA;
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
  a.workspace = scratch;  // the launcher clears the header words on the stream
  a.workspace_bytes = kStaticScratchBytes;
  // units outside the chunked kernel's log-decay range are listed behind the header, left unwritten, and replayed by
  // the exact kernel right after (it needs no scratch of its own); units that do not fit the list are an error
  a.unit_list = reinterpret_cast<int32_t *>(static_cast<unsigned char *>(scratch) + kRefreshWsHeader);
  a.unit_list_cap = static_cast<int32_t>((kStaticScratchBytes - kRefreshWsHeader) / sizeof(int32_t));
  a.short_thr = -1;
  a.domain_is_error = 0;
  int e = dasc_launch_refresh_chunked(a, cuda_stream);
  if (e == -1) return DASC_ERR_SHAPE;
  if (e == 0) {
    a.from_list = 1;
    e = dasc_launch_refresh_seq(a, cuda_stream);
  }
  return e == 0 ? DASC_OK : DASC_ERR_CUDA;
}
