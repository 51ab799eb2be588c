// INT8 checkpoint codec fused into the Store / Load copies (Appendix D, Eq. 10).
// pack_int8: gather the retained rows, take one abs-max per row (a (layer, head, key channel)
// tuple, shared over d_v), s = max(a, 1e-8)/127, q = clip(round(S/s), -127, 127) in fp32 with
// round-to-nearest-even, and write codes and scales into the request's slot.
// restore_int8: scatter back with S_hat = q * s, omitted rows zero-filled, every dense byte
// written once.  Both are HBM-bandwidth work like their fp32 counterparts: 128-bit loads of the
// fp32 side, 32-bit accesses of the code side (a warp still moves whole 128-byte lines).
//
// Slot layout (bytes): [packed_rows][d_v] int8 codes, then [packed_rows] fp32 scales; rows in
// the plan's ragged order (layers ascending, rows ascending).
#include <cuda_runtime.h>

#include "dasc_internal.h"

namespace {

#ifndef DASC_INT8_THREADS
#define DASC_INT8_THREADS 128
#endif
#ifndef DASC_INT8_PACK_UNROLL
#define DASC_INT8_PACK_UNROLL 4
#endif
#ifndef DASC_INT8_RESTORE_UNROLL
#define DASC_INT8_RESTORE_UNROLL 4
#endif
#ifndef DASC_INT8_PACK_MIN_BLOCKS
#define DASC_INT8_PACK_MIN_BLOCKS 12   /* caps registers at 40: occupancy is what hides the latency */
#endif
#ifndef DASC_INT8_RESTORE_MIN_BLOCKS
#define DASC_INT8_RESTORE_MIN_BLOCKS 16   /* caps registers at 32 */
#endif
constexpr int kThreads = DASC_INT8_THREADS;          // tuning knobs; defaults = best of a measured sweep
constexpr int kUnroll = DASC_INT8_PACK_UNROLL;       // rows (pack) / vectors (restore) in flight per thread
constexpr int kRUnroll = DASC_INT8_RESTORE_UNROLL;

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
__device__ __forceinline__ uint32_t ld_stream32(const uint32_t *p) {
  uint32_t v;
  asm volatile("ld.global.nc.L1::no_allocate.u32 %0, [%1];" : "=r"(v) : "l"(p));
  return v;
}
__device__ __forceinline__ void st_stream32(uint32_t *p, uint32_t v) {
  asm volatile("st.global.L1::no_allocate.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// One code of Eq. 10 by the formula as written: IEEE division, round to nearest even, clip to [-127, 127].
__device__ __forceinline__ uint32_t code_exact(uint32_t bits, float s) {
  float y = rintf(__fdiv_rn(__uint_as_float(bits), s));
  y = fminf(fmaxf(y, -127.0f), 127.0f);
  return static_cast<uint32_t>(static_cast<int32_t>(y)) & 0xFFu;
}

// Adding 1.5 * 2^23 to |t| < 2^22 rounds t to the nearest integer (ties to even) and leaves that
// integer, in two's complement, in the low mantissa bits.
constexpr float kRoundMagic = 12582912.0f;
// A product x * (1/s) with an approximate reciprocal is within 2^-14 of the exact quotient x / s
// for |x / s| <= 128, so it rounds to the same integer unless it lies this close to a half-integer;
// only then is the exact division taken.
constexpr float kSafeFraction = 0.5f - 1.0f / 8192.0f;

// The four codes of one 16-byte vector, bit-identical to code_exact on finite inputs.
// `a` is the row's abs-max.  (The clip of Eq. 10 never acts on finite inputs: |x| <= a gives
// |x / s| < 127.5.)
__device__ __forceinline__ uint32_t codes_of(const uint4 &v, float a) {
  float inv;  // the argument lies in [7.8e-11, 2.7e36], so the reciprocal is a normal number
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(inv) : "f"(__fmul_rn(fmaxf(a, 1e-8f), 1.0f / 127.0f)));
  // two values per instruction (packed fp32 pairs): m = x*inv + magic (one rounding: the nearest
  // integer of the product), r = m - magic, d = x*inv - r = signed distance of the product to it
  uint32_t m[4];
  float d[4];
  asm("{\n\t.reg .b64 xa, xb, iv, mg, ma, mb, ra, rb;\n\t"
      "mov.b64 xa, {%8, %9};\n\t"
      "mov.b64 xb, {%10, %11};\n\t"
      "mov.b64 iv, {%12, %12};\n\t"
      "mov.b64 mg, {%13, %13};\n\t"
      "fma.rn.f32x2 ma, xa, iv, mg;\n\t"
      "fma.rn.f32x2 mb, xb, iv, mg;\n\t"
      "sub.rn.f32x2 ra, mg, ma;\n\t"  // -(r)
      "sub.rn.f32x2 rb, mg, mb;\n\t"
      "fma.rn.f32x2 ra, xa, iv, ra;\n\t"
      "fma.rn.f32x2 rb, xb, iv, rb;\n\t"
      "mov.b64 {%0, %1}, ma;\n\t"
      "mov.b64 {%2, %3}, mb;\n\t"
      "mov.b64 {%4, %5}, ra;\n\t"
      "mov.b64 {%6, %7}, rb;\n\t}"
      : "=r"(m[0]), "=r"(m[1]), "=r"(m[2]), "=r"(m[3]), "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
      : "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w), "f"(inv), "f"(kRoundMagic));
  const float worst = fmaxf(fmaxf(fabsf(d[0]), fabsf(d[1])), fmaxf(fabsf(d[2]), fabsf(d[3])));
  uint32_t word = __byte_perm(__byte_perm(m[0], m[1], 0x0040), __byte_perm(m[2], m[3], 0x0040), 0x5410);
  if (!(worst < kSafeFraction)) {  // rare
    const float s = __fdiv_rn(fmaxf(a, 1e-8f), 127.0f);
    word = code_exact(v.x, s) | (code_exact(v.y, s) << 8) | (code_exact(v.z, s) << 16) | (code_exact(v.w, s) << 24);
  }
  return word;
}

__device__ __forceinline__ float absmax4(const uint4 &v) {
  return fmaxf(fmaxf(fabsf(__uint_as_float(v.x)), fabsf(__uint_as_float(v.y))),
               fmaxf(fabsf(__uint_as_float(v.z)), fabsf(__uint_as_float(v.w))));
}

// grid = (ceil(packed_vecs / (kThreads*kUnroll)), pairs).  A "vec" is 4 consecutive values of a row;
// a row is held by `lanes_per_row` = d_v/4 consecutive lanes of one warp (a power of two <= 32).
// FULL_WARP_ROWS: d_v = 128, a row is exactly one warp and the abs-max is one warp reduction.
template <bool FULL_WARP_ROWS>
__global__ void __launch_bounds__(kThreads, DASC_INT8_PACK_MIN_BLOCKS) pack_int8_kernel(const uint4 *__restrict__ state, int64_t layer_stride4,
                                                             int64_t req_stride4, const int32_t *__restrict__ src_req,
                                                             uint8_t *__restrict__ pool, int64_t slot_stride_bytes,
                                                             const int32_t *__restrict__ dst_slot,
                                                             const DascRowSrc *__restrict__ row_src,
                                                             uint32_t packed_vecs, uint32_t packed_rows,
                                                             uint32_t lanes_per_row_arg, int32_t n_pairs) {
  const uint32_t lanes_per_row = FULL_WARP_ROWS ? 32u : lanes_per_row_arg;
  const uint32_t base = blockIdx.x * (kThreads * kUnroll) + threadIdx.x;
  for (int32_t pair = blockIdx.y; pair < n_pairs; pair += gridDim.y) {
    const uint4 *src_base = state + static_cast<int64_t>(__ldg(src_req + pair)) * req_stride4;
    uint8_t *slot = pool + static_cast<int64_t>(__ldg(dst_slot + pair)) * slot_stride_bytes;
    uint32_t *codes = reinterpret_cast<uint32_t *>(slot);
    float *scales = reinterpret_cast<float *>(slot + static_cast<size_t>(packed_rows) * lanes_per_row * 4u);
    uint4 val[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const uint32_t i = base + u * kThreads;
      val[u] = make_uint4(0u, 0u, 0u, 0u);
      if (i < packed_vecs) {
        const uint32_t row = i / lanes_per_row;
        const uint32_t vec = i - row * lanes_per_row;
        const int2 s = __ldg(reinterpret_cast<const int2 *>(row_src) + row);  // {layer, dense row}
        val[u] = ld_stream(src_base + s.x * layer_stride4 + static_cast<int64_t>(s.y) * lanes_per_row + vec);
      }
    }
    // abs-max of each row: rows never straddle a warp, and the lanes of a row are all inside or all
    // outside the valid range, so every lane of the warp takes part in the reductions
    float amax[kUnroll];
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      float a = absmax4(val[u]);
      if constexpr (FULL_WARP_ROWS) {
        asm volatile("redux.sync.max.abs.f32 %0, %1, 0xffffffff;" : "=f"(a) : "f"(a));
      } else {
        for (uint32_t off = lanes_per_row >> 1; off > 0; off >>= 1) a = fmaxf(a, __shfl_xor_sync(0xFFFFFFFFu, a, off));
      }
      amax[u] = a;
    }
#pragma unroll
    for (int u = 0; u < kUnroll; ++u) {
      const uint32_t i = base + u * kThreads;
      const uint32_t word = codes_of(val[u], amax[u]);
      if (i < packed_vecs) st_stream32(codes + i, word);
    }
    // scales, s = max(a, 1e-8) / 127 by IEEE division
    if constexpr (FULL_WARP_ROWS) {
      // the warp's kUnroll rows are spread over its first lanes, one division each
      const uint32_t lane = threadIdx.x & 31u;
      if (lane < kUnroll) {
        float a = amax[0];
#pragma unroll
        for (int u = 1; u < kUnroll; ++u) a = lane == u ? amax[u] : a;
        const uint32_t i = base - lane + lane * kThreads;  // first vector of that row
        if (i < packed_vecs) scales[i >> 5] = __fdiv_rn(fmaxf(a, 1e-8f), 127.0f);
      }
    } else {
#pragma unroll
      for (int u = 0; u < kUnroll; ++u) {
        const uint32_t i = base + u * kThreads;
        const uint32_t row = i / lanes_per_row;
        if (i < packed_vecs && i == row * lanes_per_row) scales[row] = __fdiv_rn(fmaxf(amax[u], 1e-8f), 127.0f);
      }
    }
  }
}

// S_hat = q * s for the four codes of one word.  q is rebuilt without an integer-to-float
// conversion: byte b = q + 128 placed in the low mantissa bits of 2^23 gives 2^23 + b exactly, and
// subtracting 2^23 + 128 leaves q; then one fp32 multiply, two values per instruction.
__device__ __forceinline__ uint4 dequant4(uint32_t word, float s) {
  const uint32_t w = word ^ 0x80808080u;
  uint4 out;
  asm("{\n\t.reg .b64 fa, fb, of, sc;\n\t"
      "mov.b64 fa, {%4, %5};\n\t"
      "mov.b64 fb, {%6, %7};\n\t"
      "mov.b64 of, {%8, %8};\n\t"
      "mov.b64 sc, {%9, %9};\n\t"
      "sub.rn.f32x2 fa, fa, of;\n\t"
      "sub.rn.f32x2 fb, fb, of;\n\t"
      "mul.rn.f32x2 fa, fa, sc;\n\t"
      "mul.rn.f32x2 fb, fb, sc;\n\t"
      "mov.b64 {%0, %1}, fa;\n\t"
      "mov.b64 {%2, %3}, fb;\n\t}"
      : "=r"(out.x), "=r"(out.y), "=r"(out.z), "=r"(out.w)
      : "r"(__byte_perm(w, 0x4B000000u, 0x7540)), "r"(__byte_perm(w, 0x4B000000u, 0x7541)),
        "r"(__byte_perm(w, 0x4B000000u, 0x7542)), "r"(__byte_perm(w, 0x4B000000u, 0x7543)), "f"(8388736.0f), "f"(s));
  return out;
}

// grid = (ceil(layer_vecs / (kThreads*kRUnroll)), n_layers, pairs).
template <bool FULL_WARP_ROWS>
__global__ void __launch_bounds__(kThreads, DASC_INT8_RESTORE_MIN_BLOCKS) restore_int8_kernel(const uint8_t *__restrict__ pool,
                                                                int64_t slot_stride_bytes,
                                                                const int32_t *__restrict__ src_slot,
                                                                uint4 *__restrict__ state, int64_t layer_stride4,
                                                                int64_t req_stride4, const int32_t *__restrict__ dst_req,
                                                                const int32_t *__restrict__ row_pos, uint32_t layer_vecs,
                                                                uint32_t rows_per_layer, uint32_t packed_rows,
                                                                uint32_t lanes_per_row_arg, int32_t n_pairs) {
  const uint32_t lanes_per_row = FULL_WARP_ROWS ? 32u : lanes_per_row_arg;
  const uint32_t base = blockIdx.x * (kThreads * kRUnroll) + threadIdx.x;
  const int32_t layer = blockIdx.y;
  const int32_t *pos_l = row_pos + static_cast<int64_t>(layer) * rows_per_layer;
  for (int32_t pair = blockIdx.z; pair < n_pairs; pair += gridDim.z) {
    const uint8_t *slot = pool + static_cast<int64_t>(__ldg(src_slot + pair)) * slot_stride_bytes;
    const uint32_t *codes = reinterpret_cast<const uint32_t *>(slot);
    const float *scales = reinterpret_cast<const float *>(slot + static_cast<size_t>(packed_rows) * lanes_per_row * 4u);
    uint4 *dst_base = state + static_cast<int64_t>(__ldg(dst_req + pair)) * req_stride4 + layer * layer_stride4;
    uint32_t word[kRUnroll];
    float scale[kRUnroll];  // 0 marks an omitted row: a stored scale is at least 1e-8/127
#pragma unroll
    for (int u = 0; u < kRUnroll; ++u) {
      const uint32_t i = base + u * kThreads;
      word[u] = 0u;
      scale[u] = 0.0f;
      if (i < layer_vecs) {
        const uint32_t row = i / lanes_per_row;
        const uint32_t vec = i - row * lanes_per_row;
        const int32_t pos = __ldg(pos_l + row);
        if (pos >= 0) {
          word[u] = ld_stream32(codes + static_cast<uint32_t>(pos) * lanes_per_row + vec);
          scale[u] = __ldg(scales + pos);
        }
      }
    }
#pragma unroll
    for (int u = 0; u < kRUnroll; ++u) {
      const uint32_t i = base + u * kThreads;
      // an omitted row has all codes 0 and scale 0: 0 * 0 = +0.0f, the zero fill
      if (i < layer_vecs) st_stream(dst_base + i, dequant4(word[u], scale[u]));
    }
  }
}

}  // namespace

int dasc_launch_pack_int8(const dasc_plan_s *plan, const float *state, int64_t layer_stride, int64_t req_stride,
                          const int32_t *src_req, void *pool, int64_t slot_stride_bytes, const int32_t *dst_slot,
                          int32_t n_pairs, void *stream) {
  const uint32_t lpr = static_cast<uint32_t>(plan->info.d_v / 4);
  const uint64_t packed_vecs = static_cast<uint64_t>(plan->packed_rows) * lpr;
  if (packed_vecs == 0 || n_pairs == 0) return cudaSuccess;
  const uint32_t per_block = kThreads * kUnroll;
  dim3 grid(static_cast<uint32_t>((packed_vecs + per_block - 1) / per_block),
            static_cast<uint32_t>(n_pairs < 65535 ? n_pairs : 65535));
  auto kernel = lpr == 32 ? pack_int8_kernel<true> : pack_int8_kernel<false>;
  kernel<<<grid, kThreads, 0, static_cast<cudaStream_t>(stream)>>>(
      reinterpret_cast<const uint4 *>(state), layer_stride / 4, req_stride / 4, src_req,
      static_cast<uint8_t *>(pool), slot_stride_bytes, dst_slot, plan->d_row_src, static_cast<uint32_t>(packed_vecs),
      static_cast<uint32_t>(plan->packed_rows), lpr, n_pairs);
  return static_cast<int>(cudaGetLastError());
}

int dasc_launch_restore_int8(const dasc_plan_s *plan, const void *pool, int64_t slot_stride_bytes,
                             const int32_t *src_slot, float *state, int64_t layer_stride, int64_t req_stride,
                             const int32_t *dst_req, int32_t n_pairs, void *stream) {
  const uint32_t lpr = static_cast<uint32_t>(plan->info.d_v / 4);
  const uint64_t layer_vecs = static_cast<uint64_t>(plan->rows_per_layer) * lpr;
  if (n_pairs == 0) return cudaSuccess;
  const uint32_t per_block = kThreads * kRUnroll;
  dim3 grid(static_cast<uint32_t>((layer_vecs + per_block - 1) / per_block),
            static_cast<uint32_t>(plan->info.n_layers), static_cast<uint32_t>(n_pairs < 65535 ? n_pairs : 65535));
  auto kernel = lpr == 32 ? restore_int8_kernel<true> : restore_int8_kernel<false>;
  kernel<<<grid, kThreads, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const uint8_t *>(pool), slot_stride_bytes, src_slot, reinterpret_cast<uint4 *>(state),
      layer_stride / 4, req_stride / 4, dst_req, plan->d_row_pos, static_cast<uint32_t>(layer_vecs),
      static_cast<uint32_t>(plan->rows_per_layer), static_cast<uint32_t>(plan->packed_rows), lpr, n_pairs);
  return static_cast<int>(cudaGetLastError());
}
