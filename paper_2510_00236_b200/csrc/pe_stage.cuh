// Operand staging for the two-pass per-token second moment (Section 2.3):
//     S'[o,i] = sum_r dY[r,o]^2 * X[r,i]^2.
// The squares need 11 significant bits (bf16's 8 are not enough: all terms are non-negative, so
// rounding errors do not cancel).  IEEE half has 11 and runs on the tensor cores at the full 16-bit
// rate, but only spans 2^-24 .. 2^16, so every feature column gets a power-of-two scale of its own:
//   1. column_max_kernel   finds the largest magnitude of every column of X and of dY,
//   2. square_to_half_kernel  writes half(x^2 * 2^(13 - 2e)) for a column whose maximum lies in
//      [2^e, 2^(e+1)): the scaled squares stay below 2^15; entries more than 2^14 below their column's
//      maximum lose bits gradually and vanish 2^20 below it, where their squares are 2^-40 of the
//      column's largest term,
//   3. the plain tensor-core contraction runs on the half operands (fp32 accumulation),
//   4. unscale_kernel multiplies out[o,i] by the inverse scales of dY column o and X column i.
// Multiplying by a power of two is exact, so the only rounding is the one to half: at most 2^-11
// relative per operand, to nearest even, hence unbiased.
// All three kernels are streaming kernels bound by HBM bandwidth.
//
// The same route with fp8 (e4m3) operands, which the tensor cores contract at twice the 16-bit rate from
// half the staged bytes: the squares are written as e4m3(x^2 * 2^(6 - 2e)) (below 2^8, e4m3's largest
// finite value being 448).  e4m3 keeps 4 significant bits, so each staged square carries up to 2^-4
// relative rounding error (to nearest even, unbiased) and each term of the sum up to about 2^-3; the
// errors of different rows are independent and the terms non-negative, so the error of an entry falls
// with the square root of the number of rows that carry its sum (see the error model in the host code).
#pragma once
#include <cuda_fp16.h>
#include <cuda_fp8.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace pe {

constexpr int STAGE_THREADS = 256;          // 32 column chunks (of 8 features) x 8 rows per block and step
constexpr int STAGE_EXP_MIN = 71, STAGE_EXP_MAX = 196;   // clamp of the biased exponent: both scales stay normal floats

// Biased exponent of a column's largest magnitude, from the bf16 bit pattern of that magnitude.
__device__ __forceinline__ int stage_exponent(uint32_t max_abs_bits) {
  const int E = (int)(max_abs_bits & 0x7FFFu) >> 7;
  return E < STAGE_EXP_MIN ? STAGE_EXP_MIN : (E > STAGE_EXP_MAX ? STAGE_EXP_MAX : E);
}
// 2^(TOP - 2 (E - 127)) and its inverse; TOP = 13 for half (scaled squares below 2^15), 6 for e4m3 (below 2^8).
// Both stay normal floats for every clamped exponent (E <= 193 would suffice for TOP = 6: the clamp's upper
// end is lowered by 3 there).
template <bool FP8>
__device__ __forceinline__ int stage_exponent_for(uint32_t max_abs_bits) {
  const int E = stage_exponent(max_abs_bits);
  return (FP8 && E > STAGE_EXP_MAX - 3) ? STAGE_EXP_MAX - 3 : E;
}
template <bool FP8>
__device__ __forceinline__ float stage_scale(int E) { return __uint_as_float((uint32_t)((FP8 ? 387 : 394) - 2 * E) << 23); }
template <bool FP8>
__device__ __forceinline__ float stage_inv_scale(int E) { return __uint_as_float((uint32_t)(2 * E - (FP8 ? 133 : 140)) << 23); }

// max_bits[c] = max over rows of |src[r, c]| as a bf16 bit pattern (which orders like the magnitude).
// src: [rows, d] bf16, d a multiple of 8; max_bits: [d], zero on entry.  gridDim.x covers the columns
// in groups of 256, gridDim.y slices the rows, gridDim.z = 2 picks the tensor (0: X, 1: dY), so one
// launch serves both.
struct StageTensor {
  const uint16_t* src;     // [rows, d] bf16 bit patterns
  void* dst;               // [rows, d] scaled squares, IEEE half or e4m3 (square_to_lp_kernel only)
  uint32_t* max_bits;      // [d]
  int d;
};
__global__ void __launch_bounds__(STAGE_THREADS)
column_max_kernel(StageTensor tx_, StageTensor ty_, long long rows) {
  const StageTensor& tn = blockIdx.z == 0 ? tx_ : ty_;
  const uint16_t* __restrict__ src = tn.src;
  uint32_t* __restrict__ max_bits = tn.max_bits;
  const int d = tn.d;
  if (blockIdx.x * 256 >= d) return;          // the grid is sized for the wider tensor
  __shared__ uint32_t part[8][32][4];
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const int col = (blockIdx.x * 32 + tx) * 8;
  const long long r_begin = rows * blockIdx.y / gridDim.y, r_end = rows * (blockIdx.y + 1) / gridDim.y;
  uint32_t m[4] = {0u, 0u, 0u, 0u};
  if (col < d) {
    for (long long r = r_begin + ty; r < r_end; r += 8) {
      const uint4 v = __ldg(reinterpret_cast<const uint4*>(src + r * d + col));
      m[0] = __vmaxu2(m[0], v.x & 0x7FFF7FFFu);
      m[1] = __vmaxu2(m[1], v.y & 0x7FFF7FFFu);
      m[2] = __vmaxu2(m[2], v.z & 0x7FFF7FFFu);
      m[3] = __vmaxu2(m[3], v.w & 0x7FFF7FFFu);
    }
  }
#pragma unroll
  for (int k = 0; k < 4; ++k) part[ty][tx][k] = m[k];
  __syncthreads();
  // thread t of the block finishes column t of the block's 256
  const int c = threadIdx.x;
  if (blockIdx.x * 256 + c < d) {
    uint32_t best = 0u;
#pragma unroll
    for (int y = 0; y < 8; ++y) {
      const uint32_t w = part[y][c >> 3][(c & 7) >> 1];
      const uint32_t h = (c & 1) ? (w >> 16) : (w & 0xFFFFu);
      best = h > best ? h : best;
    }
    if (best) atomicMax(max_bits + blockIdx.x * 256 + c, best);
  }
}

// dst[r, c] = half(src[r, c]^2 * scale(c)), or the same as e4m3 (FP8).  Same grid and thread layout as
// column_max_kernel, so a thread's eight columns, and with them its scales, never change.
template <bool FP8>
__global__ void __launch_bounds__(STAGE_THREADS)
square_to_lp_kernel(StageTensor tx_, StageTensor ty_, long long rows) {
  const StageTensor& tn = blockIdx.z == 0 ? tx_ : ty_;
  const uint16_t* __restrict__ src = tn.src;
  const uint32_t* __restrict__ max_bits = tn.max_bits;
  const int d = tn.d;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const int col = (blockIdx.x * 32 + tx) * 8;
  if (col >= d) return;
  const long long r_begin = rows * blockIdx.y / gridDim.y, r_end = rows * (blockIdx.y + 1) / gridDim.y;
  float sc[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) sc[j] = stage_scale<FP8>(stage_exponent_for<FP8>(max_bits[col + j]));
  for (long long r = r_begin + ty; r < r_end; r += 8) {
    const uint4 v = __ldcs(reinterpret_cast<const uint4*>(src + r * d + col));
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    uint32_t o[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const float a = __uint_as_float(w[k] << 16), b = __uint_as_float(w[k] & 0xFFFF0000u);
      if constexpr (FP8) {
        o[k] = (uint32_t)__nv_cvt_float2_to_fp8x2(make_float2(a * a * sc[2 * k], b * b * sc[2 * k + 1]), __NV_SATFINITE, __NV_E4M3);
      } else {
        const __half2 h = __floats2half2_rn(a * a * sc[2 * k], b * b * sc[2 * k + 1]);
        o[k] = *reinterpret_cast<const uint32_t*>(&h);
      }
    }
    if constexpr (FP8) {
      *reinterpret_cast<uint2*>(static_cast<uint8_t*>(tn.dst) + r * d + col) = make_uint2(o[0] | (o[1] << 16), o[2] | (o[3] << 16));
    } else {
      *reinterpret_cast<uint4*>(static_cast<__half*>(tn.dst) + r * d + col) = make_uint4(o[0], o[1], o[2], o[3]);
    }
  }
}

// out[o, i] *= inv_scale(dY column o) * inv_scale(X column i); out: [d_out, d_in] fp32, d_in % 4 == 0.
template <bool FP8>
__global__ void __launch_bounds__(STAGE_THREADS)
unscale_kernel(float* __restrict__ out, int d_out, int d_in, const uint32_t* __restrict__ max_x,
               const uint32_t* __restrict__ max_dy) {
  const long long n4 = (long long)d_out * d_in / 4;
  const long long stride = (long long)gridDim.x * blockDim.x;
  const int q_per_row = d_in / 4;
  for (long long k = (long long)blockIdx.x * blockDim.x + threadIdx.x; k < n4; k += stride) {
    const int o = (int)(k / q_per_row), i = (int)(k - (long long)o * q_per_row) * 4;
    const float ro = stage_inv_scale<FP8>(stage_exponent_for<FP8>(max_dy[o]));
    float4 v = reinterpret_cast<float4*>(out)[k];
    v.x = v.x * stage_inv_scale<FP8>(stage_exponent_for<FP8>(max_x[i])) * ro;
    v.y = v.y * stage_inv_scale<FP8>(stage_exponent_for<FP8>(max_x[i + 1])) * ro;
    v.z = v.z * stage_inv_scale<FP8>(stage_exponent_for<FP8>(max_x[i + 2])) * ro;
    v.w = v.w * stage_inv_scale<FP8>(stage_exponent_for<FP8>(max_x[i + 3])) * ro;
    reinterpret_cast<float4*>(out)[k] = v;
  }
}

// Packed (ragged) batches, Section 2.3: example b owns token rows offsets[b] .. offsets[b+1]-1.  The tensor-core
// kernel contracts 16 tokens per instruction, so a sequence's last len % 16 tokens are copied here, followed
// by zero rows up to 16, into tails [B, 16, d] (an empty sequence gets 16 zero rows): that group is then
// contracted like any other and the zero rows add nothing.  gridDim = (B, 2): y picks X or dY.
// src: [rows, d] bf16 bit patterns, d a multiple of 8, 16-byte aligned.
struct TailTensor {
  const uint16_t* src;
  uint16_t* tails;
  int d;
};
__global__ void __launch_bounds__(STAGE_THREADS)
pack_tails_kernel(TailTensor tx_, TailTensor ty_, const int* __restrict__ offsets, long long total_rows) {
  const TailTensor& tn = blockIdx.y == 0 ? tx_ : ty_;
  const int b = blockIdx.x, d8 = tn.d / 8;
  const int r0 = offsets[b], r1 = offsets[b + 1];
  const int len = r1 > r0 ? r1 - r0 : 0;
  const int rem = len & 15;
  const long long first = (long long)r0 + (len - rem);         // first row of the partial group
  uint4* __restrict__ dst = reinterpret_cast<uint4*>(tn.tails) + (size_t)b * 16 * d8;
  for (int k = threadIdx.x; k < 16 * d8; k += STAGE_THREADS) {
    const int r = k / d8, c = k - r * d8;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    const long long row = first + r;
    if (r < rem && row >= 0 && row < total_rows) v = __ldg(reinterpret_cast<const uint4*>(tn.src) + row * d8 + c);
    dst[k] = v;
  }
}

}  // namespace pe
