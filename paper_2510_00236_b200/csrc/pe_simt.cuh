// SIMT (CUDA-core) kernels for the per-example statistics: the fp32-input path and the path for
// shapes the tensor-core kernel does not take.  One thread block owns a 64x64 tile of the
// [d_out, d_in] output and walks over the examples of its slice of the batch; the per-example
// gradient tile lives in registers and never reaches global memory.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "pe_optim.cuh"

namespace pe {

constexpr int SIMT_TILE = 64;   // output tile edge
constexpr int SIMT_TK = 16;     // tokens staged per step
constexpr int SIMT_THREADS = 256;

enum : int { MODE_STATS = 0, MODE_TOKEN = 1, MODE_NORMS = 2 };

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }

// phi: 0 identity, 1 square, 2 sign, 3 the clipping scale coef * g
__device__ __forceinline__ float apply_phi(float g, int phi, float coef) {
  if (phi == 1) return g * g;
  if (phi == 2) return (g > 0.f ? 1.f : 0.f) - (g < 0.f ? 1.f : 0.f);
  if (phi == 3) return coef * g;
  return g;
}

// What a packed batch or a clipped sum adds to the plain call; all NULL / 0 otherwise.
struct SimtExtra {
  const int* seq_offsets;     // [B + 1]: example b owns token rows offsets[b] .. offsets[b+1]-1 of X [rows, d_in], dY [rows, d_out]
  long long total_rows;       // rows of the packed tensors (reads are kept inside)
  const float* sq_norms;      // phi == 3: [B] squared norms N_b;  coef_b = min(1, clip_norm / sqrt(N_b))
  float clip_norm;
};

// MODE_STATS: out_mean = sum_b G_b, out_stat = sum_b phi(G_b)         (Section 2.3, Eq. (2))
// MODE_TOKEN: out_stat = sum_{b,t} dY^2 X^2; operands are squared as they are staged and the
//             accumulator is never reset between examples             (Section 2.3, per-token form)
// MODE_NORMS: out_stat is a [B] array, zero on entry; every tile adds its share of ||G_b||_F^2 to
//             out_stat[b] (Section 2.3, per-example squared norms); no [d_out, d_in] output
// gridDim = (ceil(d_in/64), ceil(d_out/64), nsplit); block z handles examples [z*B/nsplit, (z+1)*B/nsplit).
// With nsplit > 1 the outputs must be zero on entry and partial sums are added atomically; with
// accumulate != 0 the results are added to whatever the outputs hold.  opt.kind != 0 (nsplit == 1 only):
// the block also applies the parameter update to its tile (phi must then be square for the Adam family,
// sign for MicroSignSGD); out_mean / out_stat may then be NULL.
template <typename TIn, int MODE>
__global__ void __launch_bounds__(SIMT_THREADS)
simt_stats_kernel(const TIn* __restrict__ X, const TIn* __restrict__ dY, int B, int T, int d_in, int d_out,
                  int phi, float* __restrict__ out_mean, float* __restrict__ out_stat, int accumulate, SimtExtra ex, FusedOpt opt) {
  __shared__ float sY[SIMT_TK][SIMT_TILE];
  __shared__ float sX[SIMT_TK][SIMT_TILE];

  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int i0 = blockIdx.x * SIMT_TILE, o0 = blockIdx.y * SIMT_TILE;
  const int nsplit = gridDim.z;
  const int b_begin = (int)(((long long)B * blockIdx.z) / nsplit);
  const int b_end = (int)(((long long)B * (blockIdx.z + 1)) / nsplit);

  float g[4][4], acc_stat[4][4], acc_mean[4][4];
#pragma unroll
  for (int r = 0; r < 4; ++r)
#pragma unroll
    for (int c = 0; c < 4; ++c) g[r][c] = acc_stat[r][c] = acc_mean[r][c] = 0.f;

  for (int b = b_begin; b < b_end; ++b) {
    if (MODE == MODE_STATS || MODE == MODE_NORMS) {
#pragma unroll
      for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int c = 0; c < 4; ++c) g[r][c] = 0.f;
    }
    long long row0 = (long long)b * T;
    int Tb = T;
    if (ex.seq_offsets) {            // packed batch: this example's own token range, clamped to the tensor
      const long long r0 = ex.seq_offsets[b], r1 = ex.seq_offsets[b + 1];
      row0 = r0 < 0 ? 0 : r0;
      const long long end = r1 > ex.total_rows ? ex.total_rows : r1;
      Tb = end > row0 ? (int)(end - row0) : 0;
    }
    float coef = 1.f;
    if (phi == 3) {
      const float nrm = sqrtf(ex.sq_norms[b]);
      coef = nrm > ex.clip_norm ? ex.clip_norm / nrm : 1.f;
    }
    const TIn* Xb = X + (size_t)row0 * d_in;
    const TIn* Yb = dY + (size_t)row0 * d_out;
    for (int t0 = 0; t0 < Tb; t0 += SIMT_TK) {
      // stage SIMT_TK tokens of both operands, zero-filling past T and past the matrix edge
#pragma unroll
      for (int k = 0; k < (SIMT_TK * SIMT_TILE) / SIMT_THREADS; ++k) {
        int idx = threadIdx.x + k * SIMT_THREADS;
        int tt = idx / SIMT_TILE, cc = idx % SIMT_TILE;
        int t = t0 + tt;
        float xv = 0.f, yv = 0.f;
        if (t < Tb) {
          if (i0 + cc < d_in) xv = to_f32(Xb[(size_t)t * d_in + i0 + cc]);
          if (o0 + cc < d_out) yv = to_f32(Yb[(size_t)t * d_out + o0 + cc]);
        }
        if (MODE == MODE_TOKEN) { xv *= xv; yv *= yv; }
        sX[tt][cc] = xv;
        sY[tt][cc] = yv;
      }
      __syncthreads();
#pragma unroll
      for (int k = 0; k < SIMT_TK; ++k) {
        float y[4], x[4];
#pragma unroll
        for (int r = 0; r < 4; ++r) y[r] = sY[k][ty + 16 * r];
#pragma unroll
        for (int c = 0; c < 4; ++c) x[c] = sX[k][tx + 16 * c];
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
          for (int c = 0; c < 4; ++c) g[r][c] = fmaf(y[r], x[c], g[r][c]);
      }
      __syncthreads();
    }
    if (MODE == MODE_NORMS) {
      float s = 0.f;            // entries outside the matrix are exact zeros (their operands were zero-filled)
#pragma unroll
      for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int c = 0; c < 4; ++c) s = fmaf(g[r][c], g[r][c], s);
#pragma unroll
      for (int d = 16; d > 0; d >>= 1) s += __shfl_xor_sync(0xffffffffu, s, d);
      if ((threadIdx.x & 31) == 0) atomicAdd(out_stat + b, s);
    }
    if (MODE == MODE_STATS) {
#pragma unroll
      for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          acc_mean[r][c] += g[r][c];
          acc_stat[r][c] += apply_phi(g[r][c], phi, coef);
        }
    }
  }

  if constexpr (MODE != MODE_NORMS) {       // MODE_NORMS has no [d_out, d_in] output
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      int o = o0 + ty + 16 * r;
      if (o >= d_out) continue;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        int i = i0 + tx + 16 * c;
        if (i >= d_in) continue;
        size_t at = (size_t)o * d_in + i;
        float vs = (MODE == MODE_TOKEN) ? g[r][c] : acc_stat[r][c];
        if (nsplit == 1 && !accumulate) {
          if (out_stat) out_stat[at] = vs;
          if (MODE == MODE_STATS && out_mean) out_mean[at] = acc_mean[r][c];
          // the parameter update of Algorithm 1 / Section 3.1, applied where the sums over the whole batch are
          if (MODE == MODE_STATS && opt.kind == OPT_ADAM) fused_update_one<OPT_ADAM>(opt, (long long)at, acc_mean[r][c], vs);
          if (MODE == MODE_STATS && opt.kind == OPT_SIGN) fused_update_one<OPT_SIGN>(opt, (long long)at, vs, 0.f);
        } else {
          if (out_stat) atomicAdd(out_stat + at, vs);
          if (MODE == MODE_STATS && out_mean) atomicAdd(out_mean + at, acc_mean[r][c]);
        }
      }
    }
  }
}

}  // namespace pe
