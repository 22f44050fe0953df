// Tensor-core kernel for the sequence-level per-example statistics (Section 2.3; Eq. (2)).
//
// Work unit: a CTA PAIR (a cluster of two thread blocks on two SMs) owns a 256 x NT tile of the
// [d_out, d_in] output (NT = 128, 192 or 256) and a contiguous slice of the batch.  For every example of
// the slice the tile of G_b = dY_b^T X_b is formed by pair-wide tcgen05 MMAs (cta_group::2,
// M = 256: each block supplies 128 rows of dY_b^T and half of the NT rows of X_b^T from its own
// shared memory and receives its 128 accumulator rows in its own tensor memory), read back by the
// epilogue warps, passed through phi and added to register-resident running sums (sum_b phi(G_b)
// and, when asked for, sum_b G_b).  The per-example tile never leaves the SM.  Pairing cuts the
// operand bytes each SM pulls from L2 per flop; an SM sustains about 70 B/clk from L2, a lone
// 128 x 128 tile would need 128 B/clk at full tensor rate, a 256 x 128 pair 96, a 256 x 192 pair 75, a
// 256 x 256 pair 64.
//
//   MEAN_REGS, NT = 128: two running sums per thread (64 + 64 registers)         -- both outputs, short sequences
//   MEAN_REGS, NT = 192: two running sums per thread (96 + 96 registers; the control
//                        warps shrink to 40 registers so that the epilogue warps can take 232) -- both outputs
//   MEAN_REGS_SIGN, NT = 128: the same plus sum_b sign(G_b), counted in 16-bit halves
//                        of 32 more registers                                      -- mean, square and sign in one pass
//   MEAN_HYBRID_SIGN, NT = 192: mean, square and sign on the wider tile: sum_b G_b^2 (96 registers), the sign
//                        counts (48) and a third of sum_b G_b (32) in registers, the other two thirds of
//                        sum_b G_b in the 128 tensor-memory columns the two accumulators leave free
//   MEAN_TMEM, NT = 256: sum_b phi(G_b) in 128 registers per thread, sum_b G_b in
//                        tensor memory beside ONE per-example accumulator, one issuer -- both outputs
//   MEAN_NONE, NT = 256: one running sum per thread (128 registers)               -- only sum_b phi(G_b) wanted
//   MEAN_NORMS, NT = 256: no running sums; every example's sum of squares over the
//                        tile is reduced and added to out_norms[b]                 -- per-example squared norms
//   PHI = 0,   NT = 256: no per-example reset (accumulate in tensor memory)        -- plain contraction over all rows
// Further template arguments: RAGGED (packed batches with per-example token ranges), OPT (the parameter
// update applied by the block that completes a tile's sums), F8 (e4m3 operands for the plain contraction).
//
// Warp roles per block (12 warps): 0 = TMA producer of the dY boxes, 2 = TMEM allocator, then TMA
// producer of the X boxes, 1 and 3 = MMA issuers (leader block only), 4..11 = epilogue (warp w reads
// TMEM lanes 32*(w%4)..+31, column half (w-4)/4).  One thread needs on the order of a hundred cycles
// per TMA instruction, so the boxes are tall (BK tokens, 16 KiB for bf16) and split over two warps.
// Two examples are in flight at once, one per issuer; the 512 TMEM columns hold 512/NT accumulators,
// so the MMAs of later examples overlap the epilogue of earlier ones.  (MEAN_TMEM has one issuer and
// one accumulator: while the epilogue drains it the producers keep filling the ring, and the issuer
// then works the backlog off at full tensor rate, which absorbs the pause as long as the operand
// supply, not the tensor pipe, is what bounds the example.)
//
// Barriers.  full[s] lives in the leader block: its producer posts the byte count of BOTH blocks'
// loads, and the follower's TMA loads credit their bytes to it through the cluster window.
// empty[s] and acc_full[a] exist in both blocks and are signalled in both by one multicast commit.
// acc_empty[a] lives in the leader and collects the arrivals of both blocks' epilogue warps.
//
// Operand orientation: A = dY_b viewed as M = d_out x K = T and B = X_b viewed as N = d_in x K = T.
// In global memory the contraction index (the token) is the slow one, so both operands are
// "MN-major".  A TMA box is 128 bytes of features (64 bf16) x BK tokens; with the 128-byte swizzle that is
// exactly the canonical MN-major layout of the MMA: 8-token x 64-feature atoms of 1 KiB, the next
// 8 tokens 1 KiB further (stride byte offset), the next 64 features one box further (leading byte
// offset).  (X at NT = 192: 64 bytes of features per box row and the 64-byte swizzle, 512-byte atoms.)
#pragma once
#include "pe_optim.cuh"
#include "pe_sm100.cuh"

namespace pe {

constexpr int TC_TILE_M = 128;    // d_out rows per block (the pair covers 256)
constexpr int TC_PAIR_M = 2 * TC_TILE_M;
constexpr int TC_TMEM_COLS = 512;
constexpr int TC_THREADS = 384;
constexpr int TC_REGS_CONTROL = 64;     // setmaxnreg of warps 0..3
constexpr int TC_REGS_EPILOGUE = 216;   // setmaxnreg of warps 4..11  (4*32*64 + 8*32*216 = 63488 <= 384*168)
constexpr int TC_REGS_AT_LAUNCH = 168;  // registers per thread of a 384-thread block at one block per SM (65536 / 384, in eights)
constexpr int TC_BAR_BYTES = 512;
// operand ring; leaves room for barriers and alignment slack.  The 256 x 192 tile's four 56 KiB stages take 224 KiB.
__host__ __device__ constexpr int tc_smem_budget(int nt) { return (nt == 192 ? 224 : 200) * 1024; }

// Operand element type of the MMA.  bf16 (kind::f16, 16 tokens per instruction) for the per-example
// statistics; tf32 (kind::tf32, fp32 storage, 8 tokens per instruction) for the per-token statistic,
// whose squared operands need more than bf16's 8 significant bits.  NT = d_in columns per pair tile.
// Default tokens per pipeline stage: 128 for the 256 x 128 tile, 64 for the 256 x 256 tile, 32 for
// tf32.  With both outputs and short sequences (T <= 32) the 256 x 128 tile takes 32-token stages
// instead: a 128-token box would be mostly zero fill, and 16 small slots keep more examples in flight.
__host__ __device__ constexpr int tc_default_bk(bool tf32, int nt) { return tf32 ? 32 : (nt == 256 ? 64 : 128); }
constexpr int TC_SHORT_BK = 32;
constexpr int TC_SHORT_T = 32;
// F8: 8-bit operands (kind::f8f6f4, e4m3, 32 tokens per instruction): the scaled squares of the two-pass
// per-token statistic's fp8 form.
template <bool TF32, int NT, int BK_ = tc_default_bk(TF32, NT), bool F8 = false>
struct TcOperand {
  static_assert(!(TF32 && F8), "one operand type");
  static constexpr int ELEM_BYTES = TF32 ? 4 : (F8 ? 1 : 2);
  static constexpr int BOX_FEATS = 128 / ELEM_BYTES;            // features per 128-byte swizzle row: 64 | 32 | 128
  // tokens per pipeline stage (one TMA box is BK tokens tall), chosen so that the ring has an EVEN
  // number of stages: with two MMA issuers taking alternate stages every slot then always belongs
  // to the same issuer (see the parity note at the issuer's wait).
  static constexpr int BK = BK_;
  static constexpr int MMA_K = 32 / ELEM_BYTES;                 // tokens per MMA instruction: 16 | 8 | 32
  // Short sequences (the 32-token stages of the 256 x 128 tile): a stage holds TWO examples (the TMA box is
  // two examples deep, 32 tokens each), the issuer fills both of its accumulators from it and the epilogue
  // drains both behind one barrier: half the barrier hand-offs per example, which is what bounds T <= 32.
  static constexpr int GROUP = (!TF32 && !F8 && NT == 128 && BK_ == TC_SHORT_BK) ? 2 : 1;
  static constexpr int BOX_BYTES = 128 * BK * GROUP;            // one box: GROUP x BK tokens x 128 bytes
  static constexpr int A_BOXES = TC_TILE_M / BOX_FEATS;         // this block's 128 rows of dY^T
  static constexpr int B_FEATS = NT / 2;                        // this block's half of the tile's d_in columns
  // NT = 192: 96 columns of X per block are one and a half 128-byte rows.  X is then loaded in
  // 64-byte rows (32 features per box, TMA SWIZZLE_64B) and described to the MMA with the 64-byte
  // swizzle (descriptor layout 4: 8-token x 32-feature atoms of 512 bytes); dY keeps 128-byte rows.
  static constexpr bool B_NARROW = (B_FEATS % BOX_FEATS) != 0;
  static_assert(!B_NARROW || !TF32, "64-byte rows are only set up for 16-bit operands");
  static constexpr int B_ROW_BYTES = B_NARROW ? 64 : 128;
  static constexpr int B_BOX_FEATS = B_ROW_BYTES / ELEM_BYTES;  // 64 | 32
  static constexpr int B_BOX_BYTES = B_ROW_BYTES * BK * GROUP;
  static constexpr int B_BOXES = B_FEATS / B_BOX_FEATS;         // 1 | 2 | 3
  static constexpr int A_BYTES = A_BOXES * BOX_BYTES;           // 32 KiB (BK = 128) | 16 KiB
  static constexpr int B_BYTES = B_BOXES * B_BOX_BYTES;         // 16 KiB | 24 KiB (NT = 192)
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;         // per block: 48 KiB | 56 KiB | 32 KiB
  static constexpr int STAGES = (tc_smem_budget(NT) / STAGE_BYTES) & ~1;   // 4 | 4 | 6 | 16 with 32-token stages
  static_assert(STAGES % 2 == 0, "slots must alternate between the two issuers");
  static constexpr int K_STEP_BYTES = MMA_K * 128;              // smem advance per MMA: 2048 | 1024
  static constexpr int B_K_STEP_BYTES = MMA_K * B_ROW_BYTES;
  static constexpr int ACC_BUFS = TC_TMEM_COLS / NT;            // 4 | 2 | 2 accumulators in tensor memory
  // MN-major swizzle atoms: bf16 = 8 tokens x 128 B with 16-byte chunks (descriptor layout 2, TMA
  // SWIZZLE_128B); tf32 = 4 tokens x 128 B with 32-byte chunks (layout 1, TMA SWIZZLE_128B_ATOM_32B).
  static constexpr uint32_t DESC_LAYOUT = TF32 ? 1u : 2u;
  static constexpr uint32_t SBO_BYTES = TF32 ? 512u : 1024u;   // next swizzle atom along the tokens
  static constexpr uint32_t B_DESC_LAYOUT = B_NARROW ? 4u : DESC_LAYOUT;
  static constexpr uint32_t B_SBO_BYTES = B_NARROW ? 512u : SBO_BYTES;
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + TC_BAR_BYTES + 1024;   // + alignment slack
  // Register split between the four control warps and the eight epilogue warps (setmaxnreg).  The pool
  // is what the block was launched with, 384 threads x 168 registers, NOT the SM's whole register file: an
  // increase that the decreases of the control warps do not cover never returns.  Two running sums of
  // 96 floats each need the larger epilogue share.
  static constexpr int REGS_CONTROL = (NT == 192) ? 40 : TC_REGS_CONTROL;
  static constexpr int REGS_EPILOGUE = (NT == 192) ? 232 : TC_REGS_EPILOGUE;
  static_assert(128 * REGS_CONTROL + 256 * REGS_EPILOGUE <= TC_THREADS * TC_REGS_AT_LAUNCH, "setmaxnreg: the epilogue's increase must fit what the control warps give up");
};

// error codes latched in the device status word (which wait gave up)
enum : int { TC_WAIT_EMPTY = 1, TC_WAIT_FULL = 2, TC_WAIT_ACC_EMPTY = 3, TC_WAIT_ACC_FULL = 4 };

struct TcParams {
  int B, T, d_in, d_out;
  int pairs_m, tiles_n, band;   // tile grid: 256-row pair rows x NT-column tiles; pair rows per band of the tile order
  int nsplit;          // batch slices (gridDim.z); > 1 => outputs pre-zeroed, partials added atomically
  int per_example;     // 1: reset the accumulator for every example and apply phi (statistics)
                       // 0: one accumulation over the whole slice (plain contraction, phi = identity)
  int half_operands;   // 16-bit operands are IEEE half instead of bf16 (the staged per-token statistic)
  int accumulate;      // add the results to what the outputs hold (no zeroing kernel runs before this one)
  float* out_mean;     // may be NULL; written through tmap_mean
  float* out_stat;     // may be NULL; written through tmap_stat
  float* out_sign;     // MEAN_REGS_SIGN only: sum_b sign(G_b), written through tmap_sign
  float* out_norms;    // MEAN_NORMS only: [B], zero on entry; every tile adds its share of ||G_b||_F^2
  const int* seq_offsets;   // RAGGED only: [B + 1] token-row offsets; example b owns rows offsets[b] .. offsets[b+1]-1
  const float* sq_norms;    // PHI == 3 only: [B] per-example squared norms the clipping coefficient is taken from
  float clip_norm;          // PHI == 3 only: C of c_b = min(1, C / sqrt(N_b))
  unsigned int* dev_status;
};

// Where an example's tokens are and how many pipeline stages they take.  Fixed-length batches: the
// operand maps are 3-D (d, T, B), an example is the coordinate `seq` of the last dimension and its
// stages start at token 0.  Packed (ragged) batches: the maps are (d, rows, 1), the example starts at
// row `row0`; its whole 16-token groups (`main` tokens) come from there in `nk_main` stages, and its
// last `len % 16` tokens come, zero-padded to 16, from a side buffer that a pre-pass fills (a map
// (d, 16, B)): one more stage with one MMA step.  An empty sequence is such a tail stage of zeros, so
// that every example owns at least one stage and one accumulator.
struct SeqGeom {
  int row0, main, nk_main, nk;
};
template <bool RAGGED>
__device__ __forceinline__ SeqGeom seq_geom(const TcParams& p, int b, int bk) {
  SeqGeom g;
  if constexpr (RAGGED) {
    const int r0 = __ldg(p.seq_offsets + b), r1 = __ldg(p.seq_offsets + b + 1);
    const int len = r1 > r0 ? r1 - r0 : 0;
    g.row0 = r0;
    g.main = len & ~15;
    g.nk_main = (g.main + bk - 1) / bk;
    g.nk = g.nk_main + (((len & 15) != 0 || len == 0) ? 1 : 0);
  } else {
    g.row0 = 0;
    g.main = p.T;
    g.nk_main = g.nk = (p.T + bk - 1) / bk;
  }
  return g;
}

// Tile order.  Pairs that run at the same time should share operand panels in L2, so consecutive
// pair indices sweep the d_in tiles inside a band of p.band pair rows before moving to the next band:
// the ~74 resident pairs then touch about band*256 columns of dY and 74/band*NT columns of X per
// example instead of all of dY.  Returns this block's 128-row tile of d_out and NT-column tile of d_in.
__device__ __forceinline__ void tc_tile_of_block(const TcParams& p, uint32_t rank, int& tile_m, int& tile_n) {
  const int pair_id = blockIdx.x >> 1;
  const int per_band = p.band * p.tiles_n;
  const int band = pair_id / per_band, r = pair_id - band * per_band;
  const int rows = min(p.band, p.pairs_m - band * p.band);      // pair rows in this (possibly last, shorter) band
  tile_n = r / rows;
  tile_m = 2 * (band * p.band + (r - tile_n * rows)) + (int)rank;
}

// (sign(g) + 1) / 2, i.e. 0, 0.5 or 1, with sign(+-0) = 0, in two instructions: g is scaled by 2^64 (exact, or to
// infinity; the callers do it two columns at a time), then 2^127 * g + 0.5 is rounded and saturated to [0, 1].  The
// smallest nonzero |g|, the denormal 2^-149, arrives as 2^42, so every nonzero g saturates and zero alone gives 0.5.
// Summed over nb examples this is (sum_b sign(G_b) + nb) / 2, exact in fp32 (multiples of 0.5 below 2^23).
constexpr float SIGN_PRESCALE = 18446744073709551616.f;     // 2^64
__device__ __forceinline__ float sign_half_of_scaled(float g_scaled) {
  float u;
  asm("fma.rn.sat.f32 %0, %1, 0f7F000000, 0f3F000000;" : "=f"(u) : "f"(g_scaled));
  return u;
}
__device__ __forceinline__ float sign_half(float g) { return sign_half_of_scaled(g * SIGN_PRESCALE); }
// The same for two columns: {u(lo), u(hi)} packed for the two-wide fp32 instructions.
__device__ __forceinline__ uint64_t sign_half2(uint64_t g2) {
  float a0, a1;
  sm100::f32x2_unpack(sm100::f32x2_mul(g2, sm100::f32x2_pack(SIGN_PRESCALE, SIGN_PRESCALE)), a0, a1);
  return sm100::f32x2_pack(sign_half_of_scaled(a0), sign_half_of_scaled(a1));
}
// Two columns' sign(g) + 1 in {0, 1, 2} as the low and high 16 bits of one word: 2 u + 1.5 * 2^23 has the integer in
// the low bits of its pattern, and one byte permute packs the two low halves.
__device__ __forceinline__ uint32_t sign_plus_one_packed(uint64_t g2) {
  float t0, t1;
  sm100::f32x2_unpack(sm100::f32x2_fma(sign_half2(g2), sm100::f32x2_pack(2.f, 2.f), sm100::f32x2_pack(12582912.f, 12582912.f)), t0, t1);
  return __byte_perm(__float_as_uint(t0), __float_as_uint(t1), 0x5410);
}

template <int PHI>
__device__ __forceinline__ float phi_apply(float g) {
  if (PHI == 1) return g * g;
  if (PHI == 2) {
    // sign(g) with sign(+-0) = 0: (g != 0) as 1.0f / 0.0f, then g's sign bit copied onto it (-0.0f adds nothing)
    const float nz = (g != 0.f) ? 1.f : 0.f;
    return __uint_as_float(__float_as_uint(nz) | (__float_as_uint(g) & 0x80000000u));
  }
  return g;
}

// The operand ring and the two issuers.  Issuer x owns the ring slots of parity x (a sub-ring of
// STAGES / 2 slots with its own phase) and the examples x, x + 2, ... of the slice, so the two issuers
// run independently of each other.  The producers fill the two sub-rings in alternation, one stage of
// each in turn while both still have stages to fill: with equal sequence lengths that is stage kc of an
// even example, stage kc of the next odd one, stage kc + 1 of the even one, ...; with unequal lengths
// (packed batches) the issuer of a short example simply moves on to its next example earlier.  A parity
// wait is only meaningful while the waiter is at most one phase away from the barrier; since a slot
// only ever sees the stages of ONE sub-ring, in order, that always holds.
struct RingCursor {
  int e, kc, n;       // example (slice-local), stage within it, stages of this sub-ring filled so far
  SeqGeom g;
};

// Zeroes the outputs of a split-batch launch.  The statistics kernel that follows is launched as a
// programmatic dependent: it starts right away (it only touches the outputs in its very last step,
// behind griddepcontrol.wait), so the zeroing costs no time on the stream.  a, b, c: n4 float4 each; b and
// c may be NULL.  counters: the tile counters of a fused update (n_counters words; may be NULL).
__global__ void __launch_bounds__(256) zero_outputs_kernel(float4* __restrict__ a, float4* __restrict__ b, float4* __restrict__ c,
                                                           long long n4, unsigned int* __restrict__ counters, int n_counters) {
  sm100::griddep_launch_dependents();
  const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
  const long long stride = (long long)gridDim.x * blockDim.x;
  if (counters)
    for (long long k = (long long)blockIdx.x * blockDim.x + threadIdx.x; k < n_counters; k += stride) counters[k] = 0u;
  for (long long k = (long long)blockIdx.x * blockDim.x + threadIdx.x; k < n4; k += stride) {
    a[k] = z;
    if (b) b[k] = z;
    if (c) c[k] = z;
  }
}

// where sum_b G_b is kept in per-example mode; MEAN_REGS_SIGN = MEAN_REGS with phi = square plus the sign statistic
// MEAN_NORMS keeps no [d_out, d_in] sums at all: it reduces each G_b tile to its sum of squares
enum : int { MEAN_NONE = 0, MEAN_REGS = 1, MEAN_TMEM = 2, MEAN_REGS_SIGN = 3, MEAN_NORMS = 4, MEAN_HYBRID_SIGN = 5 };
constexpr int TC_SIGN_COUNT_MAX = 32767;   // examples per block in MEAN_REGS_SIGN mode: 2 * count must fit 16 bits

// gridDim = (2 * pairs_m * tiles_n, 1, nsplit); blockIdx.x = 2 * (pair index in the tile order) + rank in pair.
// The fused parameter update of one epilogue warp's 32-row x (PANELS * 32)-column piece of the tile.  The piece
// is walked as float4 groups, a warp instruction covering 128 float4 in row-major order (global accesses of a
// warp are whole 16-byte groups of one or two rows), whereas the running sums live one ROW per lane: the sums
// therefore come either from the warp's staged panels in shared memory (the 128-byte-swizzled 32 x 32 panels the
// write-out also hands to TMA; chunk k of row r sits at chunk position k ^ (r & 7)) or, when the batch was
// split and this block added the last partial sum, from the outputs in global memory (read past L1).  Eight
// float4 per array and lane are in flight at a time (about 100 KiB per SM): the step is a latency-bound tail
// during which the block's tensor cores idle, so what counts is the number of memory round trips.
template <int OPT, int PANELS>
__device__ __forceinline__ void fused_update_piece(const FusedOpt& o, const TcParams& p, int row0, int col0, int lane,
                                                   const uint8_t* stat_panels, const uint8_t* mean_panels) {
  constexpr int C4 = PANELS * 8;             // float4 groups per row of the piece
  constexpr int ITERS = C4;                  // 32 rows x C4 groups / 32 lanes
  constexpr int BATCH = 8;
  static_assert(ITERS % BATCH == 0, "whole batches");
  const float4 zero4 = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 1
  for (int it0 = 0; it0 < ITERS; it0 += BATCH) {
    float4 th[BATCH], mm[BATCH], vv[BATCH], s1[BATCH], s2[BATCH];
#pragma unroll
    for (int i = 0; i < BATCH; ++i) {
      const int k = (it0 + i) * 32 + lane;
      const int r = k / C4, c4 = k - r * C4;
      const int row = row0 + r, col = col0 + 4 * c4;
      const bool in = row < p.d_out && col < p.d_in;           // d_in is a multiple of 8: a group is all in or all out
      const long long idx = (long long)row * p.d_in + col;
      th[i] = in ? *reinterpret_cast<const float4*>(o.theta + idx) : zero4;
      mm[i] = in ? *reinterpret_cast<const float4*>(o.m + idx) : zero4;
      vv[i] = (OPT == OPT_ADAM && in) ? *reinterpret_cast<const float4*>(o.v + idx) : zero4;
      float4 st, mn = zero4;
      if (stat_panels) {
        const int off = (c4 >> 3) * 4096 + r * 128 + (((c4 & 7) ^ (r & 7)) << 4);
        st = *reinterpret_cast<const float4*>(stat_panels + off);
        if (OPT == OPT_ADAM) mn = *reinterpret_cast<const float4*>(mean_panels + off);
      } else {
        st = in ? __ldcg(reinterpret_cast<const float4*>(p.out_stat + idx)) : zero4;
        if (OPT == OPT_ADAM) mn = in ? __ldcg(reinterpret_cast<const float4*>(p.out_mean + idx)) : zero4;
      }
      s1[i] = (OPT == OPT_ADAM) ? mn : st;
      s2[i] = st;
    }
#pragma unroll
    for (int i = 0; i < BATCH; ++i) {
      const int k = (it0 + i) * 32 + lane;
      const int r = k / C4, c4 = k - r * C4;
      const int row = row0 + r, col = col0 + 4 * c4;
      if (row < p.d_out && col < p.d_in) {
        const long long idx = (long long)row * p.d_in + col;
        if constexpr (OPT == OPT_ADAM) {
          adam_one_rt(o.variant, th[i].x, mm[i].x, vv[i].x, s1[i].x, s2[i].x, o.adam);
          adam_one_rt(o.variant, th[i].y, mm[i].y, vv[i].y, s1[i].y, s2[i].y, o.adam);
          adam_one_rt(o.variant, th[i].z, mm[i].z, vv[i].z, s1[i].z, s2[i].z, o.adam);
          adam_one_rt(o.variant, th[i].w, mm[i].w, vv[i].w, s1[i].w, s2[i].w, o.adam);
          *reinterpret_cast<float4*>(o.v + idx) = vv[i];
        } else {
          sign_one(th[i].x, mm[i].x, s1[i].x, o.sign);
          sign_one(th[i].y, mm[i].y, s1[i].y, o.sign);
          sign_one(th[i].z, mm[i].z, s1[i].z, o.sign);
          sign_one(th[i].w, mm[i].w, s1[i].w, o.sign);
        }
        *reinterpret_cast<float4*>(o.theta + idx) = th[i];
        *reinterpret_cast<float4*>(o.m + idx) = mm[i];
        if (o.theta_lp) {
          const __nv_bfloat162 lo = __floats2bfloat162_rn(th[i].x, th[i].y), hi = __floats2bfloat162_rn(th[i].z, th[i].w);
          uint2 pk;
          pk.x = *reinterpret_cast<const unsigned int*>(&lo);
          pk.y = *reinterpret_cast<const unsigned int*>(&hi);
          *reinterpret_cast<uint2*>(o.theta_lp + idx) = pk;
        }
      }
    }
  }
}

// RAGGED: packed batch with per-example token ranges (tmap_x / tmap_dy are then (d, rows, 1), tmap_x_tail /
// tmap_dy_tail (d, 16, B) over the zero-padded last partial token groups); otherwise the tail maps are unused.
// PHI: 0 identity, 1 square, 2 sign, 3 the clipping scale c_b * g with c_b = min(1, C / sqrt(N_b)).
// OPT: the parameter update applied by the block that completes a tile's sums (OPT_ADAM needs both running
// sums, OPT_SIGN the sign statistic alone); `o` is ignored when OPT == OPT_NONE.
template <int PHI, bool TF32, int NT, int MEAN, int BKT = tc_default_bk(TF32, NT), bool RAGGED = false, int OPT = OPT_NONE, bool F8 = false>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(TC_THREADS, 1)
tc_stats_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_dy,
                const __grid_constant__ CUtensorMap tmap_mean, const __grid_constant__ CUtensorMap tmap_stat,
                const __grid_constant__ CUtensorMap tmap_sign, const __grid_constant__ CUtensorMap tmap_x_tail,
                const __grid_constant__ CUtensorMap tmap_dy_tail, TcParams p, FusedOpt o) {
  using namespace sm100;
  using Op = TcOperand<TF32, NT, BKT, F8>;
  static_assert(!F8 || (PHI == 0 && NT == 256 && !RAGGED), "8-bit operands: the plain contraction of the per-token statistic");
  constexpr bool HYBRID = (MEAN == MEAN_HYBRID_SIGN);
  constexpr bool TRIPLE = (MEAN == MEAN_REGS_SIGN) || HYBRID;
  static_assert((MEAN != MEAN_REGS && MEAN != MEAN_REGS_SIGN) || NT == 128 || (NT == 192 && MEAN == MEAN_REGS), "two running sums only fit the registers up to NT = 192");
  static_assert(NT != 192 || MEAN == MEAN_REGS || HYBRID, "the 256 x 192 tile exists for both running sums");
  static_assert(!HYBRID || (NT == 192 && !RAGGED && OPT == OPT_NONE), "the hybrid mean fills the tensor-memory columns two 192-column accumulators leave free");
  static_assert(!TRIPLE || PHI == 1, "the three-statistic mode is mean + square + sign");
  constexpr bool NORMS = (MEAN == MEAN_NORMS);
  static_assert(!NORMS || (PHI == 1 && NT == 256), "per-example norms: squares on the 256 x 256 tile");
  static_assert(MEAN != MEAN_TMEM || (NT == 256 && PHI != 0), "the tensor-memory mean sits beside one 256-column accumulator");
  static_assert(!RAGGED || (!TF32 && MEAN != MEAN_TMEM), "packed batches: 16-bit operands, two issuers");
  static_assert(PHI != 3 || MEAN == MEAN_NONE, "the clipped sum is a statistic-only pass");
  static_assert(OPT != OPT_ADAM || (MEAN == MEAN_REGS && PHI == 1), "the Adam family consumes sum_b G_b and sum_b G_b^2");
  static_assert(OPT != OPT_SIGN || (MEAN == MEAN_NONE && PHI == 2), "MicroSignSGD consumes sum_b sign(G_b)");
  constexpr int STAGES = Op::STAGES, BK = Op::BK;
  constexpr int BOX_BYTES = Op::BOX_BYTES, A_BYTES = Op::A_BYTES, STAGE_BYTES = Op::STAGE_BYTES;
  constexpr int ISSUERS = (MEAN == MEAN_TMEM) ? 1 : 2;
  constexpr int ACC_BUFS = (MEAN == MEAN_TMEM) ? 1 : Op::ACC_BUFS;
  constexpr int BUFS_PER_ISSUER = ACC_BUFS / ISSUERS;     // 2 | 1
  // GROUP examples share a stage and a pair of accumulator barriers (short sequences): the unit of work of
  // the producers, issuers and epilogue warps is then a group of GROUP consecutive examples
  constexpr int GROUP = Op::GROUP;
  constexpr int UNITS_PER_ISSUER = BUFS_PER_ISSUER / GROUP;      // accumulator units (of GROUP buffers) per issuer
  static_assert(GROUP == 1 || ((MEAN == MEAN_REGS || MEAN == MEAN_REGS_SIGN) && !RAGGED && OPT == OPT_NONE && UNITS_PER_ISSUER == 1),
                "grouped examples: the short-sequence variants of the two- and three-sum kernels");
  constexpr int MEAN_COL0 = 256;                    // first tensor-memory column of the MEAN_TMEM running sum
  constexpr int COLS = NT / 2;                      // accumulator columns per epilogue thread
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t bar_base = smem_base + STAGES * STAGE_BYTES;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (STAGES + s); };
  auto acc_full_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + a); };
  auto acc_empty_bar = [&](int a) { return bar_base + 8u * (2 * STAGES + ACC_BUFS + a); };
  static_assert(8 * (2 * STAGES + 2 * ACC_BUFS) + 16 <= TC_BAR_BYTES, "barrier area too small");
  uint8_t* tail = smem_gen + STAGES * STAGE_BYTES + 8 * (2 * STAGES + 2 * ACC_BUFS);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(tail);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tail + 8);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();          // 0 = leader of the pair
  const int b_begin = (int)(((long long)p.B * blockIdx.z) / p.nsplit);
  const int b_end = (int)(((long long)p.B * (blockIdx.z + 1)) / p.nsplit);
  const int nb = b_end - b_begin;
  const int nu = (nb + GROUP - 1) / GROUP;          // units of work: groups of GROUP examples (GROUP = 1: the examples)

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < ACC_BUFS; ++a) { mbar_init(acc_full_bar(a), 1); mbar_init(acc_empty_bar(a), 16); }
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 2) { tmem_alloc_pair(smem_u32(const_cast<uint32_t*>(tmem_slot)), TC_TMEM_COLS); tmem_relinquish_pair(); }
  tc_fence_before();
  cluster_sync_all();          // barriers of both blocks initialised before any remote arrival
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // Register budget: the epilogue warpgroups hold 128 floats of running sums plus a 32-register TMEM
  // read per thread; the producer / MMA warpgroup needs little.  Each setmaxnreg sits inside the
  // branch of the role it applies to.
  if (warp < 4) {
    setmaxnreg_dec<Op::REGS_CONTROL>();
    if (warp == 0 || warp == 2) {
      // ---------------------------------------------------------- TMA producers (both blocks)
      // Warp 0 loads this block's rows of dY^T (and, in the leader, posts the stage's byte count);
      // warp 2 loads this block's half of the X^T rows.  Both wait for the same "stage empty" phase and
      // fill the two issuers' sub-rings in alternation (see RingCursor).
      if (lane == 0) {
        const bool is_a = (warp == 0);
        int tile_m, tile_n;
        tc_tile_of_block(p, rank, tile_m, tile_n);
        const CUtensorMap* tmap = is_a ? &tmap_dy : &tmap_x;
        const CUtensorMap* tmap_tail = is_a ? &tmap_dy_tail : &tmap_x_tail;
        const int c0 = is_a ? tile_m * TC_TILE_M : tile_n * NT + (int)rank * Op::B_FEATS;   // first feature of this warp's boxes
        const int n_boxes = is_a ? Op::A_BOXES : Op::B_BOXES;
        const int box_feats = is_a ? Op::BOX_FEATS : Op::B_BOX_FEATS;
        const int box_bytes = is_a ? BOX_BYTES : Op::B_BOX_BYTES;
        prefetch_tensormap(tmap);
        if constexpr (RAGGED) prefetch_tensormap(tmap_tail);
        constexpr int SUB = STAGES / ISSUERS;            // slots per sub-ring
        auto start = [&](RingCursor& c, int x) {
          c.e = x; c.kc = 0; c.n = 0;
          if (c.e < nu) c.g = seq_geom<RAGGED>(p, b_begin + GROUP * c.e, BK);
        };
        // Fills the next stage of sub-ring x if it has one and its slot is free; never blocks, because a
        // sub-ring may stay full for as long as the OTHER one has to be filled (its issuer waits for an
        // accumulator that the epilogue frees only after the other issuer's example).
        auto try_fill = [&](RingCursor& c, int x) -> bool {
          if (c.e >= nu) return false;
          const int s = ISSUERS * (c.n % SUB) + x;
          const uint32_t ph = (uint32_t)(c.n / SUB) & 1u;
          if (!mbar_test_wait(empty_bar(s), ph ^ 1u)) return false;
          if (is_a && rank == 0) mbar_arrive_expect_tx(full_bar(s), 2 * STAGE_BYTES);     // both blocks' bytes
          const uint32_t leader_full = map_to_cta(full_bar(s), 0);
          const uint32_t dst = smem_base + s * STAGE_BYTES + (is_a ? 0 : A_BYTES);
          if constexpr (RAGGED) {
            const bool tail = c.kc >= c.g.nk_main;       // the zero-padded last partial group, from the side buffer
            for (int g = 0; g < n_boxes; ++g)
              tma_load_3d_pair(dst + g * box_bytes, tail ? tmap_tail : tmap, leader_full, c0 + g * box_feats,
                               tail ? 0 : c.g.row0 + c.kc * BK, tail ? b_begin + c.e : 0);
          } else {
            // (grouped examples: the box is GROUP examples deep; past the batch's end it reads zeros)
            for (int g = 0; g < n_boxes; ++g)
              tma_load_3d_pair(dst + g * box_bytes, tmap, leader_full, c0 + g * box_feats, c.kc * BK, b_begin + GROUP * c.e);
          }
          ++c.n;
          if (++c.kc == c.g.nk) {
            c.kc = 0;
            c.e += ISSUERS;
            if (c.e < nu) c.g = seq_geom<RAGGED>(p, b_begin + GROUP * c.e, BK);
          }
          return true;
        };
        RingCursor ca, cb;
        start(ca, 0);
        start(cb, ISSUERS == 2 ? 1 : nu);
        long long t0 = -1;
        unsigned int spins = 0;
        while (ca.e < nu || cb.e < nu) {
          bool progressed = try_fill(ca, 0);
          if (ISSUERS == 2 && try_fill(cb, 1)) progressed = true;
          if (progressed) { t0 = -1; spins = 0; continue; }
          if ((++spins & (wait_cycle_limit() < (1ll << 20) ? 0u : 0xffu)) == 0) {      // bounded like every other wait
            if (*abort_flag) break;
            if (t0 < 0) t0 = clock64();
            else if (clock64() - t0 > wait_cycle_limit()) {
              *abort_flag = 1;
              atomicCAS(p.dev_status, 0u, (unsigned int)TC_WAIT_EMPTY);
              break;
            }
          }
        }
      }
      __syncwarp();
    } else if (rank == 0 && (warp == 1 || ISSUERS == 2)) {
      // ---------------------------------------------------------- MMA issuers (leader block, warps 1 and 3)
      // Two issuing threads (one per warp).  A barrier probe right after queuing MMAs costs the
      // issuing thread a couple of hundred cycles; with two threads working on two different examples
      // (own accumulators, alternate stages) one of them always has MMAs queued.  Issuer x owns
      // examples x, x+2, ... of the slice and TMEM buffers x*BUFS_PER_ISSUER .. +BUFS_PER_ISSUER-1.
      if (lane == 0) {
        const int x = (warp == 1) ? 0 : 1;
        // operand format code 0 is IEEE half under kind::f16 and e4m3 under kind::f8f6f4
        const uint32_t idesc = (F8 || (!TF32 && p.half_operands)) ? make_idesc_half_mn_major(TC_PAIR_M, NT) : make_idesc_mn_major(TC_PAIR_M, NT, TF32);
        bool ok = true;
        uint32_t accumulate = 0;
        constexpr int SUB = STAGES / ISSUERS;              // slots of this issuer's sub-ring
        int i_local = 0;                                   // examples this issuer has started
        int n_local = 0;                                   // stages this issuer has consumed
        for (int e = x; e < nu && ok; e += ISSUERS, ++i_local) {
          const SeqGeom sg = seq_geom<RAGGED>(p, b_begin + GROUP * e, BK);
          const int grp = p.per_example ? i_local : 0;
          const int buf = UNITS_PER_ISSUER * x + (grp % UNITS_PER_ISSUER);      // accumulator unit: GROUP buffers, one barrier pair
          if (p.per_example || i_local == 0) {
            const uint32_t acc_ph = (uint32_t)(grp / UNITS_PER_ISSUER) & 1u;
            if (!mbar_wait_bounded(acc_empty_bar(buf), acc_ph ^ 1u, abort_flag, p.dev_status, TC_WAIT_ACC_EMPTY)) { ok = false; break; }
            tc_fence_after();
            accumulate = 0;
          }
          const uint32_t d_tmem = tmem_base + (uint32_t)(buf * GROUP * NT);
          for (int kc = 0; kc < sg.nk; ++kc, ++n_local) {
            const int s = ISSUERS * (n_local % SUB) + x;
            const uint32_t ph = (uint32_t)(n_local / SUB) & 1u;
            if (!mbar_wait_bounded(full_bar(s), ph, abort_flag, p.dev_status, TC_WAIT_FULL)) { ok = false; break; }
            tc_fence_after();
            const uint32_t a_src = smem_base + s * STAGE_BYTES;
            const uint32_t b_src = a_src + A_BYTES;
            // tokens of this example in this stage: the rest of its whole 16-token groups, or the padded tail group
            const int t_left = (RAGGED && kc >= sg.nk_main) ? 16 : sg.main - kc * BK;
#pragma unroll
            for (int j = 0; j < GROUP; ++j) {
              // grouped examples: example j of the group sits BK tokens further in every box and has its own accumulator
              if (GROUP > 1) { if (GROUP * e + j >= nb) break; accumulate = 0; }
#pragma unroll
              for (int k = 0; k < BK / Op::MMA_K; ++k) {
                // rows past T are zero-filled by TMA; whole MMA steps past T are skipped
                if (k * Op::MMA_K < t_left) {
                  const uint64_t ad = make_smem_desc(a_src + j * (BK * 128) + k * Op::K_STEP_BYTES, BOX_BYTES, Op::SBO_BYTES, Op::DESC_LAYOUT);
                  const uint64_t bd = make_smem_desc(b_src + j * (BK * Op::B_ROW_BYTES) + k * Op::B_K_STEP_BYTES, Op::B_BOX_BYTES, Op::B_SBO_BYTES,
                                                     Op::B_DESC_LAYOUT);
                  umma_ss_pair<TF32 ? 1 : (F8 ? 2 : 0)>(d_tmem + (uint32_t)(j * NT), ad, bd, idesc, accumulate);
                  accumulate = 1;
                }
              }
            }
            umma_commit_pair(empty_bar(s));                // stage reusable in both blocks once these MMAs retire
          }
          const bool last_of_group = p.per_example || (e + ISSUERS >= nu);
          if (ok && last_of_group) umma_commit_pair(acc_full_bar(buf));   // accumulator complete, both blocks
        }
      }
      __syncwarp();
    }
  } else {
    // ------------------------------------------------------------ epilogue (both blocks)
    setmaxnreg_inc<Op::REGS_EPILOGUE>();
    const int q = warp & 3;                 // TMEM lane quadrant this warp may access
    const int h = (warp - 4) >> 2;          // column half of the tile
    constexpr bool KEEP_MEAN = MEAN == MEAN_REGS || MEAN == MEAN_REGS_SIGN || PHI == 0;     // running sum of G_b in registers
    constexpr int N_STAT = (PHI != 0 && !NORMS) ? COLS : 1;
    // HYBRID: of a thread's 96 columns the first 64 have their running sum of G_b in tensor memory (columns
    // HYB_COL0 + 64 h ..), the last 32 in registers
    constexpr int HYB_TMEM_COLS = 64, HYB_COL0 = 2 * 192;
    constexpr int N_MEAN = KEEP_MEAN ? COLS : (HYBRID ? COLS - HYB_TMEM_COLS : 1);
    float acc_stat[N_STAT], acc_mean[N_MEAN];
    // TRIPLE: sum_b (sign(G_b) + 1) of two neighbouring columns in one register, as unsigned 16-bit
    // halves (each at most 2 nb <= 65534, so a plain 32-bit add never carries from one half into the
    // other); sum_b sign = count - nb.  The third statistic costs 32 registers instead of 64.
    constexpr int N_CNT = TRIPLE ? COLS / 2 : 1;
    uint32_t acc_cnt[N_CNT];
#pragma unroll
    for (int j = 0; j < N_CNT; ++j) acc_cnt[j] = 0u;
#pragma unroll
    for (int j = 0; j < N_STAT; ++j) acc_stat[j] = 0.f;
#pragma unroll
    for (int j = 0; j < N_MEAN; ++j) acc_mean[j] = 0.f;
    bool ok = true;
    // per-example mode: one accumulator per example, in example order (example e -> issuer e&1).
    // plain mode: one accumulator per issuer that had work.
    const int n_acc = p.per_example ? nu : (nu >= ISSUERS ? ISSUERS : nu);
    const uint32_t lane_base = tmem_base + ((uint32_t)(q * 32) << 16);
    for (int a = 0; a < n_acc; ++a) {
      const int x = a % ISSUERS, grp = p.per_example ? (a / ISSUERS) : 0;
      const int buf = UNITS_PER_ISSUER * x + (grp % UNITS_PER_ISSUER);        // accumulator unit (GROUP buffers)
      const uint32_t acc_ph = (uint32_t)(grp / UNITS_PER_ISSUER) & 1u;
      // PHI == 3: this example's clipping coefficient c_b = min(1, C / sqrt(N_b)); the load is issued before
      // the wait for the accumulator, which hides its latency.  N_b = 0 (a zero gradient) gives 1.
      uint64_t coef2 = 0;
      if constexpr (PHI == 3) {
        const float nb2 = __ldg(p.sq_norms + b_begin + a);
        const float nrm = sqrtf(nb2);
        const float c = nrm > p.clip_norm ? p.clip_norm / nrm : 1.f;
        coef2 = f32x2_pack(c, c);
      }
      // every lane polls, but the warp acts on one answer: the tensor-memory loads below are warp-wide
      // instructions, so no lane may leave the loop alone when its own wait is the one that gives up
      if (!__all_sync(0xffffffffu, mbar_wait_bounded(acc_full_bar(buf), acc_ph, abort_flag, p.dev_status, TC_WAIT_ACC_FULL))) { ok = false; break; }
      tc_fence_after();
      const uint32_t taddr = lane_base + (uint32_t)(buf * GROUP * NT + h * COLS);
      if constexpr (MEAN == MEAN_TMEM) {
        // sum_b G_b lives in tensor-memory columns MEAN_COL0.. of the same lanes: read it with G_b,
        // add, write it back (the first example just writes G_b).
        const uint32_t maddr = lane_base + (uint32_t)(MEAN_COL0 + h * COLS);
#pragma unroll
        for (int c = 0; c < COLS / 16; ++c) {
          uint32_t r[16], m[16];
          if (a == 0) tmem_ld_32x32b_x16_wait(taddr + c * 16, r);
          else tmem_ld_32x32b_x16_pair_wait(taddr + c * 16, r, maddr + c * 16, m);
          if (c == COLS / 16 - 1) {
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(map_to_cta(acc_empty_bar(buf), 0));   // G_b read: the issuer may start the next example
          }
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const float g = __uint_as_float(r[j]);
            acc_stat[c * 16 + j] += (PHI == 2) ? sign_half(g) : phi_apply<PHI>(g);
            if (a != 0) r[j] = __float_as_uint(g + __uint_as_float(m[j]));
          }
          tmem_st_32x32b_x16(maddr + c * 16, r);
        }
        tmem_st_wait();
      } else if constexpr (HYBRID) {
        const uint32_t maddr = lane_base + (uint32_t)(HYB_COL0 + h * HYB_TMEM_COLS);
#pragma unroll
        for (int c = 0; c < COLS / 16; ++c) {
          constexpr int LAST = COLS / 16 - 1;
          const bool in_tmem = c * 16 < HYB_TMEM_COLS;           // compile-time after unrolling
          uint32_t r[16], m[16];
          if (in_tmem && a != 0) tmem_ld_32x32b_x16_pair_wait(taddr + c * 16, r, maddr + c * 16, m);
          else tmem_ld_32x32b_x16_wait(taddr + c * 16, r);
          if (c == LAST) {
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(map_to_cta(acc_empty_bar(buf), 0));   // G_b read: the issuer may start its next example
          }
#pragma unroll
          for (int j = 0; j < 16; j += 2) {
            const uint64_t g2 = f32x2_pack(__uint_as_float(r[j]), __uint_as_float(r[j + 1]));
            const uint64_t s2 = f32x2_fma(g2, g2, f32x2_pack(acc_stat[c * 16 + j], acc_stat[c * 16 + j + 1]));
            f32x2_unpack(s2, acc_stat[c * 16 + j], acc_stat[c * 16 + j + 1]);
            acc_cnt[(c * 16 + j) >> 1] += sign_plus_one_packed(g2);
            if (in_tmem) {
              if (a != 0) {
                const uint64_t m2 = f32x2_add(f32x2_pack(__uint_as_float(m[j]), __uint_as_float(m[j + 1])), g2);
                float lo, hi;
                f32x2_unpack(m2, lo, hi);
                r[j] = __float_as_uint(lo);
                r[j + 1] = __float_as_uint(hi);
              }
            } else {
              const int k = c * 16 + j - HYB_TMEM_COLS;
              const uint64_t m2 = f32x2_add(f32x2_pack(acc_mean[k], acc_mean[k + 1]), g2);
              f32x2_unpack(m2, acc_mean[k], acc_mean[k + 1]);
            }
          }
          if (in_tmem) tmem_st_32x32b_x16(maddr + c * 16, r);      // the first example just writes G_b
        }
        tmem_st_wait();
      } else if constexpr (NORMS) {
        // this thread's share of ||G_b||_F^2 (its row, its 128 columns; rows and columns outside the
        // matrix are exact zeros), then the warp's, then one atomic per warp and example
        uint64_t sa = f32x2_pack(0.f, 0.f), sb = sa;
#pragma unroll
        for (int c = 0; c < COLS / 32; ++c) {
          uint32_t r[32];
          tmem_ld_32x32b_x32_wait(taddr + c * 32, r);
          if (c == COLS / 32 - 1) {
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(map_to_cta(acc_empty_bar(buf), 0));
          }
#pragma unroll
          for (int j = 0; j < 32; j += 4) {
            const uint64_t g0 = f32x2_pack(__uint_as_float(r[j]), __uint_as_float(r[j + 1]));
            const uint64_t g1 = f32x2_pack(__uint_as_float(r[j + 2]), __uint_as_float(r[j + 3]));
            sa = f32x2_fma(g0, g0, sa);
            sb = f32x2_fma(g1, g1, sb);
          }
        }
        float s0, s1;
        f32x2_unpack(f32x2_add(sa, sb), s0, s1);
        float s = s0 + s1;
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) s += __shfl_xor_sync(0xffffffffu, s, d);
        if (lane == 0) atomicAdd(p.out_norms + b_begin + a, s);
      } else {
        // CH columns per tensor-memory read: 32, or 16 where the running sums leave few registers (NT = 192; the three
        // statistics on the 256 x 128 tile, whose 160 registers of sums leave room for two reads of 16 in flight, not 32)
        constexpr int CH = (NT == 192 || TRIPLE) ? 16 : 32;
        constexpr int NCH = COLS / CH;                // reads per example
        // grouped examples: the unit's accumulators one after the other; the unit is released after the last read
        const int in_unit = (GROUP > 1) ? min(GROUP, nb - GROUP * a) : 1;
        // phi and the running sums for one read of CH columns (chunk c of this thread's COLS columns)
        auto fold = [&](const uint32_t (&r)[CH], int c) {
          if constexpr (PHI == 2) {
            // the running sum holds sum_b (sign(G_b) + 1) / 2 until the write-out turns it into sum_b sign(G_b)
#pragma unroll
            for (int j = 0; j < CH; j += 2) {
              const uint64_t g2 = f32x2_pack(__uint_as_float(r[j]), __uint_as_float(r[j + 1]));
              if (KEEP_MEAN) {
                const uint64_t m2 = f32x2_add(f32x2_pack(acc_mean[c * CH + j], acc_mean[c * CH + j + 1]), g2);
                f32x2_unpack(m2, acc_mean[c * CH + j], acc_mean[c * CH + j + 1]);
              }
              const uint64_t s2 = f32x2_add(f32x2_pack(acc_stat[c * CH + j], acc_stat[c * CH + j + 1]), sign_half2(g2));
              f32x2_unpack(s2, acc_stat[c * CH + j], acc_stat[c * CH + j + 1]);
            }
          } else {
            // two columns per instruction: packed fp32 add for sum_b G_b, packed fma for sum_b G_b^2
#pragma unroll
            for (int j = 0; j < CH; j += 2) {
              const uint64_t g2 = f32x2_pack(__uint_as_float(r[j]), __uint_as_float(r[j + 1]));
              if (KEEP_MEAN) {
                const uint64_t m2 = f32x2_add(f32x2_pack(acc_mean[c * CH + j], acc_mean[c * CH + j + 1]), g2);
                f32x2_unpack(m2, acc_mean[c * CH + j], acc_mean[c * CH + j + 1]);
              }
              if (PHI == 1 || PHI == 3) {
                const uint64_t s2 = f32x2_fma(g2, PHI == 1 ? g2 : coef2, f32x2_pack(acc_stat[c * CH + j], acc_stat[c * CH + j + 1]));
                f32x2_unpack(s2, acc_stat[c * CH + j], acc_stat[c * CH + j + 1]);
              }
              if (TRIPLE) {
                acc_cnt[(c * CH + j) >> 1] += sign_plus_one_packed(g2);
              }
            }
          }
        };
        auto release_unit = [&]() {
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(map_to_cta(acc_empty_bar(buf), 0));   // buffer(s) free for the issuer's next example(s)
        };
        // Where the registers allow two reads in flight (running sums of at most 128 floats beside two 32-column
        // reads; the three statistics' 160 registers beside two 16-column reads), the reads are software-pipelined:
        // read k+1 is issued before the arithmetic on read k, so only the first read of a unit exposes the
        // tensor-memory latency.  That latency, paid twice per example, was a third of the two-sum epilogue's time
        // per example, which is what bounds short sequences (the three-statistic epilogue, bound by its instruction
        // count, gains 2-3 %).
        constexpr bool PIPELINED = (CH == 32 && PHI != 3) || (TRIPLE && NT == 128);
        if constexpr (PIPELINED) {
          constexpr int TOTAL = GROUP * NCH;          // reads per unit when every example of the group exists
          const int n_reads = in_unit * NCH;
          uint32_t ra[CH], rb[CH];
          tmem_ld_issue(taddr, ra);
#pragma unroll
          for (int k = 0; k < TOTAL; ++k) {
            if (GROUP > 1 && k >= n_reads) break;
            if (k & 1) tmem_ld_wait_for(rb); else tmem_ld_wait_for(ra);
            if (k + 1 < n_reads) {
              const uint32_t next = taddr + (uint32_t)(((k + 1) / NCH) * NT + ((k + 1) % NCH) * CH);
              if (k & 1) tmem_ld_issue(next, ra); else tmem_ld_issue(next, rb);
            } else {
              release_unit();
            }
            if (k & 1) fold(rb, k % NCH); else fold(ra, k % NCH);
          }
        } else {
#pragma unroll
          for (int ju = 0; ju < GROUP; ++ju) {
            if (GROUP > 1 && ju >= in_unit) break;
            const uint32_t taddr_j = taddr + (uint32_t)(ju * NT);
#pragma unroll
            for (int c = 0; c < NCH; ++c) {
              uint32_t r[CH];
              if constexpr (CH == 32) tmem_ld_32x32b_x32_wait(taddr_j + c * CH, r);
              else tmem_ld_32x32b_x16_wait(taddr_j + c * CH, r);
              if (c == NCH - 1 && ju == in_unit - 1) release_unit();
              fold(r, c);
            }
          }
        }
      }
    }
    // Final write-out.  By now every MMA of this block has completed (the last accumulator was
    // committed after them), so the operand ring is free: each warp stages its 32-row x COLS-column
    // piece of an output there, 32 columns (one 128-byte-swizzled 4 KiB panel) at a time, and one lane
    // hands the panels to TMA, which stores them (or, with a split batch, adds them) and drops
    // whatever lies outside the matrix.  The tensor-memory loads are warp-wide instructions: the
    // condition around them is made uniform over the warp.
    ok = __all_sync(0xffffffffu, ok);
    if constexpr (PHI == 2) {
      // sum_b (sign(G_b) + 1) / 2  ->  sum_b sign(G_b)
      const float nbf = (float)nb;
#pragma unroll
      for (int j = 0; j < N_STAT; ++j) acc_stat[j] = fmaf(2.f, acc_stat[j], -nbf);
    }
    constexpr int PANELS = COLS / 32;
    int tile_m, tile_n;
    tc_tile_of_block(p, rank, tile_m, tile_n);
    // each epilogue warp stages in its own eighth of the operand ring: 6 panels of 4 KiB (7 at NT = 192)
    constexpr int WARP_PANELS = (STAGES * STAGE_BYTES / 8) / 4096;
    static_assert(WARP_PANELS >= PANELS, "an epilogue warp stages one output at a time");
    static_assert(OPT != OPT_ADAM || WARP_PANELS >= 2 * PANELS, "the fused Adam update reads both staged sums");
    const uint32_t stage_base = smem_base + (uint32_t)(warp - 4) * (uint32_t)(WARP_PANELS * 4096);
    const int row0 = tile_m * TC_TILE_M + q * 32;
    const int col0 = tile_n * NT + h * COLS;
    // fused update on the unsplit schedule: the sums are staged even when the caller does not want them written
    const bool stage_for_update = OPT != OPT_NONE && p.nsplit == 1;
    if (ok && n_acc > 0) {
      auto put_panel = [&](uint32_t panel_addr, const float* v) {      // v: this lane's 32 consecutive columns
        uint8_t* dst = smem_gen + (panel_addr - smem_base) + lane * 128;
#pragma unroll
        for (int k = 0; k < 8; ++k)
          *reinterpret_cast<float4*>(dst + ((k ^ (lane & 7)) << 4)) = make_float4(v[4 * k], v[4 * k + 1], v[4 * k + 2], v[4 * k + 3]);
      };
      auto send = [&](const CUtensorMap* tm, uint32_t first_panel) {
        fence_async_smem();
        __syncwarp();
        if (lane == 0 && row0 < p.d_out) {
          if (p.nsplit > 1 && !p.accumulate) griddep_wait();       // the kernel that zeroes the outputs may still be running
          for (int c = 0; c < PANELS; ++c) {
            if (col0 + c * 32 < p.d_in) {
              if (p.nsplit == 1 && !p.accumulate) tma_store_2d<false>(tm, first_panel + c * 4096, col0 + c * 32, row0);
              else tma_store_2d<true>(tm, first_panel + c * 4096, col0 + c * 32, row0);
            }
          }
          bulk_commit_group();
        }
      };
      // sum_b phi(G_b), or the plain contraction when PHI == 0
      if (p.out_stat || stage_for_update) {
#pragma unroll
        for (int c = 0; c < PANELS; ++c) put_panel(stage_base + c * 4096, (PHI != 0) ? &acc_stat[c * 32] : &acc_mean[c * 32]);
        if (p.out_stat) send(&tmap_stat, stage_base);
      }
      // sum_b G_b
      if ((p.out_mean || (stage_for_update && OPT == OPT_ADAM)) && (KEEP_MEAN || MEAN == MEAN_TMEM || HYBRID)) {
        uint32_t first = stage_base + PANELS * 4096;          // MEAN_REGS / PHI == 0: second half of the warp's 16 KiB
        if constexpr (HYBRID) {
          // two panels from tensor memory, the third from registers; staged behind the statistic's three panels
          const uint32_t maddr = lane_base + (uint32_t)(HYB_COL0 + h * HYB_TMEM_COLS);
#pragma unroll
          for (int c = 0; c < HYB_TMEM_COLS / 32; ++c) {
            uint32_t m[32];
            tmem_ld_32x32b_x32_wait(maddr + c * 32, m);
            put_panel(first + c * 4096, reinterpret_cast<const float*>(m));
          }
          put_panel(first + (HYB_TMEM_COLS / 32) * 4096, &acc_mean[0]);
        } else if constexpr (MEAN == MEAN_TMEM) {
          // the panels are needed again: wait until TMA has read the first output out of them
          if (lane == 0) bulk_wait_read_all();
          __syncwarp();
          first = stage_base;
          const uint32_t maddr = lane_base + (uint32_t)(MEAN_COL0 + h * COLS);
#pragma unroll
          for (int c = 0; c < PANELS; ++c) {
            uint32_t m[32];
            tmem_ld_32x32b_x32_wait(maddr + c * 32, m);
            put_panel(first + c * 4096, reinterpret_cast<const float*>(m));
          }
        } else if constexpr (KEEP_MEAN) {
          if constexpr (PANELS * 2 > WARP_PANELS) {           // PHI == 0 at NT = 256: one output only ever
            if (lane == 0) bulk_wait_read_all();
            __syncwarp();
            first = stage_base;
          }
#pragma unroll
          for (int c = 0; c < PANELS; ++c) put_panel(first + c * 4096, &acc_mean[c * 32]);
        }
        if (p.out_mean) send(&tmap_mean, first);
      }
      if constexpr (TRIPLE) {
        // sum_b sign(G_b): the warp's staging area is in use, so wait until TMA has read it
        if (p.out_sign) {
          if (lane == 0) bulk_wait_read_all();
          __syncwarp();
          const float nbf = (float)nb;
#pragma unroll
          for (int c = 0; c < PANELS; ++c) {
            float v[32];
#pragma unroll
            for (int j = 0; j < 32; ++j) v[j] = (float)((acc_cnt[(c * 32 + j) >> 1] >> (16 * (j & 1))) & 0xFFFFu) - nbf;
            put_panel(stage_base + c * 4096, v);
          }
          send(&tmap_sign, stage_base);
        }
      }
      if (lane == 0) bulk_wait_read_all();       // shared memory must outlive TMA's reads
    }
    __syncwarp();
    if constexpr (OPT != OPT_NONE) {
      // The parameter update, by the block that holds (unsplit batch) or has just completed (split batch)
      // the tile's sums over the whole batch.  Split batch: every block adds its partial tile to the
      // outputs, waits until those adds have been performed, and takes a ticket from the tile's counter;
      // the block that draws the last ticket reads the finished sums back and applies the update.  A block
      // that gave up on a wait marks the counter so that nobody updates the parameters from incomplete sums.
      bool apply = ok && n_acc > 0;
      if (p.nsplit > 1) {
        if (lane == 0) { bulk_wait_all(); __threadfence(); }
        __syncwarp();
        named_bar_sync(1, 256);                   // the eight epilogue warps; executed by all of them whatever `ok` says
        volatile int* last_flag = reinterpret_cast<volatile int*>(tail + 12);
        if (warp == 4 && lane == 0) {
          griddep_wait();                         // the counters are zeroed by the kernel that zeroes the outputs
          const unsigned int inc = 1u + (*abort_flag ? 0x10000u : 0u);
          const unsigned int now = atomicAdd(o.tile_counters + blockIdx.x, inc) + inc;
          int last = 0;
          if ((now & 0xffffu) == (unsigned int)p.nsplit) {
            last = (now >> 16) ? 0 : 1;
            atomicExch(o.tile_counters + blockIdx.x, 0u);
          }
          *last_flag = last;
        }
        named_bar_sync(1, 256);
        apply = (*last_flag != 0);
        if (apply) __threadfence();
      }
      if (apply) {
        const bool from_smem = p.nsplit == 1;
        const uint8_t* stat_panels = from_smem ? smem_gen + (stage_base - smem_base) : nullptr;
        fused_update_piece<OPT, PANELS>(o, p, row0, col0, lane, stat_panels, stat_panels ? stat_panels + PANELS * 4096 : nullptr);
      }
      __syncwarp();
    }
  }

  // ---------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    // A wait gave up.  Loads this block issued may still be landing in its shared memory: give them
    // time (bounded) before the block exits and its shared memory is handed to another block.
    const long long t0 = clock64();
    while (clock64() - t0 < (1ll << 22)) __nanosleep(1000);
  }
  // Neither block may leave while its peer can still arrive on its barriers or read its shared memory.
  __syncwarp();
  cluster_sync_all();
  if (warp == 2) { tc_fence_after(); tmem_dealloc_pair(tmem_base, TC_TMEM_COLS); }
}

}  // namespace pe
