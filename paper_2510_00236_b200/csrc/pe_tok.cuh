// Tensor-core kernel for the per-token second moment (Section 2.3, the "per-token" alternative):
//     S'[o,i] = sum_r dY[r,o]^2 * X[r,i]^2        over the B*T rows r,
// a plain contraction of the SQUARED operands.  Nothing is staged in global memory: the bf16 tiles
// arrive by TMA, the eight warps that later write the result out first square them on the fly
// (bf16^2 is exact in fp32), round to tf32 and lay them out in shared memory the way the tf32 MMA
// wants them, and the pair-wide tcgen05 MMAs (cta_group::2, M = 256, N = 256, kind::tf32) accumulate
// in tensor memory.  tf32 keeps 11 significant bits of each square (bf16 would keep 8), so every
// entry of the result is within about 1e-3 of the exact sum, all terms being non-negative.
// Every stage crosses shared memory four times (TMA in, converter out and back in, MMA out: 96 KiB
// per 32 rows and block), which is what bounds this kernel; it runs at about the speed of the
// two-pass variant on large layers and faster on small ones, with a third of the HBM traffic.
//
// Work unit: a CTA pair owns a 256 x 256 tile of the [d_out, d_in] output and a contiguous range of
// 32-row chunks of the B*T rows (gridDim.z slices; partial sums are added by TMA reduce).
//
// Shared memory per block: 4 "raw" stages of 16 KiB (bf16: 128 rows of dY^T as two 64-feature boxes,
// this block's 128 rows of X^T as two more; 128-byte swizzle with 16-byte chunks, as TMA writes it)
// and 4 "cooked" stages of 32 KiB (fp32 holding tf32 values: eight 32-feature boxes; 128-byte swizzle
// with 32-byte chunks, the only MN-major form of the tf32 MMA).
//
// Warps (20 per block): 0 = TMA producer of the dY boxes (also posts the stage's byte count), 2 = TMEM
// allocator, then TMA producer of the X boxes, 1 = MMA issuer (leader block only), 4..19 = converters
// (sixteen warps: the conversion is a stream of dependent shared-memory round trips, and eight warps
// only reached 1.4 instructions per clock of the SM's 4), of which 4..11 then write the result out.
// Barriers: raw_full[s] / raw_empty[s] are local to each block (its own TMA, its own converters);
// cooked_full[c] lives in the leader and collects the converter warps of both blocks (four per block
// and stage: the sixteen warps work as four groups, group g on the stages n = g mod 4, i.e. always
// on ring slot g); cooked_empty[c] and acc_full are signalled in both blocks by one multicast commit.
#pragma once
#include "pe_tc.cuh"

namespace pe {

constexpr int TOK_NT = 256;                       // d_in columns per pair tile
constexpr int TOK_BK = 32;                        // rows (tokens) per stage
constexpr int TOK_BOX_BYTES = 128 * TOK_BK;       // 4 KiB: one box, raw (64 bf16 wide) or cooked (32 fp32 wide)
constexpr int TOK_RAW_BOXES = 4;                  // per block and stage: 2 of dY^T, 2 of X^T
constexpr int TOK_RAW_STAGE = TOK_RAW_BOXES * TOK_BOX_BYTES;         // 16 KiB
constexpr int TOK_COOKED_STAGE = 2 * TOK_RAW_STAGE;                  // 32 KiB: A 16 KiB then B 16 KiB
constexpr int TOK_RAW_STAGES = 4, TOK_COOKED_STAGES = 4;
constexpr int TOK_RING_BYTES = TOK_RAW_STAGES * TOK_RAW_STAGE + TOK_COOKED_STAGES * TOK_COOKED_STAGE;   // 192 KiB
constexpr int TOK_SMEM_BYTES = TOK_RING_BYTES + TC_BAR_BYTES + 1024;
constexpr int TOK_MMA_K = 8;                      // rows per tf32 MMA
constexpr int TOK_CONV_WARPS = 16;                // converter warps per block, in groups of four
constexpr int TOK_CONV_GROUPS = TOK_CONV_WARPS / 4;
constexpr int TOK_THREADS = 128 + 32 * TOK_CONV_WARPS;          // 640: 96 registers per thread at one block per SM
static_assert(TOK_CONV_GROUPS == TOK_RAW_STAGES, "converter group g owns ring slot g");
enum : int { TOK_WAIT_RAW_EMPTY = 11, TOK_WAIT_RAW_FULL = 12, TOK_WAIT_COOKED_EMPTY = 13, TOK_WAIT_COOKED_FULL = 14, TOK_WAIT_ACC = 15 };

struct TokParams {
  long long rows;      // B * T
  int d_in, d_out;
  int pairs_m, tiles_n, band;   // tile grid and tile order, as in TcParams
  int nsplit;          // slices of the row range (gridDim.z); > 1 => output pre-zeroed, partial sums added
  unsigned int* dev_status;
};

// Two bf16 values (one 32-bit word) -> their squares rounded to tf32 (10 explicit mantissa bits,
// round to nearest even), as two fp32 bit patterns in one 64-bit register.  A bf16 is the upper half
// of an fp32 and its square is exact in fp32, so the rounding is the only error: at most 2^-11
// relative per operand, and unbiased.  The rounding is Veltkamp's split: with s = RN(8193 x),
// s - (s - x) is x rounded to 24 - 13 = 11 significant bits (nearest even; it equals the integer
// formula (u + 0xFFF + ((u >> 13) & 1)) & ~0x1FFF on every square of an 8-bit significand, where exact
// ties are frequent and rounding them upward would bias the sums by about 1e-4).  Four packed fp32
// instructions per pair.  s is formed as fma(x, 8192, x): the assembler was seen to merge a separate
// multiply by 8193 into the following subtraction, which skips the rounding of s that the split
// relies on; a multiply by a power of two is exact, so this form gives the same s however it is merged.
// Squares above 2^128 / 8193 come out as NaN instead of infinity.
__device__ __forceinline__ uint64_t tok_square_tf32_pair(uint32_t two_bf16) {
  const uint64_t v = sm100::f32x2_pack(__uint_as_float(two_bf16 << 16), __uint_as_float(two_bf16 & 0xFFFF0000u));
  const uint64_t x = sm100::f32x2_mul(v, v);
  const uint64_t s = sm100::f32x2_fma(x, sm100::f32x2_pack(8192.f, 8192.f), x);
  return sm100::f32x2_sub(s, sm100::f32x2_sub(s, x));
}

// gridDim = (2 * pairs_m * tiles_n, 1, nsplit); blockIdx.x = 2 * (pair index in the tile order) + rank in pair.
// tmap_x / tmap_dy: [rows, d] bf16 viewed as (d, rows), box 64 x 32, 128-byte swizzle.
// tmap_out: [d_out, d_in] fp32 viewed as (d_in, d_out), box 32 x 32, 128-byte swizzle.
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(TOK_THREADS, 1)
tok_sqstats_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_dy,
                   const __grid_constant__ CUtensorMap tmap_out, TokParams p) {
  using namespace sm100;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t cooked_base = smem_base + TOK_RAW_STAGES * TOK_RAW_STAGE;
  const uint32_t bar_base = smem_base + TOK_RING_BYTES;
  auto raw_full = [&](int s) { return bar_base + 8u * s; };
  auto raw_empty = [&](int s) { return bar_base + 8u * (TOK_RAW_STAGES + s); };
  auto cooked_full = [&](int c) { return bar_base + 8u * (2 * TOK_RAW_STAGES + c); };
  auto cooked_empty = [&](int c) { return bar_base + 8u * (2 * TOK_RAW_STAGES + TOK_COOKED_STAGES + c); };
  const uint32_t acc_full = bar_base + 8u * (2 * TOK_RAW_STAGES + 2 * TOK_COOKED_STAGES);
  uint8_t* tail = smem_gen + TOK_RING_BYTES + 8 * (2 * TOK_RAW_STAGES + 2 * TOK_COOKED_STAGES + 1);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(tail);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tail + 8);
  static_assert(8 * (2 * TOK_RAW_STAGES + 2 * TOK_COOKED_STAGES + 1) + 16 <= TC_BAR_BYTES, "barrier area too small");

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();          // 0 = leader of the pair
  int tile_m, tile_n;                               // 128-row tile of d_out, 256-column tile of d_in (banded tile order)
  {
    const int pair_id = blockIdx.x >> 1;
    const int per_band = p.band * p.tiles_n;
    const int band = pair_id / per_band, r = pair_id - band * per_band;
    const int rows_in_band = min(p.band, p.pairs_m - band * p.band);
    tile_n = r / rows_in_band;
    tile_m = 2 * (band * p.band + (r - tile_n * rows_in_band)) + (int)rank;
  }
  const long long n_chunks = (p.rows + TOK_BK - 1) / TOK_BK;
  const long long c_begin = n_chunks * blockIdx.z / p.nsplit, c_end = n_chunks * (blockIdx.z + 1) / p.nsplit;

  if (threadIdx.x == 0) {
    for (int s = 0; s < TOK_RAW_STAGES; ++s) { mbar_init(raw_full(s), 1); mbar_init(raw_empty(s), 4); }
    for (int c = 0; c < TOK_COOKED_STAGES; ++c) { mbar_init(cooked_full(c), 8); mbar_init(cooked_empty(c), 1); }
    mbar_init(acc_full, 1);
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 2) { tmem_alloc_pair(smem_u32(const_cast<uint32_t*>(tmem_slot)), TC_TMEM_COLS); tmem_relinquish_pair(); }
  tc_fence_before();
  cluster_sync_all();          // barriers of both blocks initialised before any remote arrival
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp < 4) {
    if (warp == 0 || warp == 2) {
      // ---------------------------------------------------------- TMA producers (each block for itself)
      if (lane == 0) {
        const bool is_a = (warp == 0);
        const CUtensorMap* tmap = is_a ? &tmap_dy : &tmap_x;
        const int c0 = is_a ? tile_m * TC_TILE_M : tile_n * TOK_NT + (int)rank * (TOK_NT / 2);
        prefetch_tensormap(tmap);
        int s = 0; uint32_t ph = 0;
        for (long long ch = c_begin; ch < c_end; ++ch) {
          if (!mbar_wait_bounded(raw_empty(s), ph ^ 1u, abort_flag, p.dev_status, TOK_WAIT_RAW_EMPTY)) break;
          if (is_a) mbar_arrive_expect_tx(raw_full(s), TOK_RAW_STAGE);          // this block's four boxes
          const uint32_t dst = smem_base + s * TOK_RAW_STAGE + (is_a ? 0 : 2 * TOK_BOX_BYTES);
          tma_load_2d(dst, tmap, raw_full(s), c0, (int)(ch * TOK_BK));
          tma_load_2d(dst + TOK_BOX_BYTES, tmap, raw_full(s), c0 + 64, (int)(ch * TOK_BK));
          if (++s == TOK_RAW_STAGES) { s = 0; ph ^= 1u; }
        }
      }
      __syncwarp();
    } else if (rank == 0 && warp == 1) {
      // ---------------------------------------------------------- MMA issuer (leader block)
      if (lane == 0) {
        constexpr uint32_t idesc = make_idesc_mn_major(TC_PAIR_M, TOK_NT, true);
        int c = 0; uint32_t ph = 0;
        uint32_t accumulate = 0;
        bool ok = true;
        for (long long ch = c_begin; ch < c_end; ++ch) {
          if (!mbar_wait_bounded(cooked_full(c), ph, abort_flag, p.dev_status, TOK_WAIT_COOKED_FULL)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a_src = cooked_base + c * TOK_COOKED_STAGE;
          const uint32_t b_src = a_src + TOK_COOKED_STAGE / 2;
#pragma unroll
          for (int k = 0; k < TOK_BK / TOK_MMA_K; ++k) {       // rows past the end are zero: no need to skip them
            const uint64_t ad = make_smem_desc(a_src + k * TOK_MMA_K * 128, TOK_BOX_BYTES, 512u, 1u);
            const uint64_t bd = make_smem_desc(b_src + k * TOK_MMA_K * 128, TOK_BOX_BYTES, 512u, 1u);
            umma_ss_pair<1>(tmem_base, ad, bd, idesc, accumulate);
            accumulate = 1;
          }
          umma_commit_pair(cooked_empty(c));             // cooked stage reusable in both blocks once these MMAs retire
          if (++c == TOK_COOKED_STAGES) { c = 0; ph ^= 1u; }
        }
        if (ok) umma_commit_pair(acc_full);              // accumulator complete, both blocks
      }
      __syncwarp();
    }
  } else {
    // ------------------------------------------------------------ converters, then write-out (both blocks)
    // (no setmaxnreg here: 640 threads x 96 registers is all a converter needs)
    const int w = warp - 4;                 // 0..15
    bool ok = true;
    {
      // The sixteen warps work as four groups of four, group g on the stages n = g, g + 4, ... (ring slot g),
      // so that the groups' shared-memory round trips and barrier hand-offs overlap one another's arithmetic.
      const int grp = w >> 2, wl = w & 3;
      for (long long n = grp; n < c_end - c_begin; n += TOK_CONV_GROUPS) {
        const int s = (int)(n % TOK_RAW_STAGES);          // raw and cooked rings advance together (same depth)
        const uint32_t ph = (uint32_t)(n / TOK_RAW_STAGES) & 1u;
        // every lane polls, the warp acts on one answer (what follows contains warp-wide instructions)
        if (!__all_sync(0xffffffffu, mbar_wait_bounded(raw_full(s), ph, abort_flag, p.dev_status, TOK_WAIT_RAW_FULL))) { ok = false; break; }
        if (!__all_sync(0xffffffffu, mbar_wait_bounded(cooked_empty(s), ph ^ 1u, abort_flag, p.dev_status, TOK_WAIT_COOKED_EMPTY))) { ok = false; break; }
        const uint8_t* raw = smem_gen + s * TOK_RAW_STAGE;
        uint8_t* cooked = smem_gen + TOK_RAW_STAGES * TOK_RAW_STAGE + s * TOK_COOKED_STAGE;
        // A stage is 1024 16-byte chunks (4 boxes x 32 rows x 8 chunks of 8 features); chunk g of the
        // stage goes to lane g % 32 of warp (g / 32) % 4 of the group.  Eight neighbouring lanes read
        // one 128-byte row; its 64 features become two 128-byte rows of two neighbouring cooked boxes.
        // All eight loads first: raw and cooked stages live in the same shared array, so a load written
        // after a store would have to stay behind it and every iteration would pay the load latency.
        uint4 vin[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int g = (i * 4 + wl) * 32 + lane;
          const int box = g >> 8, t = (g >> 3) & 31, c = g & 7;
          vin[i] = *reinterpret_cast<const uint4*>(raw + box * TOK_BOX_BYTES + t * 128 + ((c ^ (t & 7)) << 4));
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int g = (i * 4 + wl) * 32 + lane;
          const int box = g >> 8, t = (g >> 3) & 31, c = g & 7;
          const uint4 v = vin[i];
          const uint64_t o0 = tok_square_tf32_pair(v.x), o1 = tok_square_tf32_pair(v.y);
          const uint64_t o2 = tok_square_tf32_pair(v.z), o3 = tok_square_tf32_pair(v.w);
          // Lanes with c >= 4 (the second of the two boxes) store their halves in the other order, so
          // that each store instruction of the warp touches all eight 16-byte bank groups, not four.
          uint8_t* dst = cooked + (2 * box + (c >> 2)) * TOK_BOX_BYTES + t * 128 + (((c & 3) ^ (t & 3)) << 5);
          const bool swap = (c & 4) != 0;
          *reinterpret_cast<ulonglong2*>(dst + (swap ? 16 : 0)) = swap ? make_ulonglong2(o2, o3) : make_ulonglong2(o0, o1);
          *reinterpret_cast<ulonglong2*>(dst + (swap ? 0 : 16)) = swap ? make_ulonglong2(o0, o1) : make_ulonglong2(o2, o3);
        }
        fence_async_smem();                 // the MMA reads these through the async proxy
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(raw_empty(s));                                  // this block's TMA may refill the raw stage
          mbar_arrive_cluster(map_to_cta(cooked_full(s), 0));         // one of 8 arrivals the issuer waits for
        }
      }
    }
    static_assert(TOK_RAW_STAGES == TOK_COOKED_STAGES && TOK_RAW_STAGES % 2 == 0, "the two rings advance together; each slot belongs to one converter group");
    ok = __all_sync(0xffffffffu, ok);
    if (ok && w < 8) ok = __all_sync(0xffffffffu, mbar_wait_bounded(acc_full, 0, abort_flag, p.dev_status, TOK_WAIT_ACC));
    ok = __all_sync(0xffffffffu, ok);
    if (ok && w < 8) {
      // Write-out as in the statistics kernel: 32 rows x 128 columns per warp, staged in the idle ring
      // as four 128-byte-swizzled 4 KiB panels, stored (or added, with a split row range) by TMA.
      tc_fence_after();
      const int q = warp & 3, h = w >> 2;
      const uint32_t lane_base = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(h * 128);
      const uint32_t stage_base = smem_base + (uint32_t)w * (4u * 4096u);
      const int row0 = tile_m * TC_TILE_M + q * 32, col0 = tile_n * TOK_NT + h * 128;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint32_t r[32];
        tmem_ld_32x32b_x32_wait(lane_base + c * 32, r);
        uint8_t* dst = smem_gen + (stage_base - smem_base) + c * 4096 + lane * 128;
#pragma unroll
        for (int k = 0; k < 8; ++k)
          *reinterpret_cast<uint4*>(dst + ((k ^ (lane & 7)) << 4)) = make_uint4(r[4 * k], r[4 * k + 1], r[4 * k + 2], r[4 * k + 3]);
      }
      fence_async_smem();
      __syncwarp();
      if (lane == 0 && row0 < p.d_out) {
        if (p.nsplit > 1) griddep_wait();         // the kernel that zeroes the output may still be running
        for (int c = 0; c < 4; ++c) {
          if (col0 + c * 32 < p.d_in) {
            if (p.nsplit == 1) tma_store_2d<false>(&tmap_out, stage_base + c * 4096, col0 + c * 32, row0);
            else tma_store_2d<true>(&tmap_out, stage_base + c * 4096, col0 + c * 32, row0);
          }
        }
        bulk_commit_group();
        bulk_wait_read_all();               // shared memory must outlive TMA's reads
      }
    }
    __syncwarp();
  }

  // ---------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    const long long t0 = clock64();
    while (clock64() - t0 < (1ll << 22)) __nanosleep(1000);
  }
  __syncwarp();
  cluster_sync_all();           // neither block leaves while its peer can still reach its barriers or shared memory
  if (warp == 2) { tc_fence_after(); tmem_dealloc_pair(tmem_base, TC_TMEM_COLS); }
}

}  // namespace pe
