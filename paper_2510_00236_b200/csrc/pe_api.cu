// C-ABI entry points of libpestats: argument validation, path selection, tensor-map creation and
// kernel launches.  Everything that computes runs in the CUDA kernels included below.
#include <algorithm>
#include <atomic>
#include <cstdint>
#include <cstdlib>
#include <cstring>
#include <cmath>
#include <mutex>
#include <vector>

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "../../include/pestats.h"
#include "pe_optim.cuh"
#include "pe_stage.cuh"
#include "pe_simt.cuh"
#include "pe_tc.cuh"
#include "pe_tok.cuh"

namespace pe {

__device__ unsigned int g_dev_status = 0;   // first device-side wait that gave up (0 = none)

static std::atomic<int> g_path{PE_PATH_AUTO};
static std::atomic<int> g_last_path{PE_PATH_AUTO};
static std::atomic<long long> g_launches{0};
static std::atomic<int> g_fused_mode{PE_FUSED_AUTO};
// Both outputs: from this sequence length on the running sum of G_b lives in tensor memory beside a
// 256-column accumulator (measured: wins or ties at T = 4096, loses 16 % at T = 2048, 17 % at T = 1024).
constexpr int TC_MEAN_TMEM_MIN_T = 4096;
// Both outputs, phi = square or sign: from this sequence length on the pair tile is 256 x 192 instead of
// 256 x 128 (measured: ties at T = 64 and 128, 3-21 % faster from T = 256 on, 17-25 % faster than the
// tensor-memory mean at T = 4096; 18-22 % slower at T = 32), unless d_in is so narrow that the wider
// tile's padding (columns up to the next multiple of 192) eats the gain.
constexpr int TC_WIDE_MIN_T = 64;
constexpr int TC_WIDE_MAX_PAD_PERCENT = 13;
// The three-statistic pass on the 256 x 192 tile keeps two thirds of sum_b G_b in tensor memory (a read, an add
// and a write per example): it needs longer sequences than the two-sum kernel to hide that epilogue (measured: 6-8 % faster
// than the 256 x 128 one-pass kernel at T = 512 and 1024, 10 % slower at T = 256).
constexpr int TC_WIDE_TRIPLE_MIN_T = 512;
constexpr int PHI_CLIP_SCALE = 3;   // internal phi of the clipped sum: c_b * G_b (not part of pe_phi_t)
constexpr int TC_BAND = 8;          // pair rows per band of the tile order (8 x 256 rows of d_out)

constexpr int MAX_DEVICES = 64;
struct DeviceInfo {
  std::atomic<int> state{0};     // 0 unknown, 1 ready, -1 failed
  int cc_major = 0, sm_count = 0;
  unsigned int* status_ptr = nullptr;
  bool tc_attr_set[32] = {};
  bool tok_attr_set = false;
};
static DeviceInfo g_dev[MAX_DEVICES];
static std::mutex g_dev_mutex;      // guards the lazily filled per-device state (first calls from several host threads)

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static std::atomic<EncodeTiledFn> g_encode{nullptr};

static pe_status_t device_info(DeviceInfo** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) { cudaGetLastError(); return PE_ERR_CUDA; }
  DeviceInfo& d = g_dev[dev];
  if (d.state.load(std::memory_order_acquire) == 0) {
    std::lock_guard<std::mutex> lock(g_dev_mutex);
    if (d.state.load(std::memory_order_relaxed) != 0) { *out = &d; return d.cc_major == 10 ? PE_OK : PE_ERR_ARCH; }
    int major = 0, sms = 0;
    void* sp = nullptr;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
      cudaGetLastError();
      return PE_ERR_CUDA;
    }
    d.cc_major = major;
    d.sm_count = sms;
    if (major == 10) {
      if (cudaGetSymbolAddress(&sp, g_dev_status) != cudaSuccess) { cudaGetLastError(); return PE_ERR_CUDA; }
      d.status_ptr = static_cast<unsigned int*>(sp);
    }
    d.state.store(1, std::memory_order_release);
  }
  *out = &d;
  return d.cc_major == 10 ? PE_OK : PE_ERR_ARCH;
}

static EncodeTiledFn encode_fn() {
  EncodeTiledFn f = g_encode.load();
  if (f) return f;
  void* sym = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) != cudaSuccess ||
      q != cudaDriverEntryPointSuccess || !sym) {
    cudaGetLastError();
    return nullptr;
  }
  f = reinterpret_cast<EncodeTiledFn>(sym);
  g_encode.store(f);
  return f;
}

static bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

static pe_status_t check_launch() {
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return PE_ERR_CUDA;
  g_launches.fetch_add(1);
  return PE_OK;
}

// [B, T, d] row-major (bf16, or fp32 read as tf32) viewed as a 3-D tensor (d, T, B); one box = 128
// bytes of features x one pipeline stage of tokens of one example, 128-byte swizzled (16-byte chunks for bf16, 32-byte
// chunks for fp32: the MN-major tf32 MMA accepts no other layout).  rows64: 64 bytes of features per box row with
// the 64-byte swizzle (X of the 256 x 192 tile).  Tokens past T and features past d read as zero.
static pe_status_t make_operand_map(CUtensorMap* m, const void* base, int B, int T, int d, bool f32, int box_feats, int box_tokens,
                                    bool rows64 = false, int box_examples = 1) {
  EncodeTiledFn enc = encode_fn();
  if (!enc) return PE_ERR_CUDA;
  const cuuint64_t es = f32 ? 4ull : 2ull;
  cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)T, (cuuint64_t)B};
  cuuint64_t strides[2] = {(cuuint64_t)d * es, (cuuint64_t)T * (cuuint64_t)d * es};
  cuuint32_t box[3] = {(cuuint32_t)box_feats, (cuuint32_t)box_tokens, (cuuint32_t)box_examples};
  cuuint32_t estr[3] = {1u, 1u, 1u};
  CUresult r = enc(m, f32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                   CU_TENSOR_MAP_INTERLEAVE_NONE,
                   f32 ? CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B : (rows64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B),
                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? PE_OK : PE_ERR_CUDA;
}

// The tensor-core per-token statistic rounds each squared operand to 11 significant bits (tf32 in the
// one-kernel form, column-scaled IEEE half in the two-pass form): relative error at most 2^-11 per
// factor, so at most ~1e-3 on any entry, all terms being non-negative.  Tiny problems
// gain nothing from the tensor cores and take the SIMT kernel (fp32 squares).
constexpr long long TOKEN_TC_MIN_ROWS = 256;

// [d_out, d_in] fp32 output viewed as a 2-D tensor (d_in, d_out); one box = 32 columns (128 bytes,
// 128-byte swizzled) x 32 rows, the piece one epilogue warp stages at a time.
static pe_status_t make_output_map(CUtensorMap* m, float* base, int d_in, int d_out) {
  EncodeTiledFn enc = encode_fn();
  if (!enc) return PE_ERR_CUDA;
  cuuint64_t dims[2] = {(cuuint64_t)d_in, (cuuint64_t)d_out};
  cuuint64_t strides[1] = {(cuuint64_t)d_in * 4ull};
  cuuint32_t box[2] = {32u, 32u};
  cuuint32_t estr[2] = {1u, 1u};
  CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                   CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? PE_OK : PE_ERR_CUDA;
}

static bool tc_shape_ok(int B, int T, int d_in, int d_out);
static bool token_tc_ok(int B, int T, int d_in, int d_out) {
  return tc_shape_ok(B, T, d_in, d_out) && (long long)B * T >= TOKEN_TC_MIN_ROWS;
}

static bool tc_shape_ok(int B, int T, int d_in, int d_out) {
  if (B < 1 || T < 1) return false;
  if ((d_in % 8) || (d_out % 8)) return false;                        // 16-byte row pitch for TMA
  if ((long long)T * (d_in > d_out ? d_in : d_out) * 4ll >= (1ll << 40)) return false;   // TMA stride limit (fp32 staging included)
  return true;
}

// Batch slices per tile: minimise (waves of thread blocks) x (examples per slice) plus a flush term.
static int choose_nsplit(long long tiles, int B, int T, int slots, int max_split) {
  int best = 1;
  double best_cost = 1e300;
  int tt = T < 32 ? 32 : T;
  for (int ns = 1; ns <= max_split && ns <= B; ++ns) {
    long long waves = (tiles * ns + slots - 1) / slots;
    long long per = ((long long)B + ns - 1) / ns;
    double cost = (double)waves * ((double)per * tt + (ns > 1 ? 512.0 : 128.0));
    if (cost < best_cost * 0.999) { best_cost = cost; best = ns; }
  }
  return best;
}

// Pair rows per band of the tile order (tc_tile_of_block).  Thread blocks start in the order of their index, `slots`
// CTA pairs at a time, the batch slices one after the other; such a wave streams, for every example of its slice, the dY
// panels of the pair rows and the X panels of the column tiles it touches, and between two waves the batch has passed
// through L2.  So the bytes a launch reads from HBM follow the sum over waves of (pair rows x 256 + column tiles x nt):
// measured on the 8192 x 2048 layer with 256 sequences of 1024 tokens, 18.5 GB with bands of 8 pair rows, which the
// waves cut unevenly there, against 13.0 GB with bands of 1 (the model gives 2.54 and 1.88 times the operands' size).
// The candidates are walked on the host; the previous default is kept unless another band saves more than 3 %.
static int choose_band(int pairs_m, int tiles_n, int nt, int nsplit, int slots) {
  const int fallback = pairs_m < TC_BAND ? pairs_m : TC_BAND;
  const long long total = (long long)pairs_m * tiles_n;
  if (slots < 1 || pairs_m <= 1 || total * nsplit <= slots) return fallback;       // one wave: the order does not matter
  struct Key { int pairs_m, tiles_n, nt, nsplit, slots, band; };
  thread_local Key cache[16] = {};
  thread_local int cache_next = 0;
  for (const Key& k : cache)
    if (k.band > 0 && k.pairs_m == pairs_m && k.tiles_n == tiles_n && k.nt == nt && k.nsplit == nsplit && k.slots == slots) return k.band;
  // units walked per candidate: the whole launch, or its first 16 Ki thread-block pairs (over 200 waves; the pattern repeats)
  const long long units = total * nsplit < (1ll << 14) ? total * nsplit : (1ll << 14);
  thread_local std::vector<int> row_seen, col_seen;
  row_seen.assign((size_t)pairs_m, -1);
  col_seen.assign((size_t)tiles_n, -1);
  static const int candidates[] = {TC_BAND, 1, 2, 3, 4, 6, 12, 16};
  double best_cost = 0.0, fallback_cost = 0.0;
  int best = fallback;
  for (int band : candidates) {
    if (band > pairs_m) band = pairs_m;
    std::fill(row_seen.begin(), row_seen.end(), -1);
    std::fill(col_seen.begin(), col_seen.end(), -1);
    const long long per_band = (long long)band * tiles_n;
    double cost = 0.0;
    for (long long u = 0; u < units; ++u) {
      const int wave = (int)(u / slots);
      const long long pair_id = u % total;
      const int b = (int)(pair_id / per_band);
      const int r = (int)(pair_id - (long long)b * per_band);
      const int rows = band < pairs_m - b * band ? band : pairs_m - b * band;
      const int tile_n = r / rows, pair_row = b * band + (r - tile_n * rows);
      if (row_seen[pair_row] != wave) { row_seen[pair_row] = wave; cost += TC_PAIR_M; }
      if (col_seen[tile_n] != wave) { col_seen[tile_n] = wave; cost += nt; }
    }
    if (band == fallback) fallback_cost = cost;
    if (best_cost == 0.0 || cost < best_cost) { best_cost = cost; best = band; }
  }
  if (fallback_cost > 0.0 && best_cost > 0.97 * fallback_cost) best = fallback;
  cache[cache_next] = Key{pairs_m, tiles_n, nt, nsplit, slots, best};
  cache_next = (cache_next + 1) % 16;
  return best;
}

static pe_status_t zero_outputs(float* a, float* b, size_t bytes, cudaStream_t st) {
  if (a && cudaMemsetAsync(a, 0, bytes, st) != cudaSuccess) { cudaGetLastError(); return PE_ERR_CUDA; }
  if (b && cudaMemsetAsync(b, 0, bytes, st) != cudaSuccess) { cudaGetLastError(); return PE_ERR_CUDA; }
  return PE_OK;
}

// Zeroes up to three [d_out, d_in] outputs with a kernel that lets its successor start at once.
static pe_status_t zero_for_split(DeviceInfo* di, float* a, float* b, size_t n, cudaStream_t st, float* c = nullptr,
                                  unsigned int* counters = nullptr, int n_counters = 0) {
  float* first = a ? a : b;
  float* second = a ? b : nullptr;
  if (!first) return PE_OK;
  const long long n4 = (long long)(n / 4);          // d_in % 8 == 0 on this path
  long long blocks = (n4 + 255) / 256;
  if (blocks > di->sm_count) blocks = di->sm_count;   // few blocks: the dependent kernel needs the SMs
  zero_outputs_kernel<<<(int)(blocks < 1 ? 1 : blocks), 256, 0, st>>>(reinterpret_cast<float4*>(first), reinterpret_cast<float4*>(second),
                                                                            reinterpret_cast<float4*>(c), n4, counters, n_counters);
  return check_launch();
}

// Launches `kernel`; as a programmatic dependent of the zeroing kernel when the batch is split.
template <typename Kernel, typename... Args>
static pe_status_t launch_pair_kernel_t(Kernel kernel, dim3 grid, int threads, int smem, cudaStream_t st, bool after_zeroing, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = dim3(threads); cfg.dynamicSmemBytes = (size_t)smem; cfg.stream = st;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr; cfg.numAttrs = after_zeroing ? 1 : 0;
  if (cudaLaunchKernelEx(&cfg, kernel, args...) != cudaSuccess) { cudaGetLastError(); return PE_ERR_CUDA; }
  return check_launch();
}
template <typename Kernel, typename... Args>
static pe_status_t launch_pair_kernel(Kernel kernel, dim3 grid, int smem, cudaStream_t st, bool after_zeroing, Args... args) {
  return launch_pair_kernel_t(kernel, grid, TC_THREADS, smem, st, after_zeroing, args...);
}

// mxt, myt: the maps of the zero-padded tail groups of a packed batch (RAGGED); any valid map otherwise.
template <int PHI, bool TF32, int NT, int MEAN, int BKT = tc_default_bk(TF32, NT), bool RAGGED = false, int OPT = OPT_NONE, bool F8 = false>
static pe_status_t launch_tc_inst(DeviceInfo* di, int slot, const CUtensorMap& mx, const CUtensorMap& my, const CUtensorMap& mm,
                                  const CUtensorMap& ms, const CUtensorMap& msgn, const TcParams& p, dim3 grid, cudaStream_t st,
                                  const CUtensorMap* mxt = nullptr, const CUtensorMap* myt = nullptr, const FusedOpt* opt = nullptr) {
  const bool after_zeroing = p.nsplit > 1 && !p.accumulate;
  constexpr int smem = TcOperand<TF32, NT, BKT, F8>::SMEM_BYTES;
  {
    std::lock_guard<std::mutex> lock(g_dev_mutex);
    if (!di->tc_attr_set[slot]) {
      if (cudaFuncSetAttribute(tc_stats_kernel<PHI, TF32, NT, MEAN, BKT, RAGGED, OPT, F8>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) {
        cudaGetLastError();
        return PE_ERR_CUDA;
      }
      di->tc_attr_set[slot] = true;
    }
  }
  return launch_pair_kernel(tc_stats_kernel<PHI, TF32, NT, MEAN, BKT, RAGGED, OPT, F8>, grid, smem, st, after_zeroing, mx, my, mm, ms, msgn,
                            mxt ? *mxt : mx, myt ? *myt : my, p, opt ? *opt : FusedOpt{});
}

// Tensor-core launch.  per_example = 0 runs the plain contraction over all B*T rows (its result goes
// to whichever of out_mean / out_stat is not NULL).  With per_example = 1 and both outputs wanted the
// pair tile is 256 x 128 (two running sums per thread); with only out_stat it is 256 x 256.
static pe_status_t launch_tc(DeviceInfo* di, const void* X, const void* dY, int B, int T, int d_in, int d_out, int phi,
                             int per_example, float* out_mean, float* out_stat, cudaStream_t st, bool half_ops = false,
                             float* out_sign = nullptr, bool accumulate = false, const float* sq_norms = nullptr, float clip_norm = 0.f) {
  const bool triple = out_sign != nullptr;       // mean + square + sign in one pass (phi = square, all three outputs given)
  const bool both = per_example && out_mean && out_stat;
  // Both outputs: sum_b G_b in tensor memory beside a 256-wide accumulator, unless the sequences are
  // so short that the per-example drain of that single accumulator would dominate.
  const int forced = g_path.load();
  // 256 x 192 tile: 22 % less operand traffic per flop than 256 x 128
  const long long pad192 = (long long)((d_in + 191) / 192) * 192, pad128 = (long long)((d_in + 127) / 128) * 128;
  const bool wide = both && forced != PE_PATH_TENSOR_NARROW &&
                    (forced == PE_PATH_TENSOR_WIDE || (T >= (triple ? TC_WIDE_TRIPLE_MIN_T : TC_WIDE_MIN_T) &&
                                                       pad192 * 100 <= pad128 * (100 + TC_WIDE_MAX_PAD_PERCENT)));
  const bool mean_regs = both && (triple || wide || T < TC_MEAN_TMEM_MIN_T || forced == PE_PATH_TENSOR_NARROW);
  const int nt = mean_regs ? (wide ? 192 : 128) : 256;
  const int box_feats = TcOperand<false, 256>::BOX_FEATS;
  const bool short_seq = mean_regs && !wide && T <= TC_SHORT_T;      // many short examples, both sums in registers: small stages
  const int box_tokens = short_seq ? TC_SHORT_BK : tc_default_bk(false, nt);
  CUtensorMap mx, my;
  // short sequences: a box is two examples deep (a stage holds two examples of 32 tokens each)
  const int box_examples = short_seq ? TcOperand<false, 128, TC_SHORT_BK>::GROUP : 1;
  pe_status_t rc = wide ? make_operand_map(&mx, X, B, T, d_in, false, TcOperand<false, 192>::B_BOX_FEATS, box_tokens, true)
                        : make_operand_map(&mx, X, B, T, d_in, false, box_feats, box_tokens, false, box_examples);
  if (rc != PE_OK) return rc;
  rc = make_operand_map(&my, dY, B, T, d_out, false, box_feats, box_tokens, false, box_examples);
  if (rc != PE_OK) return rc;
  CUtensorMap mm, ms;       // an output that is not wanted gets the other one's map and is never used
  rc = make_output_map(&mm, out_mean ? out_mean : out_stat, d_in, d_out);
  if (rc != PE_OK) return rc;
  rc = make_output_map(&ms, out_stat ? out_stat : out_mean, d_in, d_out);
  if (rc != PE_OK) return rc;
  CUtensorMap msgn = ms;
  if (triple && (rc = make_output_map(&msgn, out_sign, d_in, d_out)) != PE_OK) return rc;
  const int tiles_n = (d_in + nt - 1) / nt, pairs_m = (d_out + TC_PAIR_M - 1) / TC_PAIR_M;
  if ((long long)tiles_n * pairs_m > (1ll << 29)) return PE_ERR_DIM;
  int ns = choose_nsplit((long long)tiles_n * pairs_m, B, T, di->sm_count / 2 > 0 ? di->sm_count / 2 : 1, 16);
  if (triple && (B + ns - 1) / ns > TC_SIGN_COUNT_MAX) ns = (B + TC_SIGN_COUNT_MAX - 1) / TC_SIGN_COUNT_MAX;   // 16-bit sign counters
  if (ns > 1 && !accumulate) {
    rc = zero_for_split(di, out_mean, out_stat, (size_t)d_in * d_out, st, out_sign);
    if (rc != PE_OK) return rc;
  }
  TcParams p;
  p.B = B; p.T = T; p.d_in = d_in; p.d_out = d_out; p.nsplit = ns; p.per_example = per_example; p.half_operands = half_ops ? 1 : 0;
  p.accumulate = accumulate ? 1 : 0;
  p.pairs_m = pairs_m; p.tiles_n = tiles_n; p.band = choose_band(pairs_m, tiles_n, nt, ns, di->sm_count / 2);
  p.out_mean = out_mean; p.out_stat = out_stat; p.out_sign = out_sign; p.out_norms = nullptr; p.dev_status = di->status_ptr;
  p.seq_offsets = nullptr; p.sq_norms = sq_norms; p.clip_norm = clip_norm;
  dim3 grid(2 * pairs_m * tiles_n, 1, ns);
  if (phi == PHI_CLIP_SCALE) return launch_tc_inst<3, false, 256, MEAN_NONE>(di, 14, mx, my, mm, ms, msgn, p, grid, st);
  if (triple && wide) return launch_tc_inst<1, false, 192, MEAN_HYBRID_SIGN>(di, 26, mx, my, mm, ms, msgn, p, grid, st);
  if (triple && short_seq) return launch_tc_inst<1, false, 128, MEAN_REGS_SIGN, TC_SHORT_BK>(di, 27, mx, my, mm, ms, msgn, p, grid, st);
  if (triple) return launch_tc_inst<1, false, 128, MEAN_REGS_SIGN>(di, 10, mx, my, mm, ms, msgn, p, grid, st);
  if (!per_example) return launch_tc_inst<0, false, 256, MEAN_NONE>(di, 4, mx, my, mm, ms, msgn, p, grid, st);
  if (short_seq) {
    if (phi == PE_PHI_SQUARE) return launch_tc_inst<1, false, 128, MEAN_REGS, TC_SHORT_BK>(di, 8, mx, my, mm, ms, msgn, p, grid, st);
    return launch_tc_inst<2, false, 128, MEAN_REGS, TC_SHORT_BK>(di, 9, mx, my, mm, ms, msgn, p, grid, st);
  }
  if (wide) {
    if (phi == PE_PHI_SQUARE) return launch_tc_inst<1, false, 192, MEAN_REGS>(di, 12, mx, my, mm, ms, msgn, p, grid, st);
    return launch_tc_inst<2, false, 192, MEAN_REGS>(di, 13, mx, my, mm, ms, msgn, p, grid, st);
  }
  if (mean_regs) {
    if (phi == PE_PHI_SQUARE) return launch_tc_inst<1, false, 128, MEAN_REGS>(di, 0, mx, my, mm, ms, msgn, p, grid, st);
    return launch_tc_inst<2, false, 128, MEAN_REGS>(di, 1, mx, my, mm, ms, msgn, p, grid, st);
  }
  if (both) {
    if (phi == PE_PHI_SQUARE) return launch_tc_inst<1, false, 256, MEAN_TMEM>(di, 6, mx, my, mm, ms, msgn, p, grid, st);
    return launch_tc_inst<2, false, 256, MEAN_TMEM>(di, 7, mx, my, mm, ms, msgn, p, grid, st);
  }
  if (phi == PE_PHI_SQUARE) return launch_tc_inst<1, false, 256, MEAN_NONE>(di, 2, mx, my, mm, ms, msgn, p, grid, st);
  return launch_tc_inst<2, false, 256, MEAN_NONE>(di, 3, mx, my, mm, ms, msgn, p, grid, st);
}

// Per-example squared norms on the tensor cores: the statistic-only 256 x 256 schedule, but every
// example's tile is reduced to one number and added to norms[b] (zeroed by the caller of this function).
static pe_status_t launch_tc_norms(DeviceInfo* di, const void* X, const void* dY, int B, int T, int d_in, int d_out, float* norms,
                                   cudaStream_t st) {
  CUtensorMap mx, my;
  const int box_feats = TcOperand<false, 256>::BOX_FEATS, box_tokens = tc_default_bk(false, 256);
  pe_status_t rc = make_operand_map(&mx, X, B, T, d_in, false, box_feats, box_tokens);
  if (rc != PE_OK) return rc;
  rc = make_operand_map(&my, dY, B, T, d_out, false, box_feats, box_tokens);
  if (rc != PE_OK) return rc;
  const int tiles_n = (d_in + 255) / 256, pairs_m = (d_out + TC_PAIR_M - 1) / TC_PAIR_M;
  if ((long long)tiles_n * pairs_m > (1ll << 29)) return PE_ERR_DIM;
  const int ns = choose_nsplit((long long)tiles_n * pairs_m, B, T, di->sm_count / 2 > 0 ? di->sm_count / 2 : 1, 16);
  TcParams p;
  p.B = B; p.T = T; p.d_in = d_in; p.d_out = d_out; p.nsplit = ns; p.per_example = 1; p.half_operands = 0;
  p.accumulate = 1;       // nothing is zeroed by a preceding kernel and no matrix is written
  p.pairs_m = pairs_m; p.tiles_n = tiles_n; p.band = choose_band(pairs_m, tiles_n, 256, ns, di->sm_count / 2);
  p.out_mean = nullptr; p.out_stat = nullptr; p.out_sign = nullptr; p.out_norms = norms; p.dev_status = di->status_ptr;
  p.seq_offsets = nullptr; p.sq_norms = nullptr; p.clip_norm = 0.f;
  // the three output maps are never used by this variant: any valid map will do
  return launch_tc_inst<1, false, 256, MEAN_NORMS>(di, 11, mx, my, mx, mx, mx, p, dim3(2 * pairs_m * tiles_n, 1, ns), st);
}

template <typename TIn, int MODE>
static pe_status_t launch_simt(DeviceInfo* di, const TIn* X, const TIn* dY, int B, int T, int d_in, int d_out, int phi,
                               float* out_mean, float* out_stat, cudaStream_t st, bool accumulate = false, SimtExtra ex = SimtExtra{},
                               const FusedOpt* opt = nullptr) {
  const int tx = (d_in + SIMT_TILE - 1) / SIMT_TILE, ty = (d_out + SIMT_TILE - 1) / SIMT_TILE;
  if (ty > 65535) return PE_ERR_DIM;
  // a fused update needs the whole batch in one block (this kernel has no cross-block completion protocol)
  const int ns = opt ? 1 : choose_nsplit((long long)tx * ty, B, T, di->sm_count * 3, 64);
  if (ns > 1 && !accumulate) {
    pe_status_t rc = zero_outputs(out_mean, out_stat, (size_t)d_in * d_out * sizeof(float), st);
    if (rc != PE_OK) return rc;
  }
  simt_stats_kernel<TIn, MODE><<<dim3(tx, ty, ns), SIMT_THREADS, 0, st>>>(X, dY, B, T, d_in, d_out, phi, out_mean, out_stat, accumulate ? 1 : 0, ex,
                                                                            opt ? *opt : FusedOpt{});
  return check_launch();
}

// Side buffer of a packed batch: the zero-padded last partial 16-token group of every sequence, X's [B, 16, d_in]
// then dY's [B, 16, d_out] (bf16), each part 256-byte aligned.
struct RaggedLayout {
  size_t x_bytes, y_bytes;
  size_t total() const { return x_bytes + y_bytes; }
};
static RaggedLayout ragged_layout(int B, int d_in, int d_out) {
  RaggedLayout l;
  l.x_bytes = ((size_t)B * 16 * (size_t)d_in * 2 + 255) / 256 * 256;
  l.y_bytes = ((size_t)B * 16 * (size_t)d_out * 2 + 255) / 256 * 256;
  return l;
}

// Tensor-core launch for a packed batch.  norms != NULL: per-example squared norms (zeroed by the caller);
// otherwise the statistics of pe_linear_stats.  phi = identity (or only out_mean wanted) runs the per-example
// kernel with the identity, whose running sum is sum_b G_b.
static pe_status_t launch_tc_ragged(DeviceInfo* di, const void* X, const void* dY, const int* offsets, int B, long long rows, int d_in,
                                    int d_out, int phi, float* out_mean, float* out_stat, float* norms, void* ws, cudaStream_t st) {
  const RaggedLayout l = ragged_layout(B, d_in, d_out);
  uint16_t* xt = static_cast<uint16_t*>(ws);
  uint16_t* yt = reinterpret_cast<uint16_t*>(static_cast<char*>(ws) + l.x_bytes);
  const TailTensor tx = {static_cast<const uint16_t*>(X), xt, d_in}, ty = {static_cast<const uint16_t*>(dY), yt, d_out};
  pack_tails_kernel<<<dim3((unsigned)B, 2, 1), STAGE_THREADS, 0, st>>>(tx, ty, offsets, rows);
  pe_status_t rc = check_launch();
  if (rc != PE_OK) return rc;
  const bool both = !norms && out_mean && out_stat && phi != PE_PHI_IDENTITY;
  const bool plain = !norms && (phi == PE_PHI_IDENTITY || !out_stat);      // only sum_b G_b
  const int nt = both ? 192 : 256;
  const int box_tokens = tc_default_bk(false, nt);
  const int rows_i = (int)(rows > 0 ? rows : 1);
  CUtensorMap mx, my, mxt, myt;
  const int bf = TcOperand<false, 256>::BOX_FEATS;
  if (both) {
    rc = make_operand_map(&mx, X, 1, rows_i, d_in, false, TcOperand<false, 192>::B_BOX_FEATS, box_tokens, true);
    if (rc == PE_OK) rc = make_operand_map(&mxt, xt, B, 16, d_in, false, TcOperand<false, 192>::B_BOX_FEATS, box_tokens, true);
  } else {
    rc = make_operand_map(&mx, X, 1, rows_i, d_in, false, bf, box_tokens);
    if (rc == PE_OK) rc = make_operand_map(&mxt, xt, B, 16, d_in, false, bf, box_tokens);
  }
  if (rc == PE_OK) rc = make_operand_map(&my, dY, 1, rows_i, d_out, false, bf, box_tokens);
  if (rc == PE_OK) rc = make_operand_map(&myt, yt, B, 16, d_out, false, bf, box_tokens);
  if (rc != PE_OK) return rc;
  float* first = plain ? (out_mean ? out_mean : out_stat) : out_stat;
  CUtensorMap mm = mx, ms = mx;       // never used by the norms variant
  if (!norms) {
    rc = make_output_map(&ms, first, d_in, d_out);
    if (rc == PE_OK) rc = make_output_map(&mm, both ? out_mean : first, d_in, d_out);
    if (rc != PE_OK) return rc;
  }
  const int tiles_n = (d_in + nt - 1) / nt, pairs_m = (d_out + TC_PAIR_M - 1) / TC_PAIR_M;
  if ((long long)tiles_n * pairs_m > (1ll << 29)) return PE_ERR_DIM;
  const long long t_avg = rows / B > 0 ? rows / B : 1;
  const int ns = choose_nsplit((long long)tiles_n * pairs_m, B, (int)(t_avg > (1 << 20) ? (1 << 20) : t_avg),
                               di->sm_count / 2 > 0 ? di->sm_count / 2 : 1, 16);
  if (ns > 1 && !norms) {
    rc = zero_for_split(di, both ? out_mean : nullptr, first, (size_t)d_in * d_out, st);
    if (rc != PE_OK) return rc;
  }
  TcParams p;
  p.B = B; p.T = 0; p.d_in = d_in; p.d_out = d_out; p.nsplit = ns; p.per_example = 1; p.half_operands = 0;
  p.accumulate = norms ? 1 : 0;
  p.pairs_m = pairs_m; p.tiles_n = tiles_n; p.band = choose_band(pairs_m, tiles_n, nt, ns, di->sm_count / 2);
  p.out_mean = both ? out_mean : nullptr; p.out_stat = norms ? nullptr : first; p.out_sign = nullptr; p.out_norms = norms;
  p.seq_offsets = offsets; p.sq_norms = nullptr; p.clip_norm = 0.f; p.dev_status = di->status_ptr;
  const dim3 grid(2 * pairs_m * tiles_n, 1, ns);
  if (norms) return launch_tc_inst<1, false, 256, MEAN_NORMS, 64, true>(di, 15, mx, my, mm, ms, ms, p, grid, st, &mxt, &myt);
  if (plain) {
    rc = launch_tc_inst<0, false, 256, MEAN_NONE, 64, true>(di, 20, mx, my, mm, ms, ms, p, grid, st, &mxt, &myt);
    if (rc == PE_OK && out_mean && out_stat &&
        cudaMemcpyAsync(out_stat, out_mean, (size_t)d_in * d_out * sizeof(float), cudaMemcpyDeviceToDevice, st) != cudaSuccess) {
      cudaGetLastError();
      return PE_ERR_CUDA;
    }
    return rc;
  }
  if (both) {
    if (phi == PE_PHI_SQUARE) return launch_tc_inst<1, false, 192, MEAN_REGS, 128, true>(di, 16, mx, my, mm, ms, ms, p, grid, st, &mxt, &myt);
    return launch_tc_inst<2, false, 192, MEAN_REGS, 128, true>(di, 17, mx, my, mm, ms, ms, p, grid, st, &mxt, &myt);
  }
  if (phi == PE_PHI_SQUARE) return launch_tc_inst<1, false, 256, MEAN_NONE, 64, true>(di, 18, mx, my, mm, ms, ms, p, grid, st, &mxt, &myt);
  return launch_tc_inst<2, false, 256, MEAN_NONE, 64, true>(di, 19, mx, my, mm, ms, ms, p, grid, st, &mxt, &myt);
}

static pe_status_t validate_stats(const void* X, const void* dY, int B, int T, int d_in, int d_out, const float* o1,
                                  const float* o2, bool need_both_null_check, size_t in_align) {
  if (B < 0 || T < 0 || d_in < 1 || d_out < 1) return PE_ERR_DIM;
  if ((!X || !dY) && B > 0 && T > 0) return PE_ERR_NULL;      // empty inputs may be NULL
  if (need_both_null_check && !o1 && !o2) return PE_ERR_NULL;
  if ((long long)B * T * (long long)(d_in > d_out ? d_in : d_out) >= (1ll << 40)) return PE_ERR_DIM;
  if ((long long)d_in * d_out >= (1ll << 40)) return PE_ERR_DIM;
  if (!aligned(X, in_align) || !aligned(dY, in_align)) return PE_ERR_ALIGN;
  if ((o1 && !aligned(o1, 16)) || (o2 && !aligned(o2, 16))) return PE_ERR_ALIGN;
  return PE_OK;
}

// A plain contraction over all B*T rows does not care where one sequence ends: short sequences are
// regrouped into full two-stage "examples" when the rows divide evenly (fewer, fuller pipeline stages).
static void regroup_rows(int& B, int& T) {
  constexpr int REGROUP = 2 * TcOperand<false, 256>::BK;
  const long long rows = (long long)B * T;
  if (T < REGROUP && rows % REGROUP == 0) { B = (int)(rows / REGROUP); T = REGROUP; }
}

template <typename TIn>
static pe_status_t linear_stats_impl(const TIn* X, const TIn* dY, int B, int T, int d_in, int d_out, pe_phi_t phi,
                                     float* out_mean, float* out_stat, cudaStream_t st, bool allow_tc, bool accumulate = false) {
  pe_status_t rc = validate_stats(X, dY, B, T, d_in, d_out, out_mean, out_stat, true, allow_tc ? 16 : 4);
  if (rc != PE_OK) return rc;
  if (phi != PE_PHI_IDENTITY && phi != PE_PHI_SQUARE && phi != PE_PHI_SIGN) return PE_ERR_PHI;
  DeviceInfo* di = nullptr;
  rc = device_info(&di);
  if (rc != PE_OK) return rc;
  if (B == 0 || T == 0) return accumulate ? PE_OK : zero_outputs(out_mean, out_stat, (size_t)d_in * d_out * sizeof(float), st);
  const int forced = g_path.load();
  const bool tc_ok = allow_tc && tc_shape_ok(B, T, d_in, d_out);
  if (forced >= PE_PATH_TENSOR && !tc_ok) return PE_ERR_UNSUPPORTED_SHAPE;
  if (tc_ok && forced != PE_PATH_SIMT) {
    if constexpr (sizeof(TIn) == 2) {
      g_last_path.store(PE_PATH_TENSOR);
      if (phi == PE_PHI_IDENTITY) {
        // phi = identity: both outputs are the plain contraction over all B*T rows, and B and T only enter
        // through B*T: regroup short sequences into full two-stage "examples" when the rows divide evenly.
        regroup_rows(B, T);
        float* first = out_mean ? out_mean : out_stat;
        rc = launch_tc(di, X, dY, B, T, d_in, d_out, phi, 0, first, nullptr, st, false, nullptr, accumulate);
        if (rc == PE_OK && out_mean && out_stat && accumulate)      // a copy would overwrite: contract once more into the second
          return launch_tc(di, X, dY, B, T, d_in, d_out, phi, 0, out_stat, nullptr, st, false, nullptr, true);
        if (rc == PE_OK && out_mean && out_stat) {
          if (cudaMemcpyAsync(out_stat, out_mean, (size_t)d_in * d_out * sizeof(float), cudaMemcpyDeviceToDevice, st) != cudaSuccess) {
            cudaGetLastError();
            return PE_ERR_CUDA;
          }
        }
        return rc;
      }
      if (!out_stat) {    // only sum_b G_b wanted: the plain contraction
        regroup_rows(B, T);
        return launch_tc(di, X, dY, B, T, d_in, d_out, phi, 0, out_mean, nullptr, st, false, nullptr, accumulate);
      }
      return launch_tc(di, X, dY, B, T, d_in, d_out, phi, 1, out_mean, out_stat, st, false, nullptr, accumulate);
    }
  }
  g_last_path.store(PE_PATH_SIMT);
  return launch_simt<TIn, MODE_STATS>(di, X, dY, B, T, d_in, d_out, (int)phi, out_mean, out_stat, st, accumulate);
}

static size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Constants of one Adam-family step (Algorithm 1): the scales that turn the sums into averages, the
// bias corrections of step t, and the factor 1 / (1 - 1/B) of Eq. (6).
static AdamParams make_adam_params(int B, float grad_scale, float lr, float beta1, float beta2, float eps, int eps_inside_sqrt,
                                   float weight_decay, int step) {
  AdamParams p;
  p.mu_scale = (float)((double)grad_scale / (double)B);
  p.nu_scale = (float)((double)grad_scale * (double)grad_scale / (double)B);
  p.beta1 = beta1; p.beta2 = beta2;
  p.inv_c1 = (float)(1.0 / (1.0 - std::pow((double)beta1, (double)step)));
  p.inv_c2 = (float)(1.0 / (1.0 - std::pow((double)beta2, (double)step)));
  p.eps = eps; p.lr = lr; p.wd = weight_decay; p.eps_inside = eps_inside_sqrt ? 1 : 0;
  p.inv_B = (float)(1.0 / (double)B);
  p.bessel = B > 1 ? (float)(1.0 / (1.0 - 1.0 / (double)B)) : 1.f;
  return p;
}

// Words of tile counters a fused statistics + update launch may need: one per thread block of the widest grid
// (256 x 128 tiles), i.e. two per pair tile.
static size_t fused_counter_words(int d_in, int d_out) {
  return 2 * (size_t)((d_out + TC_PAIR_M - 1) / TC_PAIR_M) * (size_t)((d_in + 127) / 128);
}

// Statistics and parameter update in one tensor-core launch.  kind = OPT_ADAM: sum_b G_b and sum_b G_b^2 (256 x 192 or
// 256 x 128 tile, both sums in registers) feed Algorithm 1; kind = OPT_SIGN: sum_b sign(G_b) (256 x 256 tile) feeds
// MicroSignSGD.  out_a = out_mean (Adam only), out_b = the statistic; they may be NULL when the schedule does not
// split the batch, which is forced when they (or the counters) are missing.
static pe_status_t launch_tc_fused(DeviceInfo* di, const void* X, const void* dY, int B, int T, int d_in, int d_out, int kind,
                                   float* out_a, float* out_b, FusedOpt opt, unsigned int* counters, size_t counter_words,
                                   cudaStream_t st) {
  const bool adam = kind == OPT_ADAM;
  const long long pad192 = (long long)((d_in + 191) / 192) * 192, pad128 = (long long)((d_in + 127) / 128) * 128;
  const int forced = g_path.load();
  const bool wide = adam && forced != PE_PATH_TENSOR_NARROW &&
                    (forced == PE_PATH_TENSOR_WIDE || (T >= TC_WIDE_MIN_T && pad192 * 100 <= pad128 * (100 + TC_WIDE_MAX_PAD_PERCENT)));
  const int nt = adam ? (wide ? 192 : 128) : 256;
  const int box_feats = TcOperand<false, 256>::BOX_FEATS, box_tokens = tc_default_bk(false, nt);
  CUtensorMap mx, my, mm, ms;
  pe_status_t rc = wide ? make_operand_map(&mx, X, B, T, d_in, false, TcOperand<false, 192>::B_BOX_FEATS, box_tokens, true)
                        : make_operand_map(&mx, X, B, T, d_in, false, box_feats, box_tokens);
  if (rc == PE_OK) rc = make_operand_map(&my, dY, B, T, d_out, false, box_feats, box_tokens);
  // an output that is not wanted gets a map over the parameters and is never written through it
  if (rc == PE_OK) rc = make_output_map(&mm, out_a ? out_a : opt.theta, d_in, d_out);
  if (rc == PE_OK) rc = make_output_map(&ms, out_b ? out_b : opt.theta, d_in, d_out);
  if (rc != PE_OK) return rc;
  const int tiles_n = (d_in + nt - 1) / nt, pairs_m = (d_out + TC_PAIR_M - 1) / TC_PAIR_M;
  if ((long long)tiles_n * pairs_m > (1ll << 29)) return PE_ERR_DIM;
  int ns = choose_nsplit((long long)tiles_n * pairs_m, B, T, di->sm_count / 2 > 0 ? di->sm_count / 2 : 1, 16);
  const size_t blocks = 2 * (size_t)tiles_n * pairs_m;
  if (ns > 1 && (!out_b || (adam && !out_a) || !counters || counter_words < blocks)) ns = 1;
  if (ns > 1) {
    rc = zero_for_split(di, adam ? out_a : nullptr, out_b, (size_t)d_in * d_out, st, nullptr, counters, (int)blocks);
    if (rc != PE_OK) return rc;
  }
  TcParams p;
  p.B = B; p.T = T; p.d_in = d_in; p.d_out = d_out; p.nsplit = ns; p.per_example = 1; p.half_operands = 0; p.accumulate = 0;
  p.pairs_m = pairs_m; p.tiles_n = tiles_n; p.band = choose_band(pairs_m, tiles_n, nt, ns, di->sm_count / 2);
  p.out_mean = adam ? out_a : nullptr; p.out_stat = out_b; p.out_sign = nullptr; p.out_norms = nullptr; p.dev_status = di->status_ptr;
  p.seq_offsets = nullptr; p.sq_norms = nullptr; p.clip_norm = 0.f;
  opt.kind = kind;
  opt.tile_counters = counters;
  const dim3 grid((unsigned)blocks, 1, ns);
  if (!adam) return launch_tc_inst<2, false, 256, MEAN_NONE, 64, false, OPT_SIGN>(di, 23, mx, my, mm, ms, ms, p, grid, st, nullptr, nullptr, &opt);
  if (wide) return launch_tc_inst<1, false, 192, MEAN_REGS, 128, false, OPT_ADAM>(di, 21, mx, my, mm, ms, ms, p, grid, st, nullptr, nullptr, &opt);
  return launch_tc_inst<1, false, 128, MEAN_REGS, 128, false, OPT_ADAM>(di, 22, mx, my, mm, ms, ms, p, grid, st, nullptr, nullptr, &opt);
}

static int grid_for(long long work_items, int sm_count) {
  long long blocks = (work_items + OPT_THREADS - 1) / OPT_THREADS;
  long long cap = (long long)sm_count * 8;
  if (blocks < 1) blocks = 1;
  return (int)(blocks < cap ? blocks : cap);
}

// Fused per-token statistic: squares, rounds to tf32 and contracts inside one kernel.
static pe_status_t launch_tok(DeviceInfo* di, const void* X, const void* dY, long long rows, int d_in, int d_out, float* out,
                              cudaStream_t st) {
  EncodeTiledFn enc = encode_fn();
  if (!enc) return PE_ERR_CUDA;
  CUtensorMap mx, my, mo;
  auto operand_map = [&](CUtensorMap* m, const void* base, int d) {
    cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)d * 2ull};
    cuuint32_t box[2] = {64u, (cuuint32_t)TOK_BK};
    cuuint32_t estr[2] = {1u, 1u};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
  };
  if (!operand_map(&mx, X, d_in) || !operand_map(&my, dY, d_out)) return PE_ERR_CUDA;
  pe_status_t rc = make_output_map(&mo, out, d_in, d_out);
  if (rc != PE_OK) return rc;
  const int tiles_n = (d_in + TOK_NT - 1) / TOK_NT, pairs_m = (d_out + TC_PAIR_M - 1) / TC_PAIR_M;
  if ((long long)tiles_n * pairs_m > (1ll << 29)) return PE_ERR_DIM;
  const long long n_chunks = (rows + TOK_BK - 1) / TOK_BK;
  const int units = n_chunks > (1 << 30) ? (1 << 30) : (int)n_chunks;
  const int ns = choose_nsplit((long long)tiles_n * pairs_m, units, TOK_BK, di->sm_count / 2 > 0 ? di->sm_count / 2 : 1, 32);
  if (ns > 1) {
    rc = zero_for_split(di, out, nullptr, (size_t)d_in * d_out, st);
    if (rc != PE_OK) return rc;
  }
  {
    std::lock_guard<std::mutex> lock(g_dev_mutex);
    if (!di->tok_attr_set) {
      if (cudaFuncSetAttribute(tok_sqstats_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, TOK_SMEM_BYTES) != cudaSuccess) {
        cudaGetLastError();
        return PE_ERR_CUDA;
      }
      di->tok_attr_set = true;
    }
  }
  TokParams p;
  p.rows = rows; p.d_in = d_in; p.d_out = d_out; p.pairs_m = pairs_m; p.tiles_n = tiles_n;
  p.band = choose_band(pairs_m, tiles_n, TOK_NT, ns, di->sm_count / 2); p.nsplit = ns; p.dev_status = di->status_ptr;
  return launch_pair_kernel_t(tok_sqstats_kernel, dim3(2 * pairs_m * tiles_n, 1, ns), TOK_THREADS, TOK_SMEM_BYTES, st, ns > 1, mx, my, mo, p);
}

}  // namespace pe

using namespace pe;

extern "C" {

pe_status_t pe_linear_stats(const void* X, const void* dY, int B, int T, int d_in, int d_out, pe_phi_t phi,
                            float* out_mean, float* out_stat, pe_stream_t stream) {
  return linear_stats_impl<__nv_bfloat16>(static_cast<const __nv_bfloat16*>(X), static_cast<const __nv_bfloat16*>(dY), B, T,
                                          d_in, d_out, phi, out_mean, out_stat, reinterpret_cast<cudaStream_t>(stream), true);
}

pe_status_t pe_example_sqnorms(const void* X, const void* dY, int B, int T, int d_in, int d_out, float* out_norms,
                               pe_stream_t stream) {
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  if (!out_norms && B > 0) return PE_ERR_NULL;
  pe_status_t rc = validate_stats(X, dY, B, T, d_in, d_out, nullptr, nullptr, false, 16);
  if (rc != PE_OK) return rc;
  if (out_norms && !aligned(out_norms, 4)) return PE_ERR_ALIGN;
  DeviceInfo* di = nullptr;
  rc = device_info(&di);
  if (rc != PE_OK) return rc;
  if (B == 0) return PE_OK;
  if (cudaMemsetAsync(out_norms, 0, (size_t)B * sizeof(float), st) != cudaSuccess) { cudaGetLastError(); return PE_ERR_CUDA; }
  if (T == 0) return PE_OK;
  const int forced = g_path.load();
  const bool tc_ok = tc_shape_ok(B, T, d_in, d_out);
  if (forced >= PE_PATH_TENSOR && !tc_ok) return PE_ERR_UNSUPPORTED_SHAPE;
  if (tc_ok && forced != PE_PATH_SIMT) {
    g_last_path.store(PE_PATH_TENSOR);
    return launch_tc_norms(di, X, dY, B, T, d_in, d_out, out_norms, st);
  }
  g_last_path.store(PE_PATH_SIMT);
  // every block handles whole examples of its slice and adds to out_norms[b]: "accumulate" keeps launch_simt from zeroing
  return launch_simt<__nv_bfloat16, MODE_NORMS>(di, static_cast<const __nv_bfloat16*>(X), static_cast<const __nv_bfloat16*>(dY), B, T,
                                                d_in, d_out, 1, nullptr, out_norms, st, true);
}

pe_status_t pe_linear_stats_accumulate(const void* X, const void* dY, int B, int T, int d_in, int d_out, pe_phi_t phi,
                                       float* out_mean, float* out_stat, pe_stream_t stream) {
  return linear_stats_impl<__nv_bfloat16>(static_cast<const __nv_bfloat16*>(X), static_cast<const __nv_bfloat16*>(dY), B, T,
                                          d_in, d_out, phi, out_mean, out_stat, reinterpret_cast<cudaStream_t>(stream), true, true);
}

pe_status_t pe_linear_stats_all(const void* X, const void* dY, int B, int T, int d_in, int d_out, float* out_mean,
                                float* out_square, float* out_sign, pe_stream_t stream) {
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  if (!out_mean || !out_square || !out_sign) return PE_ERR_NULL;
  pe_status_t rc = validate_stats(X, dY, B, T, d_in, d_out, out_mean, out_square, true, 16);
  if (rc != PE_OK) return rc;
  if (!aligned(out_sign, 16)) return PE_ERR_ALIGN;
  DeviceInfo* di = nullptr;
  rc = device_info(&di);
  if (rc != PE_OK) return rc;
  const int forced = g_path.load();
  // One pass when the tensor-core kernel takes the shape; otherwise the two calls this one stands for.
  if (B > 0 && T > 0 && forced != PE_PATH_SIMT && tc_shape_ok(B, T, d_in, d_out)) {
    g_last_path.store(PE_PATH_TENSOR);
    return launch_tc(di, X, dY, B, T, d_in, d_out, PE_PHI_SQUARE, 1, out_mean, out_square, st, false, out_sign);
  }
  const __nv_bfloat16* Xb = static_cast<const __nv_bfloat16*>(X);
  const __nv_bfloat16* Yb = static_cast<const __nv_bfloat16*>(dY);
  rc = linear_stats_impl<__nv_bfloat16>(Xb, Yb, B, T, d_in, d_out, PE_PHI_SQUARE, out_mean, out_square, st, true);
  if (rc != PE_OK) return rc;
  return linear_stats_impl<__nv_bfloat16>(Xb, Yb, B, T, d_in, d_out, PE_PHI_SIGN, nullptr, out_sign, st, true);
}

size_t pe_linear_stats_ragged_workspace_bytes(int B, int d_in, int d_out) {
  if (B < 1 || d_in < 1 || d_out < 1 || (d_in % 8) || (d_out % 8) || g_path.load() == PE_PATH_SIMT) return 0;
  return ragged_layout(B, d_in, d_out).total();
}

// Shared by pe_linear_stats_ragged and pe_example_sqnorms_ragged (norms != NULL).
static pe_status_t ragged_impl(const void* X, const void* dY, const int* seq_offsets, int B, long long total_rows, int d_in, int d_out,
                               int phi, float* out_mean, float* out_stat, float* norms, void* workspace, size_t workspace_bytes,
                               cudaStream_t st) {
  if (B < 0 || total_rows < 0 || total_rows >= (1ll << 31) || d_in < 1 || d_out < 1) return PE_ERR_DIM;
  if (B > 0 && !seq_offsets) return PE_ERR_NULL;
  if ((!X || !dY) && B > 0 && total_rows > 0) return PE_ERR_NULL;
  if (!norms && !out_mean && !out_stat) return PE_ERR_NULL;
  if (total_rows * (long long)(d_in > d_out ? d_in : d_out) >= (1ll << 40) || (long long)d_in * d_out >= (1ll << 40)) return PE_ERR_DIM;
  if (!aligned(X, 16) || !aligned(dY, 16) || !aligned(seq_offsets, 4)) return PE_ERR_ALIGN;
  if ((out_mean && !aligned(out_mean, 16)) || (out_stat && !aligned(out_stat, 16)) || (norms && !aligned(norms, 4))) return PE_ERR_ALIGN;
  if (!norms && phi != PE_PHI_IDENTITY && phi != PE_PHI_SQUARE && phi != PE_PHI_SIGN) return PE_ERR_PHI;
  DeviceInfo* di = nullptr;
  pe_status_t rc = device_info(&di);
  if (rc != PE_OK) return rc;
  if (norms) {
    if (B == 0) return PE_OK;
    if (cudaMemsetAsync(norms, 0, (size_t)B * sizeof(float), st) != cudaSuccess) { cudaGetLastError(); return PE_ERR_CUDA; }
  }
  if (B == 0 || total_rows == 0) return norms ? PE_OK : zero_outputs(out_mean, out_stat, (size_t)d_in * d_out * sizeof(float), st);
  const int forced = g_path.load();
  const bool tc_ok = (d_in % 8) == 0 && (d_out % 8) == 0;
  if (forced >= PE_PATH_TENSOR && !tc_ok) return PE_ERR_UNSUPPORTED_SHAPE;
  if (tc_ok && forced != PE_PATH_SIMT) {
    if (!workspace || workspace_bytes < ragged_layout(B, d_in, d_out).total()) return PE_ERR_WORKSPACE;
    if (!aligned(workspace, 256)) return PE_ERR_ALIGN;
    g_last_path.store(PE_PATH_TENSOR);
    return launch_tc_ragged(di, X, dY, seq_offsets, B, total_rows, d_in, d_out, phi, out_mean, out_stat, norms, workspace, st);
  }
  g_last_path.store(PE_PATH_SIMT);
  SimtExtra ex{};
  ex.seq_offsets = seq_offsets; ex.total_rows = total_rows;
  const long long t_avg = total_rows / B > 0 ? total_rows / B : 1;
  const __nv_bfloat16* Xb = static_cast<const __nv_bfloat16*>(X);
  const __nv_bfloat16* Yb = static_cast<const __nv_bfloat16*>(dY);
  if (norms) return launch_simt<__nv_bfloat16, MODE_NORMS>(di, Xb, Yb, B, (int)t_avg, d_in, d_out, 1, nullptr, norms, st, true, ex);
  return launch_simt<__nv_bfloat16, MODE_STATS>(di, Xb, Yb, B, (int)t_avg, d_in, d_out, phi, out_mean, out_stat, st, false, ex);
}

pe_status_t pe_linear_stats_ragged(const void* X, const void* dY, const int* seq_offsets, int B, long long total_rows, int d_in,
                                   int d_out, pe_phi_t phi, float* out_mean, float* out_stat, void* workspace,
                                   size_t workspace_bytes, pe_stream_t stream) {
  return ragged_impl(X, dY, seq_offsets, B, total_rows, d_in, d_out, (int)phi, out_mean, out_stat, nullptr, workspace, workspace_bytes,
                     reinterpret_cast<cudaStream_t>(stream));
}

pe_status_t pe_example_sqnorms_ragged(const void* X, const void* dY, const int* seq_offsets, int B, long long total_rows, int d_in,
                                      int d_out, float* out_norms, void* workspace, size_t workspace_bytes, pe_stream_t stream) {
  if (!out_norms && B > 0) return PE_ERR_NULL;
  return ragged_impl(X, dY, seq_offsets, B, total_rows, d_in, d_out, PE_PHI_SQUARE, nullptr, nullptr, out_norms, workspace,
                     workspace_bytes, reinterpret_cast<cudaStream_t>(stream));
}

pe_status_t pe_linear_clipped_sum(const void* X, const void* dY, int B, int T, int d_in, int d_out, float clip_norm, float* sq_norms,
                                  int norms_given, float* out_sum, pe_stream_t stream) {
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  if (!out_sum || (!sq_norms && B > 0)) return PE_ERR_NULL;
  if (!(clip_norm >= 0.f)) return PE_ERR_DIM;
  pe_status_t rc = validate_stats(X, dY, B, T, d_in, d_out, out_sum, nullptr, false, 16);
  if (rc != PE_OK) return rc;
  if (sq_norms && !aligned(sq_norms, 4)) return PE_ERR_ALIGN;
  DeviceInfo* di = nullptr;
  rc = device_info(&di);
  if (rc != PE_OK) return rc;
  if (B == 0 || T == 0) return zero_outputs(out_sum, nullptr, (size_t)d_in * d_out * sizeof(float), st);
  if (!norms_given) {
    rc = pe_example_sqnorms(X, dY, B, T, d_in, d_out, sq_norms, stream);
    if (rc != PE_OK) return rc;
  }
  const int forced = g_path.load();
  const bool tc_ok = tc_shape_ok(B, T, d_in, d_out);
  if (forced >= PE_PATH_TENSOR && !tc_ok) return PE_ERR_UNSUPPORTED_SHAPE;
  if (tc_ok && forced != PE_PATH_SIMT) {
    g_last_path.store(PE_PATH_TENSOR);
    return launch_tc(di, X, dY, B, T, d_in, d_out, PHI_CLIP_SCALE, 1, nullptr, out_sum, st, false, nullptr, false, sq_norms, clip_norm);
  }
  g_last_path.store(PE_PATH_SIMT);
  SimtExtra ex{};
  ex.sq_norms = sq_norms; ex.clip_norm = clip_norm;
  return launch_simt<__nv_bfloat16, MODE_STATS>(di, static_cast<const __nv_bfloat16*>(X), static_cast<const __nv_bfloat16*>(dY), B, T,
                                                d_in, d_out, PHI_CLIP_SCALE, nullptr, out_sum, st, false, ex);
}

size_t pe_linear_fused_workspace_bytes(int d_in, int d_out) {
  if (d_in < 1 || d_out < 1) return 0;
  return align_up(fused_counter_words(d_in, d_out) * sizeof(unsigned int), 256);
}

// Shared by the three fused entry points.  kind: OPT_ADAM / OPT_SIGN; out_a: sum_b G_b (Adam), out_b: the statistic.
extern "C++" template <typename TIn>
pe_status_t fused_impl(const TIn* X, const TIn* dY, int B, int T, int d_in, int d_out, int kind, float* theta, void* theta_lp,
                              float* m, float* v, float* out_a, float* out_b, FusedOpt opt, void* workspace, size_t workspace_bytes,
                              cudaStream_t st, bool allow_tc) {
  if (!theta || !m || (kind == OPT_ADAM && !v)) return PE_ERR_NULL;
  if (B < 1 || T < 1) return PE_ERR_DIM;
  pe_status_t rc = validate_stats(X, dY, B, T, d_in, d_out, out_a, out_b, false, allow_tc ? 16 : 4);
  if (rc != PE_OK) return rc;
  if (!aligned(theta, 16) || !aligned(m, 16) || (v && !aligned(v, 16)) || (theta_lp && !aligned(theta_lp, 16))) return PE_ERR_ALIGN;
  if (workspace && !aligned(workspace, 256)) return PE_ERR_ALIGN;
  DeviceInfo* di = nullptr;
  rc = device_info(&di);
  if (rc != PE_OK) return rc;
  opt.kind = kind;
  opt.theta = theta; opt.theta_lp = static_cast<__nv_bfloat16*>(theta_lp); opt.m = m; opt.v = v; opt.tile_counters = nullptr;
  const int forced = g_path.load();
  const bool tc_ok = allow_tc && tc_shape_ok(B, T, d_in, d_out);
  if (forced >= PE_PATH_TENSOR && !tc_ok) return PE_ERR_UNSUPPORTED_SHAPE;
  if (tc_ok && forced != PE_PATH_SIMT) {
    if constexpr (sizeof(TIn) == 2) {
      g_last_path.store(PE_PATH_TENSOR);
      // The update inside the statistics kernel cannot overlap the contraction: the blocks of a wave finish
      // together, so a wave's update traffic reaches memory at once while the tensor cores idle (measured: about
      // 25 us per wave, against a separate update kernel that streams at the HBM rate).  Fusing saves memory (no
      // [d_out, d_in] statistic buffers) rather than time.  PE_FUSED_AUTO
      // therefore fuses only when the caller gave no buffers for the statistics; with buffers it runs the
      // statistics kernel and the update kernel back to back.
      const int mode = g_fused_mode.load();
      const bool have_stats = out_b && (kind != OPT_ADAM || out_a);
      if (mode == PE_FUSED_NEVER && !have_stats) return PE_ERR_NULL;
      if (mode == PE_FUSED_NEVER || (mode == PE_FUSED_AUTO && have_stats)) {
        rc = launch_tc(di, X, dY, B, T, d_in, d_out, kind == OPT_ADAM ? (int)PE_PHI_SQUARE : (int)PE_PHI_SIGN, 1,
                       kind == OPT_ADAM ? out_a : nullptr, out_b, st);
        if (rc != PE_OK) return rc;
        const long long n = (long long)d_in * d_out;
        const int grid = grid_for(n / 4 + 4, di->sm_count);
        __nv_bfloat16* lp = static_cast<__nv_bfloat16*>(theta_lp);
        if (kind == OPT_ADAM) {
          switch (opt.variant) {
            case ADAM_ORIGINAL: microadam_kernel<ADAM_ORIGINAL><<<grid, OPT_THREADS, 0, st>>>(theta, lp, m, v, out_a, out_b, n, opt.adam, di->status_ptr); break;
            case ADAM_MICRO: microadam_kernel<ADAM_MICRO><<<grid, OPT_THREADS, 0, st>>>(theta, lp, m, v, out_a, out_b, n, opt.adam, di->status_ptr); break;
            case ADAM_MICRO_VAR: microadam_kernel<ADAM_MICRO_VAR><<<grid, OPT_THREADS, 0, st>>>(theta, lp, m, v, out_a, out_b, n, opt.adam, di->status_ptr); break;
            default: microadam_kernel<ADAM_MICRO_MSQ><<<grid, OPT_THREADS, 0, st>>>(theta, lp, m, v, out_a, out_b, n, opt.adam, di->status_ptr); break;
          }
        } else {
          microsignsgd_kernel<<<grid, OPT_THREADS, 0, st>>>(theta, lp, m, out_b, n, opt.sign, di->status_ptr);
        }
        return check_launch();
      }
      return launch_tc_fused(di, X, dY, B, T, d_in, d_out, kind, out_a, out_b, opt, static_cast<unsigned int*>(workspace),
                             workspace_bytes / sizeof(unsigned int), st);
    }
  }
  g_last_path.store(PE_PATH_SIMT);
  return launch_simt<TIn, MODE_STATS>(di, X, dY, B, T, d_in, d_out, kind == OPT_ADAM ? (int)PE_PHI_SQUARE : (int)PE_PHI_SIGN, out_a, out_b, st,
                                      false, SimtExtra{}, &opt);
}

static pe_status_t check_adam_args(int B, pe_adam_variant_t variant, int step) {
  if (B < 1 || step < 1) return PE_ERR_DIM;
  if ((int)variant < 0 || (int)variant > 3) return PE_ERR_PHI;
  if (((int)variant == ADAM_MICRO_VAR || (int)variant == ADAM_MICRO_MSQ) && B < 2) return PE_ERR_DIM;
  return PE_OK;
}

pe_status_t pe_linear_microadam_step(const void* X, const void* dY, int B, int T, int d_in, int d_out, float* theta, void* theta_lp,
                                     float* m, float* v, float* out_mean, float* out_stat, pe_adam_variant_t variant, float grad_scale,
                                     float lr, float beta1, float beta2, float eps, int eps_inside_sqrt, float weight_decay, int step,
                                     void* workspace, size_t workspace_bytes, pe_stream_t stream) {
  pe_status_t rc = check_adam_args(B, variant, step);
  if (rc != PE_OK) return rc;
  FusedOpt opt{};
  opt.variant = (int)variant;
  opt.adam = make_adam_params(B, grad_scale, lr, beta1, beta2, eps, eps_inside_sqrt, weight_decay, step);
  return fused_impl<__nv_bfloat16>(static_cast<const __nv_bfloat16*>(X), static_cast<const __nv_bfloat16*>(dY), B, T, d_in, d_out, OPT_ADAM,
                                   theta, theta_lp, m, v, out_mean, out_stat, opt, workspace, workspace_bytes,
                                   reinterpret_cast<cudaStream_t>(stream), true);
}

pe_status_t pe_linear_microadam_step_f32(const float* X, const float* dY, int B, int T, int d_in, int d_out, float* theta, void* theta_lp,
                                         float* m, float* v, float* out_mean, float* out_stat, pe_adam_variant_t variant,
                                         float grad_scale, float lr, float beta1, float beta2, float eps, int eps_inside_sqrt,
                                         float weight_decay, int step, pe_stream_t stream) {
  pe_status_t rc = check_adam_args(B, variant, step);
  if (rc != PE_OK) return rc;
  FusedOpt opt{};
  opt.variant = (int)variant;
  opt.adam = make_adam_params(B, grad_scale, lr, beta1, beta2, eps, eps_inside_sqrt, weight_decay, step);
  return fused_impl<float>(X, dY, B, T, d_in, d_out, OPT_ADAM, theta, theta_lp, m, v, out_mean, out_stat, opt, nullptr, 0,
                           reinterpret_cast<cudaStream_t>(stream), false);
}

pe_status_t pe_linear_microsignsgd_step(const void* X, const void* dY, int B, int T, int d_in, int d_out, float* theta, void* theta_lp,
                                        float* m, float* out_sign, float lr, float beta, float weight_decay, void* workspace,
                                        size_t workspace_bytes, pe_stream_t stream) {
  if (B < 1) return PE_ERR_DIM;
  FusedOpt opt{};
  opt.sign.inv_B = (float)(1.0 / (double)B); opt.sign.beta = beta; opt.sign.lr = lr; opt.sign.wd = weight_decay;
  return fused_impl<__nv_bfloat16>(static_cast<const __nv_bfloat16*>(X), static_cast<const __nv_bfloat16*>(dY), B, T, d_in, d_out, OPT_SIGN,
                                   theta, theta_lp, m, nullptr, nullptr, out_sign, opt, workspace, workspace_bytes,
                                   reinterpret_cast<cudaStream_t>(stream), true);
}

pe_status_t pe_linear_stats_f32(const float* X, const float* dY, int B, int T, int d_in, int d_out, pe_phi_t phi,
                                float* out_mean, float* out_stat, pe_stream_t stream) {
  return linear_stats_impl<float>(X, dY, B, T, d_in, d_out, phi, out_mean, out_stat, reinterpret_cast<cudaStream_t>(stream), false);
}

pe_status_t pe_token_sqstats(const void* X, const void* dY, int B, int T, int d_in, int d_out, float* out_stat,
                             pe_stream_t stream) {
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  if (!out_stat) return PE_ERR_NULL;
  pe_status_t rc = validate_stats(X, dY, B, T, d_in, d_out, out_stat, nullptr, false, 16);
  if (rc != PE_OK) return rc;
  DeviceInfo* di = nullptr;
  rc = device_info(&di);
  if (rc != PE_OK) return rc;
  if (B == 0 || T == 0) return zero_outputs(out_stat, nullptr, (size_t)d_in * d_out * sizeof(float), st);
  const int forced = g_path.load();
  const long long rows = (long long)B * T;
  const bool shape_ok = tc_shape_ok(B, T, d_in, d_out) && rows < (1ll << 31);
  if (forced >= PE_PATH_TENSOR && !shape_ok) return PE_ERR_UNSUPPORTED_SHAPE;
  if (shape_ok && rows >= TOKEN_TC_MIN_ROWS && forced != PE_PATH_SIMT) {
    g_last_path.store(PE_PATH_TENSOR);
    return launch_tok(di, X, dY, rows, d_in, d_out, out_stat, st);
  }
  g_last_path.store(PE_PATH_SIMT);
  return launch_simt<__nv_bfloat16, MODE_TOKEN>(di, static_cast<const __nv_bfloat16*>(X), static_cast<const __nv_bfloat16*>(dY), B, T,
                                                d_in, d_out, 0, nullptr, out_stat, st);
}

// Workspace of the staged per-token statistic: the column maxima of X and dY (one 32-bit word per
// column), then the scaled squares of X and of dY (IEEE half, or e4m3 in the fp8 form), each part 256-byte aligned.
struct StagedLayout {
  size_t max_bytes, x_bytes, y_bytes;
  size_t total() const { return max_bytes + x_bytes + y_bytes; }
};
static StagedLayout staged_layout(int B, int T, int d_in, int d_out, bool fp8 = false) {
  const size_t rows = (size_t)B * (size_t)T, es = fp8 ? 1 : 2;
  StagedLayout l;
  l.max_bytes = align_up(((size_t)d_in + (size_t)d_out) * 4, 256);
  l.x_bytes = align_up(rows * d_in * es, 256);
  l.y_bytes = align_up(rows * d_out * es, 256);
  return l;
}
// the fp8 form stages one byte per element: TMA wants 16-byte row pitches
static bool token_fp8_ok(int B, int T, int d_in, int d_out) { return token_tc_ok(B, T, d_in, d_out) && (d_in % 16) == 0 && (d_out % 16) == 0; }

size_t pe_token_sqstats_staged_workspace_bytes(int B, int T, int d_in, int d_out) {
  if (g_path.load() == PE_PATH_SIMT || !token_tc_ok(B, T, d_in, d_out)) return 0;
  return staged_layout(B, T, d_in, d_out).total();
}
size_t pe_token_sqstats_fp8_workspace_bytes(int B, int T, int d_in, int d_out) {
  if (g_path.load() == PE_PATH_SIMT || !token_tc_ok(B, T, d_in, d_out)) return 0;
  return staged_layout(B, T, d_in, d_out, token_fp8_ok(B, T, d_in, d_out)).total();
}

// Grid of the column-wise staging kernels: x covers the columns in groups of 256, y slices the rows
// so that the whole grid is a few blocks per SM.
static dim3 stage_grid(long long rows, int d, int sm_count) {
  const int gx = (d + 255) / 256;
  long long gy = ((long long)sm_count * 8 + gx - 1) / gx;
  const long long max_gy = rows / 64 > 0 ? rows / 64 : 1;
  if (gy > max_gy) gy = max_gy;
  if (gy > 65535) gy = 65535;
  if (gy < 1) gy = 1;
  return dim3((unsigned)gx, (unsigned)gy, 1);
}

// The plain contraction of e4m3 operands x8 [B, T, d_in], y8 [B, T, d_out] (one byte per element) into out.
static pe_status_t launch_tc_fp8(DeviceInfo* di, const void* x8, const void* y8, int B, int T, int d_in, int d_out, float* out,
                                 cudaStream_t st) {
  using Op = TcOperand<false, 256, 128, true>;
  EncodeTiledFn enc = encode_fn();
  if (!enc) return PE_ERR_CUDA;
  auto operand_map = [&](CUtensorMap* m, const void* base, int d) {
    cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)T, (cuuint64_t)B};
    cuuint64_t strides[2] = {(cuuint64_t)d, (cuuint64_t)T * (cuuint64_t)d};
    cuuint32_t box[3] = {(cuuint32_t)Op::BOX_FEATS, (cuuint32_t)Op::BK, 1u};
    cuuint32_t estr[3] = {1u, 1u, 1u};
    return enc(m, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
               CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
  };
  CUtensorMap mx, my, mo;
  if (!operand_map(&mx, x8, d_in) || !operand_map(&my, y8, d_out)) return PE_ERR_CUDA;
  pe_status_t rc = make_output_map(&mo, out, d_in, d_out);
  if (rc != PE_OK) return rc;
  const int tiles_n = (d_in + 255) / 256, pairs_m = (d_out + TC_PAIR_M - 1) / TC_PAIR_M;
  if ((long long)tiles_n * pairs_m > (1ll << 29)) return PE_ERR_DIM;
  const int ns = choose_nsplit((long long)tiles_n * pairs_m, B, T, di->sm_count / 2 > 0 ? di->sm_count / 2 : 1, 16);
  if (ns > 1) {
    rc = zero_for_split(di, out, nullptr, (size_t)d_in * d_out, st);
    if (rc != PE_OK) return rc;
  }
  TcParams p;
  p.B = B; p.T = T; p.d_in = d_in; p.d_out = d_out; p.nsplit = ns; p.per_example = 0; p.half_operands = 0; p.accumulate = 0;
  p.pairs_m = pairs_m; p.tiles_n = tiles_n; p.band = choose_band(pairs_m, tiles_n, 256, ns, di->sm_count / 2);
  p.out_mean = nullptr; p.out_stat = out; p.out_sign = nullptr; p.out_norms = nullptr; p.dev_status = di->status_ptr;
  p.seq_offsets = nullptr; p.sq_norms = nullptr; p.clip_norm = 0.f;
  return launch_tc_inst<0, false, 256, MEAN_NONE, 128, false, OPT_NONE, true>(di, 25, mx, my, mo, mo, mo, p, dim3(2 * pairs_m * tiles_n, 1, ns), st);
}

// The two-pass per-token statistic on half (fp8 = false) or e4m3 (fp8 = true) squares.
static pe_status_t token_staged_impl(const void* X, const void* dY, int B, int T, int d_in, int d_out, float* out_stat, void* workspace,
                                     size_t workspace_bytes, cudaStream_t st, bool want_fp8) {
  if (!out_stat) return PE_ERR_NULL;
  pe_status_t rc = validate_stats(X, dY, B, T, d_in, d_out, out_stat, nullptr, false, 16);
  if (rc != PE_OK) return rc;
  DeviceInfo* di = nullptr;
  rc = device_info(&di);
  if (rc != PE_OK) return rc;
  if (B == 0 || T == 0) return zero_outputs(out_stat, nullptr, (size_t)d_in * d_out * sizeof(float), st);
  const int forced = g_path.load();
  const bool tc_ok = token_tc_ok(B, T, d_in, d_out);
  if (forced >= PE_PATH_TENSOR && !tc_shape_ok(B, T, d_in, d_out)) return PE_ERR_UNSUPPORTED_SHAPE;
  if (tc_ok && forced != PE_PATH_SIMT) {
    const bool fp8 = want_fp8 && token_fp8_ok(B, T, d_in, d_out);
    const long long rows = (long long)B * T;
    const StagedLayout l = staged_layout(B, T, d_in, d_out, fp8);
    if (!workspace || workspace_bytes < l.total()) return PE_ERR_WORKSPACE;
    if (!aligned(workspace, 256)) return PE_ERR_ALIGN;
    uint32_t* max_x = static_cast<uint32_t*>(workspace);
    uint32_t* max_y = max_x + d_in;
    void* x2 = static_cast<char*>(workspace) + l.max_bytes;
    void* y2 = static_cast<char*>(workspace) + l.max_bytes + l.x_bytes;
    const uint16_t* Xb = static_cast<const uint16_t*>(X);
    const uint16_t* Yb = static_cast<const uint16_t*>(dY);
    if (cudaMemsetAsync(max_x, 0, ((size_t)d_in + (size_t)d_out) * 4, st) != cudaSuccess) { cudaGetLastError(); return PE_ERR_CUDA; }
    // one launch per pass serves both tensors (gridDim.z picks X or dY; the grid is sized for the wider one)
    dim3 grid = stage_grid(rows, d_in > d_out ? d_in : d_out, di->sm_count);
    grid.y = (grid.y + 1) / 2;
    grid.z = 2;
    const StageTensor sx = {Xb, x2, max_x, d_in}, sy = {Yb, y2, max_y, d_out};
    column_max_kernel<<<grid, STAGE_THREADS, 0, st>>>(sx, sy, rows);
    if ((rc = check_launch()) != PE_OK) return rc;
    if (fp8) square_to_lp_kernel<true><<<grid, STAGE_THREADS, 0, st>>>(sx, sy, rows);
    else square_to_lp_kernel<false><<<grid, STAGE_THREADS, 0, st>>>(sx, sy, rows);
    if ((rc = check_launch()) != PE_OK) return rc;
    // B and T only enter through B*T: regroup the rows into two-stage "examples" when possible so
    // the batch split has many units to balance.
    const int regroup = fp8 ? 2 * TcOperand<false, 256, 128, true>::BK : 2 * TcOperand<false, 256>::BK;
    int Bp = B, Tp = T;
    if (T % regroup == 0 && rows / regroup < (1ll << 30)) { Bp = (int)(rows / regroup); Tp = regroup; }
    g_last_path.store(PE_PATH_TENSOR);
    rc = fp8 ? launch_tc_fp8(di, x2, y2, Bp, Tp, d_in, d_out, out_stat, st)
             : launch_tc(di, x2, y2, Bp, Tp, d_in, d_out, PE_PHI_IDENTITY, 0, nullptr, out_stat, st, true);
    if (rc != PE_OK) return rc;
    const int ugrid = grid_for((long long)d_in * d_out / 4 + 4, di->sm_count);
    if (fp8) unscale_kernel<true><<<ugrid, STAGE_THREADS, 0, st>>>(out_stat, d_out, d_in, max_x, max_y);
    else unscale_kernel<false><<<ugrid, STAGE_THREADS, 0, st>>>(out_stat, d_out, d_in, max_x, max_y);
    return check_launch();
  }
  g_last_path.store(PE_PATH_SIMT);
  return launch_simt<__nv_bfloat16, MODE_TOKEN>(di, static_cast<const __nv_bfloat16*>(X), static_cast<const __nv_bfloat16*>(dY), B, T,
                                                d_in, d_out, 0, nullptr, out_stat, st);
}

pe_status_t pe_token_sqstats_staged(const void* X, const void* dY, int B, int T, int d_in, int d_out, float* out_stat,
                                    void* workspace, size_t workspace_bytes, pe_stream_t stream) {
  return token_staged_impl(X, dY, B, T, d_in, d_out, out_stat, workspace, workspace_bytes, reinterpret_cast<cudaStream_t>(stream), false);
}

pe_status_t pe_token_sqstats_fp8(const void* X, const void* dY, int B, int T, int d_in, int d_out, float* out_stat,
                                 void* workspace, size_t workspace_bytes, pe_stream_t stream) {
  return token_staged_impl(X, dY, B, T, d_in, d_out, out_stat, workspace, workspace_bytes, reinterpret_cast<cudaStream_t>(stream), true);
}

// ---------------------------------------------------------------------------------------------
// Allocation-free per-token statistic.  The staging buffer is a device array inside this module's
// image.  In host code its name is only a handle for the runtime's symbol lookups, never a device
// address: the address each device gave the array is looked up once per device (with that device
// current) and cached; that looked-up pointer is what the kernels receive.
static __device__ __align__(256) unsigned char g_static_scratch[PE_STATIC_SCRATCH_BYTES];

struct StaticScratchSlot {
  std::atomic<int> ready{0};
  void* ptr = nullptr;
};
static StaticScratchSlot g_static_slot[MAX_DEVICES];

static pe_status_t static_scratch_ptr(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) { cudaGetLastError(); return PE_ERR_CUDA; }
  StaticScratchSlot& slot = g_static_slot[dev];
  if (!slot.ready.load(std::memory_order_acquire)) {
    void* p = nullptr;
    if (cudaGetSymbolAddress((void**)&p, g_static_scratch) != cudaSuccess || !p) { cudaGetLastError(); return PE_ERR_CUDA; }
    slot.ptr = p;                       // concurrent first calls look up the same address
    slot.ready.store(1, std::memory_order_release);
  }
  *out = slot.ptr;
  return PE_OK;
}

pe_status_t pe_token_sqstats_static(const void* X, const void* dY, int B, int T, int d_in, int d_out, float* out_stat,
                                    pe_stream_t stream) {
  if (!out_stat) return PE_ERR_NULL;
  pe_status_t rc = validate_stats(X, dY, B, T, d_in, d_out, out_stat, nullptr, false, 16);
  if (rc != PE_OK) return rc;
  // Refuse what does not fit before touching the device.
  if (pe_token_sqstats_staged_workspace_bytes(B, T, d_in, d_out) > (size_t)PE_STATIC_SCRATCH_BYTES) return PE_ERR_WORKSPACE;
  DeviceInfo* di = nullptr;
  rc = device_info(&di);
  if (rc != PE_OK) return rc;
  void* scratch = nullptr;
  rc = static_scratch_ptr(&scratch);
  if (rc != PE_OK) return rc;
  // Nothing in the array has to start at zero: the squaring pre-pass rewrites every element the
  // contraction reads.  Everything below only enqueues kernels and memsets on `stream`.
  return pe_token_sqstats_staged(X, dY, B, T, d_in, d_out, out_stat, scratch, (size_t)PE_STATIC_SCRATCH_BYTES, stream);
}

pe_status_t pe_token_sqstats_f32(const float* X, const float* dY, int B, int T, int d_in, int d_out, float* out_stat,
                                 pe_stream_t stream) {
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  if (!out_stat) return PE_ERR_NULL;
  pe_status_t rc = validate_stats(X, dY, B, T, d_in, d_out, out_stat, nullptr, false, 4);
  if (rc != PE_OK) return rc;
  DeviceInfo* di = nullptr;
  rc = device_info(&di);
  if (rc != PE_OK) return rc;
  if (B == 0 || T == 0) return zero_outputs(out_stat, nullptr, (size_t)d_in * d_out * sizeof(float), st);
  g_last_path.store(PE_PATH_SIMT);
  return launch_simt<float, MODE_TOKEN>(di, X, dY, B, T, d_in, d_out, 0, nullptr, out_stat, st);
}

pe_status_t microadam_family_step(float* theta, void* theta_lp, float* m, float* v, const float* sum_g, const float* sum_g2,
                                  long long n, int B, pe_adam_variant_t variant, float grad_scale, float lr, float beta1,
                                  float beta2, float eps, int eps_inside_sqrt, float weight_decay, int step,
                                  pe_stream_t stream) {
  if (!theta || !m || !v || !sum_g || !sum_g2) return PE_ERR_NULL;
  if (n < 0 || B < 1 || step < 1) return PE_ERR_DIM;
  if ((int)variant < 0 || (int)variant > 3) return PE_ERR_PHI;
  if (((int)variant == ADAM_MICRO_VAR || (int)variant == ADAM_MICRO_MSQ) && B < 2) return PE_ERR_DIM;   // a variance needs two examples
  if (!aligned(theta, 16) || !aligned(m, 16) || !aligned(v, 16) || !aligned(sum_g, 16) || !aligned(sum_g2, 16) ||
      (theta_lp && !aligned(theta_lp, 16)))
    return PE_ERR_ALIGN;
  DeviceInfo* di = nullptr;
  pe_status_t rc = device_info(&di);
  if (rc != PE_OK) return rc;
  if (n == 0) return PE_OK;
  const AdamParams p = make_adam_params(B, grad_scale, lr, beta1, beta2, eps, eps_inside_sqrt, weight_decay, step);
  const int grid = grid_for(n / 4 + 4, di->sm_count);
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  __nv_bfloat16* lp = static_cast<__nv_bfloat16*>(theta_lp);
  switch ((int)variant) {
    case ADAM_ORIGINAL: microadam_kernel<ADAM_ORIGINAL><<<grid, OPT_THREADS, 0, st>>>(theta, lp, m, v, sum_g, sum_g2, n, p); break;
    case ADAM_MICRO: microadam_kernel<ADAM_MICRO><<<grid, OPT_THREADS, 0, st>>>(theta, lp, m, v, sum_g, sum_g2, n, p); break;
    case ADAM_MICRO_VAR: microadam_kernel<ADAM_MICRO_VAR><<<grid, OPT_THREADS, 0, st>>>(theta, lp, m, v, sum_g, sum_g2, n, p); break;
    default: microadam_kernel<ADAM_MICRO_MSQ><<<grid, OPT_THREADS, 0, st>>>(theta, lp, m, v, sum_g, sum_g2, n, p); break;
  }
  return check_launch();
}

pe_status_t microadam_step(float* theta, void* theta_lp, float* m, float* v, const float* sum_g, const float* sum_g2,
                           long long n, int B, float grad_scale, float lr, float beta1, float beta2, float eps,
                           int eps_inside_sqrt, float weight_decay, int step, pe_stream_t stream) {
  return microadam_family_step(theta, theta_lp, m, v, sum_g, sum_g2, n, B, PE_ADAM_MICRO, grad_scale, lr, beta1, beta2, eps,
                               eps_inside_sqrt, weight_decay, step, stream);
}

pe_status_t microsignsgd_step(float* theta, void* theta_lp, float* m, const float* sum_sign, long long n, int B, float lr,
                              float beta, float weight_decay, pe_stream_t stream) {
  if (!theta || !m || !sum_sign) return PE_ERR_NULL;
  if (n < 0 || B < 1) return PE_ERR_DIM;
  if (!aligned(theta, 16) || !aligned(m, 16) || !aligned(sum_sign, 16) || (theta_lp && !aligned(theta_lp, 16))) return PE_ERR_ALIGN;
  DeviceInfo* di = nullptr;
  pe_status_t rc = device_info(&di);
  if (rc != PE_OK) return rc;
  if (n == 0) return PE_OK;
  SignParams p;
  p.inv_B = (float)(1.0 / (double)B); p.beta = beta; p.lr = lr; p.wd = weight_decay;
  microsignsgd_kernel<<<grid_for(n / 4 + 4, di->sm_count), OPT_THREADS, 0, reinterpret_cast<cudaStream_t>(stream)>>>(
      theta, static_cast<__nv_bfloat16*>(theta_lp), m, sum_sign, n, p);
  return check_launch();
}

const char* pe_status_string(pe_status_t s) {
  switch (s) {
    case PE_OK: return "PE_OK";
    case PE_ERR_NULL: return "PE_ERR_NULL";
    case PE_ERR_DIM: return "PE_ERR_DIM";
    case PE_ERR_ALIGN: return "PE_ERR_ALIGN";
    case PE_ERR_UNSUPPORTED_SHAPE: return "PE_ERR_UNSUPPORTED_SHAPE";
    case PE_ERR_PHI: return "PE_ERR_PHI";
    case PE_ERR_ARCH: return "PE_ERR_ARCH";
    case PE_ERR_CUDA: return "PE_ERR_CUDA";
    case PE_ERR_TIMEOUT: return "PE_ERR_TIMEOUT";
    case PE_ERR_WORKSPACE: return "PE_ERR_WORKSPACE";
  }
  return "PE_ERR_UNKNOWN";
}

pe_status_t pe_get_async_status(pe_stream_t stream, int* detail) {
  if (detail) *detail = 0;
  DeviceInfo* di = nullptr;
  pe_status_t rc = device_info(&di);
  if (rc != PE_OK) return rc;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  if (cudaStreamSynchronize(st) != cudaSuccess) { cudaGetLastError(); return PE_ERR_CUDA; }
  unsigned int word = 0;
  if (cudaMemcpy(&word, di->status_ptr, sizeof word, cudaMemcpyDeviceToHost) != cudaSuccess) { cudaGetLastError(); return PE_ERR_CUDA; }
  if (word == 0) return PE_OK;
  if (cudaMemset(di->status_ptr, 0, sizeof word) != cudaSuccess) { cudaGetLastError(); return PE_ERR_CUDA; }
  if (detail) *detail = (int)word;
  return PE_ERR_TIMEOUT;
}

pe_status_t pe_set_wait_limit_cycles(long long cycles) {
  DeviceInfo* di = nullptr;
  pe_status_t rc = device_info(&di);
  if (rc != PE_OK) return rc;
  const long long v = cycles > 0 ? cycles : sm100::WAIT_CYCLE_LIMIT_DEFAULT;
  if (cudaMemcpyToSymbol(sm100::g_wait_cycle_limit, &v, sizeof v) != cudaSuccess) { cudaGetLastError(); return PE_ERR_CUDA; }
  return PE_OK;
}

int pe_set_fused_update(int mode) {
  if (mode < PE_FUSED_AUTO || mode > PE_FUSED_NEVER) return -1;
  return g_fused_mode.exchange(mode);
}

int pe_set_path(int path) {
  if (path < PE_PATH_AUTO || path > PE_PATH_TENSOR_WIDE) return -1;
  return g_path.exchange(path);
}
int pe_tile_order_band(int d_in, int d_out, int tile_cols, int batch_slices, int sm_count) {
  if (d_in < 1 || d_out < 1 || batch_slices < 1 || sm_count < 2) return 0;
  if (tile_cols != 128 && tile_cols != 192 && tile_cols != 256) return 0;
  const long long tiles_n = ((long long)d_in + tile_cols - 1) / tile_cols, pairs_m = ((long long)d_out + pe::TC_PAIR_M - 1) / pe::TC_PAIR_M;
  if (tiles_n * pairs_m > (1ll << 29)) return 0;
  return pe::choose_band((int)pairs_m, (int)tiles_n, tile_cols, batch_slices, sm_count / 2);
}
int pe_last_path(void) { return g_last_path.load(); }
long long pe_launch_count(void) { return g_launches.load(); }
void pe_reset_launch_count(void) { g_launches.store(0); }

}  // extern "C"
