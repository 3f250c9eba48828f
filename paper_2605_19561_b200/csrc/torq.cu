// C-ABI entry points of the library (see include/torq.h): argument validation, TMA descriptor
// encoding, kernel selection and launch.  Nothing here computes on the host.
#include <cuda.h>
#include <cuda_runtime.h>
#include <atomic>
#include <mutex>

#include "../../include/torq.h"
#include "mxfp4_gemm.cuh"
#include "mxfp4_gemm_pair.cuh"
#include "quantize.cuh"
#include "nvfp4_quantize.cuh"
#include "mxint4_quantize.cuh"
#include "rotate_quantize.cuh"
#include "rotate_quantize_pair.cuh"
#include "rotate_splitk.cuh"
#include "rotate_fewtok.cuh"
#include "gemm_fewtok.cuh"
#include "rotate_structured.cuh"
#include "fp4_peak_probe.cuh"
#include "calibrate.cuh"
#include "wait_selftest.cuh"
#include "prepare_weights.cuh"
#include "sm100_ptx.cuh"

namespace torq {

__device__ int g_error_word = 0;

constexpr int kMaxDevices = 64;
struct DeviceState {
  bool ready = false;
  bool arch_ok = false;
  int sm_count = 0;
  int rot_pairs = 0;    // CTA pairs of the pair kernels that can be resident at once
  int gemm_pairs = 0;
  int* err_word = nullptr;
};
static DeviceState g_dev[kMaxDevices];
static std::mutex g_mutex;
static std::atomic<int64_t> g_launches{0};

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                   const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                   const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn g_encode = nullptr;

template <typename K>
static bool opt_in_smem(K kernel, int bytes) {
  return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) ==
         cudaSuccess;
}

// How many 2-CTA clusters of `kernel` fit on the device at once (GPC boundaries can leave a few
// SMs unpaired, so this may be below sm_count / 2).
template <typename K>
static int max_active_pairs(K kernel, int threads, int smem, int sm_count) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(sm_count / 2 * 2), 1, 1);
  cfg.blockDim = dim3((unsigned)threads, 1, 1);
  cfg.dynamicSmemBytes = (size_t)smem;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, kernel, &cfg) != cudaSuccess) return 0;
  return n < sm_count / 2 ? n : sm_count / 2;
}

// Per-device one-time set-up: architecture check, SM count, error-word address, shared-memory
// opt-in of the tensor-core kernels.  Returns nullptr when CUDA itself fails.
static DeviceState* device_state() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  std::lock_guard<std::mutex> lock(g_mutex);
  DeviceState& st = g_dev[dev];
  if (st.ready) return &st;
  int major = 0;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
    return nullptr;
  if (cudaDeviceGetAttribute(&st.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return nullptr;
  st.arch_ok = (major == 10);
  if (st.arch_ok) {
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&st.err_word), g_error_word) != cudaSuccess)
      return nullptr;
    if (!g_encode) {
      void* fn = nullptr;
      cudaDriverEntryPointQueryResult qres;
      if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) !=
              cudaSuccess || qres != cudaDriverEntryPointSuccess || fn == nullptr)
        return nullptr;
      g_encode = reinterpret_cast<EncodeTiledFn>(fn);
    }
    bool ok = opt_in_smem(mxfp4_gemm_kernel<256, 1>, GemmCfg<256, 1>::SMEM_BYTES) &&
              opt_in_smem(mxfp4_gemm_kernel<128, 2>, GemmCfg<128, 2>::SMEM_BYTES) &&
              opt_in_smem(mxfp4_gemm_kernel<256, 1, FMT_NVFP4>, GemmCfg<256, 1, FMT_NVFP4>::SMEM_BYTES) &&
              opt_in_smem(mxfp4_gemm_kernel<128, 2, FMT_NVFP4>, GemmCfg<128, 2, FMT_NVFP4>::SMEM_BYTES) &&
              opt_in_smem(rotate_quantize_kernel<256>, RotCfg<256>::SMEM_BYTES) &&
              opt_in_smem(rotate_quantize_kernel<128>, RotCfg<128>::SMEM_BYTES) &&
              opt_in_smem(rotate_quantize_kernel<256, FMT_NVFP4>, RotCfg<256>::SMEM_BYTES) &&
              opt_in_smem(rotate_quantize_pair_kernel<FMT_MXFP4>, RotPairCfg::SMEM_BYTES) &&
              opt_in_smem(rotate_quantize_pair_kernel<FMT_NVFP4>, RotPairCfg::SMEM_BYTES) &&
              opt_in_smem(rotate_splitk_kernel, RotSplitCfg::SMEM_BYTES) &&
              opt_in_smem(rotate_structured_kernel<FMT_MXFP4>, RotStructCfg::SMEM_BYTES) &&
              opt_in_smem(rotate_structured_kernel<FMT_NVFP4>, RotStructCfg::SMEM_BYTES) &&
              opt_in_smem(mxfp4_gemm_pair_kernel<FMT_MXFP4>, GemmPairCfg::SMEM_BYTES) &&
              opt_in_smem(mxfp4_gemm_pair_kernel<FMT_NVFP4>, GemmPairCfgT<FMT_NVFP4>::SMEM_BYTES) &&
              opt_in_smem(mxfp4_gemm_kernel<256, 1, FMT_MXINT4>, GemmCfg<256, 1, FMT_MXINT4>::SMEM_BYTES) &&
              opt_in_smem(mxfp4_gemm_kernel<128, 2, FMT_MXINT4>, GemmCfg<128, 2, FMT_MXINT4>::SMEM_BYTES) &&
              opt_in_smem(mxfp4_gemm_pair_kernel<FMT_MXINT4>, GemmPairCfgT<FMT_MXINT4>::SMEM_BYTES) &&
              opt_in_smem(rotate_quantize_kernel<256, FMT_MXINT4>, RotCfg<256>::SMEM_BYTES) &&
              opt_in_smem(rotate_quantize_pair_kernel<FMT_MXINT4>, RotPairCfg::SMEM_BYTES) &&
              opt_in_smem(rotate_structured_kernel<FMT_MXINT4>, RotStructCfg::SMEM_BYTES) &&
              opt_in_smem(rotate_fewtok_kernel<FMT_MXFP4, 1>, RotFewCfg::max_smem_bytes()) &&
              opt_in_smem(rotate_fewtok_kernel<FMT_MXFP4, 2>, RotFewCfg::max_smem_bytes()) &&
              opt_in_smem(rotate_fewtok_kernel<FMT_NVFP4, 1>, RotFewCfg::max_smem_bytes()) &&
              opt_in_smem(rotate_fewtok_kernel<FMT_NVFP4, 2>, RotFewCfg::max_smem_bytes()) &&
              opt_in_smem(rotate_fewtok_kernel<FMT_MXINT4, 1>, RotFewCfg::max_smem_bytes()) &&
              opt_in_smem(rotate_fewtok_kernel<FMT_MXINT4, 2>, RotFewCfg::max_smem_bytes()) &&
              opt_in_smem(gemm_fewtok_kernel<FMT_MXFP4, 1>, GemmFewCfg<FMT_MXFP4>::max_smem_bytes()) &&
              opt_in_smem(gemm_fewtok_kernel<FMT_MXFP4, 2>, GemmFewCfg<FMT_MXFP4>::max_smem_bytes()) &&
              opt_in_smem(gemm_fewtok_kernel<FMT_NVFP4, 1>, GemmFewCfg<FMT_NVFP4>::max_smem_bytes()) &&
              opt_in_smem(gemm_fewtok_kernel<FMT_NVFP4, 2>, GemmFewCfg<FMT_NVFP4>::max_smem_bytes()) &&
              opt_in_smem(gemm_fewtok_kernel<FMT_MXINT4, 1>, GemmFewCfg<FMT_MXINT4>::max_smem_bytes()) &&
              opt_in_smem(gemm_fewtok_kernel<FMT_MXINT4, 2>, GemmFewCfg<FMT_MXINT4>::max_smem_bytes()) &&
              opt_in_smem(rotate_quantize_kernel<256, FMT_F32OUT>, RotCfg<256>::SMEM_BYTES) &&
              opt_in_smem(rotate_quantize_pair_kernel<FMT_F32OUT>, RotPairCfg::SMEM_BYTES);
    if (!ok) return nullptr;
    st.rot_pairs = max_active_pairs(rotate_quantize_pair_kernel<FMT_MXFP4>, RotPairCfg::THREADS,
                                    RotPairCfg::SMEM_BYTES, st.sm_count);
    st.gemm_pairs = max_active_pairs(mxfp4_gemm_pair_kernel<FMT_NVFP4>, GemmPairCfg::THREADS,
                                     GemmPairCfgT<FMT_NVFP4>::SMEM_BYTES, st.sm_count);
    if (st.rot_pairs < 1 || st.gemm_pairs < 1) return nullptr;
    cudaGetLastError();
  }
  st.ready = true;
  return &st;
}

// 2-D row-major tensor [rows, cols] of `elem_bytes`-byte elements, box [box_rows, box_cols],
// 128-byte swizzle, zero fill outside the tensor.
static bool encode_2d(CUtensorMap* map, CUtensorMapDataType dt, int elem_bytes, const void* base,
                      uint64_t rows, uint64_t cols, uint32_t box_rows, uint32_t box_cols,
                      CUtensorMapSwizzle swizzle = CU_TENSOR_MAP_SWIZZLE_128B) {
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {cols * (uint64_t)elem_bytes};
  cuuint32_t box[2] = {box_cols, box_rows};
  cuuint32_t estr[2] = {1, 1};
  return g_encode(map, dt, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// X [M, d] bf16 seen as (position k: 32, token: M, block: d/32) with box (32, 1, 64): the box lands
// in shared memory as 64 rows (blocks) of 64 bytes (one token's 32 positions), 64-byte swizzle.
static bool encode_x_blocks_3d(CUtensorMap* map, const void* base, uint64_t M, uint64_t d) {
  cuuint64_t dims[3] = {32, M, d / 32};
  cuuint64_t strides[2] = {d * 2, 64};
  cuuint32_t box[3] = {32, 1, 64};
  cuuint32_t estr[3] = {1, 1, 1};
  return g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

static inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static inline int ew_grid(int64_t items, int per_block, int sm_count) {
  int64_t blocks = (items + per_block - 1) / per_block;
  int64_t cap = (int64_t)sm_count * 16;
  return (int)(blocks < 1 ? 1 : (blocks > cap ? cap : blocks));
}
static inline torq_status launch_status() {
  g_launches.fetch_add(1, std::memory_order_relaxed);
  return cudaGetLastError() == cudaSuccess ? TORQ_OK : TORQ_ERR_LAUNCH;
}

// Launch of a persistent tensor-core kernel: `cluster` CTAs per cluster along x (1 or 2; the grid
// is a multiple of it) and programmatic stream serialization, so that the launch processing of
// this kernel overlaps the tail of the kernel before it (the kernel itself waits for that kernel
// to complete before it touches global memory).
template <typename... KArgs, typename... Args>
static void launch_tc(void (*kernel)(KArgs...), int cluster, int grid, int threads, int smem, cudaStream_t s,
                      Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid, 1, 1);
  cfg.blockDim = dim3((unsigned)threads, 1, 1);
  cfg.dynamicSmemBytes = (size_t)smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = (unsigned)cluster;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = cluster > 1 ? 2 : 1;
  cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// K splits of the few-token rotation: as many as fill the SMs, each at least two 64-element steps.
// `sm_count` <= 0 gives the bound used for sizing workspaces (any device up to 160 SMs).
static int rotation_splits(int64_t M, int64_t d, int sm_count) {
  const int64_t tiles = ((M + 127) / 128) * ((d + 255) / 256);
  const int sms = sm_count > 0 ? sm_count : 160;
  if (2 * tiles > sms) return 1;
  const int k_tiles = (int)((d + 63) / 64);
  int s = (int)(sms / tiles);
  if (s > RotSplitCfg::MAX_SPLITS) s = RotSplitCfg::MAX_SPLITS;
  if (s > k_tiles / 2) s = k_tiles / 2;
  return s < 2 ? 1 : s;
}
constexpr int kRotFewMaxTokens = 256;    // up to here the rotation streams R_inter through the few-token kernel
constexpr int kGemmFewMaxTokens = 128;   // and the GEMM the weights
static_assert(kRotFewMaxTokens <= RotFewCfg::MAX_TOK && kGemmFewMaxTokens <= GemmFewCfg<FMT_MXFP4>::MAX_TOK, "few-token limits");
// Few-token kernels: tokens per instruction and the cluster size = number of K splits of
// one 128-feature tile.  Two of these CTAs fit on an SM, and a grid of about 1.4 CTAs per SM measured
// fastest (more loads in flight; beyond that the clusters no longer all become resident at once):
// the largest S <= 8 with tiles * S <= 1.4 SMs, each split at least `min_k` K steps.  7 is skipped:
// clusters of 7 did not all become resident at sizes where 6 and 8 did.
static inline int fewtok_ntok(int64_t M) { return M <= 16 ? 16 : (M <= 32 ? 32 : (M <= 64 ? 64 : (M <= 128 ? 128 : 256))); }
static inline int fewtok_cluster(int64_t tiles, int64_t k_steps, int min_k, int sm_count, int ctas_per_sm) {
  // two CTAs fit on an SM: 1.4 per SM on average keeps the most bytes in flight; one: one wave
  int64_t s = (int64_t)sm_count * (ctas_per_sm >= 2 ? 14 : 10) / 10 / (tiles > 0 ? tiles : 1);
  if (s > 8) s = 8;
  if (s > k_steps / min_k) s = k_steps / min_k;
  if (s == 7) s = 6;
  return s < 1 ? 1 : (int)s;
}
constexpr double kNarrowTileCost = 0.88;   // a 192-column tile against a 256-column one: 0.75 of the math, 0.875 of the operand bytes

// Tile list of a pair kernel: `rows` 256-row tiles by `cols` columns on `max_pairs` CTA pairs, tiles dealt
// round robin.  When the 256-column tiles do not fill the last wave, trading three of them for four 192-column
// tiles (one unit) in some row tiles shortens that wave from one tile time to about three quarters.  The number
// of units is the one with the smallest longest-pair time, a narrow tile counted as `narrow_cost` wide tiles;
// zero unless it wins by at least 1 % (and always zero when the columns are not whole 256-column tiles).
static MixedTiles plan_pair_tiles(int rows, int64_t cols, int max_pairs, double narrow_cost) {
  const int wide_cols = (int)((cols + 255) / 256);
  if (cols % 256 != 0 || rows < 1) return mixed_tiles_make(rows < 1 ? 1 : rows, wide_cols, 0);
  struct Memo { int rows, wide_cols, max_pairs; double cost; int units; };
  static thread_local Memo memo[8] = {};
  static thread_local int memo_next = 0;
  for (const Memo& m : memo)
    if (m.rows == rows && m.wide_cols == wide_cols && m.max_pairs == max_pairs && m.cost == narrow_cost)
      return mixed_tiles_make(rows, wide_cols, m.units);
  auto longest = [&](int units) {
    const int wide = rows * wide_cols - 3 * units, narrow = 4 * units;
    const int P = wide + narrow < max_pairs ? wide + narrow : max_pairs;
    double worst = 0.0;
    for (int p = 0; p < P; ++p) {
      const int w = wide / P + (p < wide % P ? 1 : 0);
      // narrow tiles have the numbers wide .. wide + narrow - 1; pair p takes those congruent to p
      const int first = wide + ((p - wide) % P + P) % P;
      const int n = first < wide + narrow ? (wide + narrow - 1 - first) / P + 1 : 0;
      const double t = w + narrow_cost * n;
      if (t > worst) worst = t;
    }
    return worst;
  };
  const int max_units = rows * (wide_cols / 3);
  const double base = longest(0);
  double best = base;
  int best_units = 0;
  for (int u = 1; u <= max_units && 4 * u <= max_pairs + 8; ++u) {
    // the row tiles that trade one unit more must have the three wide tiles to give
    if (u % rows != 0 && 3 * (u / rows + 1) > wide_cols) break;
    const double t = longest(u);
    if (t < best - 1e-9) { best = t; best_units = u; }
  }
  if (best > 0.99 * base) best_units = 0;
  memo[memo_next] = Memo{rows, wide_cols, max_pairs, narrow_cost, best_units};
  memo_next = (memo_next + 1) % 8;
  return mixed_tiles_make(rows, wide_cols, best_units);
}

static size_t quantized_bytes(int64_t M, int64_t d) {    // codes, then 256-byte aligned the scales
  return ((size_t)M * (size_t)(d / 2) + 255) / 256 * 256 + torq_scales_bytes(M, d);
}
static size_t splitk_scratch_bytes(int64_t M, int64_t d, int splits) {
  return splits < 2 ? 0 : (size_t)splits * (size_t)((M + 127) / 128 * 128) * (size_t)d * sizeof(float);
}

static torq_status quantize_impl(DeviceState* st, const void* Z, torq_dtype dt, int64_t M, int64_t d,
                                 void* codes, void* scales, cudaStream_t s) {
  const int64_t kb4 = (d / 32 + 3) / 4;
  const int64_t items = ((M + 127) / 128 * 128) * ((kb4 * 128 + 255) / 256);   // warps
  const int grid = ew_grid(items, 8, st->sm_count);
  if (dt == TORQ_F32)
    quantize_kernel<float><<<grid, 256, 0, s>>>(static_cast<const float*>(Z), M, d,
                                                static_cast<uint8_t*>(codes), static_cast<uint8_t*>(scales));
  else
    quantize_kernel<__nv_bfloat16><<<grid, 256, 0, s>>>(static_cast<const __nv_bfloat16*>(Z), M, d,
                                                        static_cast<uint8_t*>(codes),
                                                        static_cast<uint8_t*>(scales));
  return launch_status();
}

}  // namespace torq

using namespace torq;

extern "C" {

size_t torq_scales_bytes(int64_t rows, int64_t k) {
  if (rows <= 0 || k <= 0) return 0;
  return (size_t)((rows + 127) / 128) * (size_t)((k / 32 + 3) / 4) * 512;
}

size_t torq_scale_offset(int64_t row, int64_t kblock, int64_t k) {
  return scale_offset(row, kblock, (k / 32 + 3) / 4);
}

size_t torq_workspace_bytes(int64_t M, int64_t d, int64_t N) {
  (void)N;
  if (M <= 0 || d <= 0) return 0;
  return quantized_bytes(M, d) + splitk_scratch_bytes(M, d, rotation_splits(M, d, 0));
}

const char* torq_status_string(torq_status s) {
  switch (s) {
    case TORQ_OK: return "ok";
    case TORQ_ERR_NULL: return "null pointer";
    case TORQ_ERR_SHAPE: return "unsupported shape";
    case TORQ_ERR_ALIGN: return "pointer not 16-byte aligned";
    case TORQ_ERR_ARCH: return "device is not compute capability 10.x";
    case TORQ_ERR_LAUNCH: return "CUDA launch or descriptor error";
    case TORQ_ERR_TIMEOUT: return "a bounded device wait ran out";
    case TORQ_ERR_WORKSPACE: return "workspace missing or too small";
  }
  return "unknown";
}

int64_t torq_pair_tile_list(int64_t rows, int64_t cols, int32_t pairs, int32_t* out, int64_t cap) {
  if (rows < 1 || cols < 1 || pairs < 1 || rows > INT32_MAX / 2 || cols > INT32_MAX / 2) return -1;
  const torq::MixedTiles t = torq::plan_pair_tiles((int)((rows + 255) / 256), cols, pairs, torq::kNarrowTileCost);
  for (int i = 0; out && i < t.total && i < cap; ++i) {
    int mp, col0;
    bool narrow;
    torq::mixed_tile_coords(i, t, mp, col0, narrow);
    out[3 * i] = mp;
    out[3 * i + 1] = col0;
    out[3 * i + 2] = narrow ? torq::kNarrowCols : 256;
  }
  return t.total;
}

int64_t torq_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

int torq_last_device_error(void* stream) {
  DeviceState* st = device_state();
  if (!st || !st->arch_ok) return 0;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (cudaStreamSynchronize(s) != cudaSuccess) return TORQ_ERR_LAUNCH;
  int v = 0, zero = 0;
  if (cudaMemcpy(&v, st->err_word, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess)
    return TORQ_ERR_LAUNCH;
  if (v != 0) cudaMemcpy(st->err_word, &zero, sizeof(int), cudaMemcpyHostToDevice);
  return v;
}

torq_status torq_quantize_mxfp4(const void* Z, torq_dtype z_dtype, int64_t M, int64_t d,
                                void* out_codes, void* out_scales, void* stream) {
  if (!Z || !out_codes || !out_scales) return TORQ_ERR_NULL;
  if (M < 1 || d < 32 || d % 32 != 0 || M > (1 << 30) || d > (1 << 30)) return TORQ_ERR_SHAPE;
  if (z_dtype != TORQ_F32 && z_dtype != TORQ_BF16) return TORQ_ERR_SHAPE;
  if (!aligned16(Z) || !aligned16(out_codes) || !aligned16(out_scales)) return TORQ_ERR_ALIGN;
  DeviceState* st = device_state();
  if (!st) return TORQ_ERR_LAUNCH;
  if (!st->arch_ok) return TORQ_ERR_ARCH;
  return quantize_impl(st, Z, z_dtype, M, d, out_codes, out_scales, static_cast<cudaStream_t>(stream));
}

// Steps 1-4.  `scratch` (may be NULL) is fp32 room for the split-K partials of the few-token path;
// without enough of it the single-pass kernels run.  `fmt` FMT_NVFP4 (with its tensor scale) needs R_inter.
// FMT_F32OUT: out_codes is float32 [M, d] and receives the rotated values (out_scales unused, may be
// NULL); `x_terms` > 1: X is [M, x_terms * d], the sum of its d-wide column groups is what is rotated.
static torq_status rotate_quantize_impl(const void* X, const void* R_inter, const void* R_intra, int64_t M,
                                        int64_t d, void* out_codes, void* out_scales, void* scratch,
                                        size_t scratch_bytes, void* stream, int fmt = FMT_MXFP4,
                                        float tensor_scale = 0.0f, int x_terms = 1) {
  if (!X || !out_codes || (!out_scales && fmt != FMT_F32OUT)) return TORQ_ERR_NULL;
  if (fmt != FMT_MXFP4 && !R_inter) return TORQ_ERR_NULL;
  if (M < 1 || d < 32 || d % 32 != 0 || M > (1 << 30) || d > (1 << 24)) return TORQ_ERR_SHAPE;
  if (x_terms < 1 || x_terms > 4 || (x_terms > 1 && d % 64 != 0)) return TORQ_ERR_SHAPE;
  if (!aligned16(X) || !aligned16(out_codes) || (out_scales && !aligned16(out_scales)) ||
      (R_inter && !aligned16(R_inter)) || (R_intra && !aligned16(R_intra)))
    return TORQ_ERR_ALIGN;
  DeviceState* st = device_state();
  if (!st) return TORQ_ERR_LAUNCH;
  if (!st->arch_ok) return TORQ_ERR_ARCH;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  uint8_t* codes = static_cast<uint8_t*>(out_codes);
  uint8_t* scales = static_cast<uint8_t*>(out_scales);
  if (!R_inter) {
    if (!R_intra) return quantize_impl(st, X, TORQ_BF16, M, d, codes, scales, s);
    const int64_t items = ((M + 127) / 128 * 128) * (((d / 32 + 3) / 4) * 4);
    intra_quantize_kernel<<<ew_grid(items, 128, st->sm_count), 128, 0, s>>>(
        static_cast<const __nv_bfloat16*>(X), static_cast<const __nv_bfloat16*>(R_intra), M, d, codes,
        scales);
    return launch_status();
  }
  CUtensorMap tmX, tmR;
  if (M <= kRotFewMaxTokens && d % 128 == 0 && x_terms == 1 && fmt != FMT_F32OUT) {
    // Few tokens: 128 features x all tokens per CTA, K split over a cluster, reduced through
    // distributed shared memory; one launch, no scratch.
    const int ntok = fewtok_ntok(M);
    const int tiles = (int)(d / 128);
    const int S = fewtok_cluster(tiles, d / 64, 2, st->sm_count, RotFewCfg::ctas_per_sm(ntok));
    if (!encode_2d(&tmX, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, X, (uint64_t)M, (uint64_t)d, (uint32_t)ntok, 64) ||
        !encode_2d(&tmR, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, R_inter, (uint64_t)d, (uint64_t)d, 64, 64))
      return TORQ_ERR_LAUNCH;
    const int smem = RotFewCfg::smem_bytes(ntok);
    const float ts = fmt == FMT_NVFP4 ? tensor_scale : 0.0f;
    const __nv_bfloat16* ri = static_cast<const __nv_bfloat16*>(R_intra);
    if (RotFewCfg::ctas_per_sm(ntok) >= 2) {             // up to 64 tokens: one set of epilogue warps, two CTAs per SM
      if (fmt == FMT_MXINT4)
        launch_tc(rotate_fewtok_kernel<FMT_MXINT4, 1>, S, tiles * S, 192, smem, s, tmX, tmR, ri, codes, scales, (int)M,
                  (int)d, ntok, S, ts, st->err_word);
      else if (fmt == FMT_NVFP4)
        launch_tc(rotate_fewtok_kernel<FMT_NVFP4, 1>, S, tiles * S, 192, smem, s, tmX, tmR, ri, codes, scales, (int)M,
                  (int)d, ntok, S, ts, st->err_word);
      else
        launch_tc(rotate_fewtok_kernel<FMT_MXFP4, 1>, S, tiles * S, 192, smem, s, tmX, tmR, ri, codes, scales, (int)M,
                  (int)d, ntok, S, ts, st->err_word);
    } else {                                             // 128 or 256 tokens: two sets
      if (fmt == FMT_MXINT4)
        launch_tc(rotate_fewtok_kernel<FMT_MXINT4, 2>, S, tiles * S, 320, smem, s, tmX, tmR, ri, codes, scales, (int)M,
                  (int)d, ntok, S, ts, st->err_word);
      else if (fmt == FMT_NVFP4)
        launch_tc(rotate_fewtok_kernel<FMT_NVFP4, 2>, S, tiles * S, 320, smem, s, tmX, tmR, ri, codes, scales, (int)M,
                  (int)d, ntok, S, ts, st->err_word);
      else
        launch_tc(rotate_fewtok_kernel<FMT_MXFP4, 2>, S, tiles * S, 320, smem, s, tmX, tmR, ri, codes, scales, (int)M,
                  (int)d, ntok, S, ts, st->err_word);
    }
    return launch_status();
  }
  if (!encode_2d(&tmX, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, X, (uint64_t)M, (uint64_t)d * x_terms, 128, 64) ||
      !encode_2d(&tmR, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, R_inter, (uint64_t)d, (uint64_t)d, 64, 64))
    return TORQ_ERR_LAUNCH;
  const int splits = (fmt == FMT_F32OUT || x_terms > 1) ? 1 : rotation_splits(M, d, st->sm_count);
  if (splits >= 2 && scratch && scratch_bytes >= splitk_scratch_bytes(M, d, splits) &&
      (reinterpret_cast<uintptr_t>(scratch) & 15u) == 0) {
    // Few tokens: split K over the SMs, partial tiles to scratch, then reduce + intra + quantize.
    CUtensorMap tmP;
    const int m_tiles = (int)((M + 127) / 128);
    if (!encode_2d(&tmP, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, scratch, (uint64_t)splits * m_tiles * 128, (uint64_t)d,
                   32, 32))
      return TORQ_ERR_LAUNCH;
    const int n_tiles = (int)((d + 255) / 256);
    launch_tc(rotate_splitk_kernel, 1, m_tiles * n_tiles * splits, RotSplitCfg::THREADS, RotSplitCfg::SMEM_BYTES, s, tmX, tmR,
              tmP, (int)M, (int)d, splits, st->err_word);
    if (launch_status() != TORQ_OK) return TORQ_ERR_LAUNCH;
    if (fmt == FMT_MXINT4)
      launch_tc(splitk_reduce_quantize_kernel<FMT_MXINT4>, 1, (int)(((d / 32 + 3) / 4) * 4) * m_tiles * 4, 256, 0, s,
                static_cast<const float*>(scratch), static_cast<const __nv_bfloat16*>(R_intra), (int)M, (int)d, splits,
                0.0f, codes, scales);
    else if (fmt == FMT_NVFP4)
      launch_tc(splitk_reduce_quantize_kernel<FMT_NVFP4>, 1, (int)(((d / 16 + 3) / 4) * 2) * m_tiles * 4, 256, 0, s,
                static_cast<const float*>(scratch), static_cast<const __nv_bfloat16*>(R_intra), (int)M, (int)d, splits,
                tensor_scale, codes, scales);
    else
      launch_tc(splitk_reduce_quantize_kernel<FMT_MXFP4>, 1, (int)(((d / 32 + 3) / 4) * 4) * m_tiles * 4, 256, 0, s,
                static_cast<const float*>(scratch), static_cast<const __nv_bfloat16*>(R_intra), (int)M, (int)d, splits,
                0.0f, codes, scales);
    return launch_status();
  }
  if (M > 128) {
    // CTA pairs: 256 x 256 tiles (the last wave 256 x 192 where that fills it better), one pair per two SMs.
    const int max_pairs = st->rot_pairs;
    CUtensorMap tmRn;                                      // second half of a narrow tile's 96 columns per CTA
    if (!encode_2d(&tmRn, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, R_inter, (uint64_t)d, (uint64_t)d, 64, 32))
      return TORQ_ERR_LAUNCH;
    const MixedTiles tiles = plan_pair_tiles((int)((M + 255) / 256), d, max_pairs, kNarrowTileCost);
    const int pairs = tiles.total < max_pairs ? tiles.total : max_pairs;
    if (fmt == FMT_MXINT4)
      launch_tc(rotate_quantize_pair_kernel<FMT_MXINT4>, 2, 2 * pairs, RotPairCfg::THREADS, RotPairCfg::SMEM_BYTES,
                s, tmX, tmR, tmRn, static_cast<const __nv_bfloat16*>(R_intra), codes, scales, (int)M, (int)d, 0.0f,
                x_terms, tiles, st->err_word);
    else if (fmt == FMT_NVFP4)
      launch_tc(rotate_quantize_pair_kernel<FMT_NVFP4>, 2, 2 * pairs, RotPairCfg::THREADS, RotPairCfg::SMEM_BYTES,
                s, tmX, tmR, tmRn, static_cast<const __nv_bfloat16*>(R_intra), codes, scales, (int)M, (int)d,
                tensor_scale, x_terms, tiles, st->err_word);
    else if (fmt == FMT_F32OUT)
      launch_tc(rotate_quantize_pair_kernel<FMT_F32OUT>, 2, 2 * pairs, RotPairCfg::THREADS, RotPairCfg::SMEM_BYTES,
                s, tmX, tmR, tmRn, static_cast<const __nv_bfloat16*>(R_intra), codes, scales, (int)M, (int)d, 0.0f,
                x_terms, tiles, st->err_word);
    else
      launch_tc(rotate_quantize_pair_kernel<FMT_MXFP4>, 2, 2 * pairs, RotPairCfg::THREADS, RotPairCfg::SMEM_BYTES,
                s, tmX, tmR, tmRn, static_cast<const __nv_bfloat16*>(R_intra), codes, scales, (int)M, (int)d, 0.0f,
                x_terms, tiles, st->err_word);
    return launch_status();
  }
  const int m_tiles = (int)((M + 127) / 128);
  const int tiles = m_tiles * (int)((d + 255) / 256);
  const int grid = tiles < st->sm_count ? tiles : st->sm_count;
  if (fmt == FMT_MXINT4)
    launch_tc(rotate_quantize_kernel<256, FMT_MXINT4>, 1, grid, RotCfg<256>::THREADS, RotCfg<256>::SMEM_BYTES, s,
              tmX, tmR, static_cast<const __nv_bfloat16*>(R_intra), codes, scales, (int)M, (int)d, 0.0f,
              x_terms, st->err_word);
  else if (fmt == FMT_NVFP4)
    launch_tc(rotate_quantize_kernel<256, FMT_NVFP4>, 1, grid, RotCfg<256>::THREADS, RotCfg<256>::SMEM_BYTES, s,
              tmX, tmR, static_cast<const __nv_bfloat16*>(R_intra), codes, scales, (int)M, (int)d, tensor_scale,
              x_terms, st->err_word);
  else if (fmt == FMT_F32OUT)
    launch_tc(rotate_quantize_kernel<256, FMT_F32OUT>, 1, grid, RotCfg<256>::THREADS, RotCfg<256>::SMEM_BYTES, s,
              tmX, tmR, static_cast<const __nv_bfloat16*>(R_intra), codes, scales, (int)M, (int)d, 0.0f,
              x_terms, st->err_word);
  else
    launch_tc(rotate_quantize_kernel<256>, 1, grid, RotCfg<256>::THREADS, RotCfg<256>::SMEM_BYTES, s, tmX, tmR,
              static_cast<const __nv_bfloat16*>(R_intra), codes, scales, (int)M, (int)d, 0.0f, x_terms,
              st->err_word);
  return launch_status();
}

torq_status torq_rotate_quantize(const void* X, const void* R_inter, const void* R_intra, int64_t M,
                                 int64_t d, void* out_codes, void* out_scales, void* stream) {
  return rotate_quantize_impl(X, R_inter, R_intra, M, d, out_codes, out_scales, nullptr, 0, stream);
}

static torq_status rotate_structured_impl(const void* X, const void* R_B, const void* R_intra, int64_t M, int64_t d,
                                          void* out_codes, void* out_scales, void* stream, int fmt,
                                          float tensor_scale) {
  if (!X || !R_B || !out_codes || !out_scales) return TORQ_ERR_NULL;
  if (M < 1 || d < 256 || d % 256 != 0 || M > (1 << 30) || d > (1 << 24)) return TORQ_ERR_SHAPE;
  if (!aligned16(X) || !aligned16(R_B) || !aligned16(out_codes) || !aligned16(out_scales) ||
      (R_intra && !aligned16(R_intra)))
    return TORQ_ERR_ALIGN;
  DeviceState* st = device_state();
  if (!st) return TORQ_ERR_LAUNCH;
  if (!st->arch_ok) return TORQ_ERR_ARCH;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int64_t nb = d / 32;
  CUtensorMap tmRB, tmX3;
  if (!encode_2d(&tmRB, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, R_B, (uint64_t)nb, (uint64_t)nb, 128, 64) ||
      !encode_x_blocks_3d(&tmX3, X, (uint64_t)M, (uint64_t)d))
    return TORQ_ERR_LAUNCH;
  const int64_t tiles = ((nb + 127) / 128) * ((M + RotStructCfg::TOK - 1) / RotStructCfg::TOK);
  const int grid = (int)(tiles < st->sm_count ? tiles : st->sm_count);
  if (fmt == FMT_MXINT4)
    launch_tc(rotate_structured_kernel<FMT_MXINT4>, 1, grid, RotStructCfg::THREADS, RotStructCfg::SMEM_BYTES, s, tmRB,
              tmX3, static_cast<const __nv_bfloat16*>(R_intra), static_cast<uint8_t*>(out_codes),
              static_cast<uint8_t*>(out_scales), (int)M, (int)d, 0.0f, st->err_word);
  else if (fmt == FMT_NVFP4)
    launch_tc(rotate_structured_kernel<FMT_NVFP4>, 1, grid, RotStructCfg::THREADS, RotStructCfg::SMEM_BYTES, s, tmRB,
              tmX3, static_cast<const __nv_bfloat16*>(R_intra), static_cast<uint8_t*>(out_codes),
              static_cast<uint8_t*>(out_scales), (int)M, (int)d, tensor_scale, st->err_word);
  else
    launch_tc(rotate_structured_kernel<FMT_MXFP4>, 1, grid, RotStructCfg::THREADS, RotStructCfg::SMEM_BYTES, s, tmRB,
              tmX3, static_cast<const __nv_bfloat16*>(R_intra), static_cast<uint8_t*>(out_codes),
              static_cast<uint8_t*>(out_scales), (int)M, (int)d, 0.0f, st->err_word);
  if (launch_status() != TORQ_OK) return TORQ_ERR_LAUNCH;
  const int64_t ns = fmt == FMT_NVFP4 ? 2 * nb : nb;     // scale bytes per row
  const int64_t kc = (ns + 3) / 4 * 4, mpad = (M + 127) / 128 * 128;
  const int64_t pad = (mpad - M) * kc + M * (kc - ns);
  if (pad > 0) {
    scale_padding_kernel<<<ew_grid(pad, 256, st->sm_count), 256, 0, s>>>(static_cast<uint8_t*>(out_scales), M, ns);
    return launch_status();
  }
  return TORQ_OK;
}

torq_status torq_rotate_quantize_structured(const void* X, const void* R_B, const void* R_intra, int64_t M,
                                            int64_t d, void* out_codes, void* out_scales, void* stream) {
  return rotate_structured_impl(X, R_B, R_intra, M, d, out_codes, out_scales, stream, FMT_MXFP4, 0.0f);
}

torq_status torq_rotate_quantize_structured_nvfp4(const void* X, const void* R_B, const void* R_intra, int64_t M,
                                                  int64_t d, float tensor_scale, void* out_codes, void* out_scales,
                                                  void* stream) {
  if (!(tensor_scale > 0.0f && tensor_scale <= 3.0e38f)) return TORQ_ERR_SHAPE;
  return rotate_structured_impl(X, R_B, R_intra, M, d, out_codes, out_scales, stream, FMT_NVFP4, tensor_scale);
}

}  // extern "C"

// Step 5 for either format; `alpha` multiplies the NVFP4 result (product of the tensor scales).
template <int FMT>
static torq_status gemm_impl(const void* Aq, const void* As, const void* Wq, const void* Ws, int64_t M,
                             int64_t N, int64_t K, void* Y, torq_dtype y_dtype, float alpha, void* stream) {
  if (!Aq || !As || !Wq || !Ws || !Y) return TORQ_ERR_NULL;
  if (M < 1 || N < 8 || K < 128 || K % 128 != 0 || N % 8 != 0 || M > (1 << 30) || N > (1 << 30) ||
      K > (1 << 24))
    return TORQ_ERR_SHAPE;
  if (y_dtype != TORQ_F32 && y_dtype != TORQ_BF16) return TORQ_ERR_SHAPE;
  if (!aligned16(Aq) || !aligned16(As) || !aligned16(Wq) || !aligned16(Ws) || !aligned16(Y))
    return TORQ_ERR_ALIGN;
  DeviceState* st = device_state();
  if (!st) return TORQ_ERR_LAUNCH;
  if (!st->arch_ok) return TORQ_ERR_ARCH;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  constexpr int BN = 256;
  const uint64_t krow = (uint64_t)(FMT == FMT_MXINT4 ? K : K / 2);   // operand bytes per row
  CUtensorMap tmA, tmB;
  if (M <= kGemmFewMaxTokens) {
    // Few tokens: 128 output features x all tokens per CTA, K split over a cluster, reduced through
    // distributed shared memory.
    using FC = GemmFewCfg<FMT>;
    const int ntok = fewtok_ntok(M);
    const int tiles = (int)((N + 127) / 128);
    const int S = fewtok_cluster(tiles, (K + FC::BK - 1) / FC::BK, 1, st->sm_count, FC::ctas_per_sm(ntok));
    if (!encode_2d(&tmB, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, Wq, (uint64_t)N, krow, 128, 128) ||
        !encode_2d(&tmA, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, Aq, (uint64_t)M, krow, (uint32_t)ntok, 128))
      return TORQ_ERR_LAUNCH;
    if (FC::ctas_per_sm(ntok) >= 2)                      // up to 64 tokens: one set of epilogue warps, two CTAs per SM
      launch_tc(gemm_fewtok_kernel<FMT, 1>, S, tiles * S, 192, FC::smem_bytes(ntok), s, tmB, tmA,
                static_cast<const uint8_t*>(As), static_cast<const uint8_t*>(Ws), Y, y_dtype == TORQ_BF16 ? 1 : 0, (int)M,
                (int)N, (int)K, ntok, S, alpha, st->err_word);
    else                                                 // 128 tokens: two sets
      launch_tc(gemm_fewtok_kernel<FMT, 2>, S, tiles * S, 320, FC::smem_bytes(ntok), s, tmB, tmA,
                static_cast<const uint8_t*>(As), static_cast<const uint8_t*>(Ws), Y, y_dtype == TORQ_BF16 ? 1 : 0, (int)M,
                (int)N, (int)K, ntok, S, alpha, st->err_word);
    return launch_status();
  }
  // CTA pairs from two row tiles on -- except for exactly two row tiles with so few 256-column tiles
  // that the pairs would leave more than half of the SMs idle: 128 x 128 tiles on single CTAs then
  // put four times as many SMs to work on streaming W.
  const int64_t pair_tiles = ((M + 255) / 256) * ((N + BN - 1) / BN);
  const bool use_pairs = M > 128 && !(M <= 256 && 4 * pair_tiles <= st->sm_count);
  if (use_pairs) {
    CUtensorMap tmSFA, tmSFB;
    const uint64_t kb4 = (uint64_t)(K / (FMT == FMT_NVFP4 ? 64 : 128));   // 512-byte scale chunks per row
    constexpr uint32_t sf_box = GemmPairCfgT<FMT>::SF_BOX_WORDS;
    if (!encode_2d(&tmA, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, Aq, (uint64_t)M, krow, 128, 128) ||
        !encode_2d(&tmB, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, Wq, (uint64_t)N, krow, BN / 2, 128) ||
        !encode_2d(&tmSFA, CU_TENSOR_MAP_DATA_TYPE_UINT32, 4, As, (uint64_t)((M + 127) / 128), kb4 * 128, 1, sf_box,
                   CU_TENSOR_MAP_SWIZZLE_NONE) ||
        !encode_2d(&tmSFB, CU_TENSOR_MAP_DATA_TYPE_UINT32, 4, Ws, (uint64_t)((N + 127) / 128), kb4 * 128, 1, sf_box,
                   CU_TENSOR_MAP_SWIZZLE_NONE))
      return TORQ_ERR_LAUNCH;
    CUtensorMap tmY;
    const bool ybf = y_dtype == TORQ_BF16;
    if (!encode_2d(&tmY, ybf ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, ybf ? 2 : 4,
                   Y, (uint64_t)M, (uint64_t)N, 32, ybf ? 64 : 32))
      return TORQ_ERR_LAUNCH;
    CUtensorMap tmBn;                                      // half of a 192-column tile: 96 rows of W
    if (!encode_2d(&tmBn, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, Wq, (uint64_t)N, krow, kNarrowCols / 2, 128))
      return TORQ_ERR_LAUNCH;
    const int max_pairs = st->gemm_pairs;
    const MixedTiles tiles = plan_pair_tiles((int)((M + 255) / 256), N, max_pairs, kNarrowTileCost);
    const int pairs = tiles.total < max_pairs ? tiles.total : max_pairs;
    launch_tc(mxfp4_gemm_pair_kernel<FMT>, 2, 2 * pairs, GemmPairCfgT<FMT>::THREADS, GemmPairCfgT<FMT>::SMEM_BYTES, s,
              tmA, tmB, tmSFA, tmSFB, tmY, tmBn, tiles, ybf ? 1 : 0, (int)M, (int)N, (int)K, alpha, st->err_word);
    return launch_status();
  }
  // One or two row tiles: the work is streaming W once, so prefer the narrower tile while it still leaves
  // SMs idle (128-column tiles double the number of CTAs pulling on memory).
  const bool narrow = 2 * (int)((M + 127) / 128) * (int)((N + BN - 1) / BN) <= st->sm_count;
  const uint32_t bn = narrow ? 128 : BN;
  if (!encode_2d(&tmA, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, Aq, (uint64_t)M, krow, 128, 128) ||
      !encode_2d(&tmB, CU_TENSOR_MAP_DATA_TYPE_UINT8, 1, Wq, (uint64_t)N, krow, bn, 128))
    return TORQ_ERR_LAUNCH;
  const int tiles = (int)((M + 127) / 128) * (int)((N + bn - 1) / bn);
  const int grid = tiles < st->sm_count ? tiles : st->sm_count;
  if (narrow)
    launch_tc(mxfp4_gemm_kernel<128, 2, FMT>, 1, grid, GemmCfg<128, 2, FMT>::THREADS, GemmCfg<128, 2, FMT>::SMEM_BYTES,
              s, tmA, tmB, static_cast<const uint8_t*>(As), static_cast<const uint8_t*>(Ws), Y,
              y_dtype == TORQ_BF16 ? 1 : 0, (int)M, (int)N, (int)K, alpha, st->err_word);
  else
    launch_tc(mxfp4_gemm_kernel<BN, 1, FMT>, 1, grid, GemmCfg<BN, 1, FMT>::THREADS, GemmCfg<BN, 1, FMT>::SMEM_BYTES, s,
              tmA, tmB, static_cast<const uint8_t*>(As), static_cast<const uint8_t*>(Ws), Y,
              y_dtype == TORQ_BF16 ? 1 : 0, (int)M, (int)N, (int)K, alpha, st->err_word);
  return launch_status();
}

extern "C" {

torq_status torq_mxfp4_gemm(const void* Aq, const void* As, const void* Wq, const void* Ws, int64_t M,
                            int64_t N, int64_t K, void* Y, torq_dtype y_dtype, void* stream) {
  return gemm_impl<FMT_MXFP4>(Aq, As, Wq, Ws, M, N, K, Y, y_dtype, 1.0f, stream);
}

static inline bool scale_ok(float s) { return s > 0.0f && s <= 3.0e38f; }   // positive, finite

torq_status torq_nvfp4_gemm(const void* Aq, const void* As, float a_tensor_scale, const void* Wq, const void* Ws,
                            float w_tensor_scale, int64_t M, int64_t N, int64_t K, void* Y, torq_dtype y_dtype,
                            void* stream) {
  if (!scale_ok(a_tensor_scale) || !scale_ok(w_tensor_scale)) return TORQ_ERR_SHAPE;
  return gemm_impl<FMT_NVFP4>(Aq, As, Wq, Ws, M, N, K, Y, y_dtype, a_tensor_scale * w_tensor_scale, stream);
}

size_t torq_nvfp4_scales_bytes(int64_t rows, int64_t k) {
  if (rows <= 0 || k <= 0) return 0;
  return (size_t)((rows + 127) / 128) * (size_t)((k / 16 + 3) / 4) * 512;
}

static size_t nvfp4_quantized_bytes(int64_t M, int64_t d) {
  return ((size_t)M * (size_t)(d / 2) + 255) / 256 * 256 + torq_nvfp4_scales_bytes(M, d);
}

size_t torq_nvfp4_workspace_bytes(int64_t M, int64_t d, int64_t N) {
  (void)N;
  if (M <= 0 || d <= 0) return 0;
  return nvfp4_quantized_bytes(M, d) + splitk_scratch_bytes(M, d, rotation_splits(M, d, 0));
}

torq_status torq_expand_intra16(const void* R_intra16, int64_t d, void* R_intra32, void* stream) {
  if (!R_intra16 || !R_intra32) return TORQ_ERR_NULL;
  if (d < 32 || d % 32 != 0 || d > (1 << 24)) return TORQ_ERR_SHAPE;
  DeviceState* st = device_state();
  if (!st) return TORQ_ERR_LAUNCH;
  if (!st->arch_ok) return TORQ_ERR_ARCH;
  expand_intra16_kernel<<<ew_grid(d * 32, 256, st->sm_count), 256, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const __nv_bfloat16*>(R_intra16), d / 32, static_cast<__nv_bfloat16*>(R_intra32));
  return launch_status();
}

torq_status torq_quantize_nvfp4(const void* Z, torq_dtype z_dtype, int64_t M, int64_t d, float tensor_scale,
                                void* out_codes, void* out_scales, void* stream) {
  if (!Z || !out_codes || !out_scales) return TORQ_ERR_NULL;
  if (M < 1 || d < 16 || d % 16 != 0 || M > (1 << 30) || d > (1 << 30) || !scale_ok(tensor_scale))
    return TORQ_ERR_SHAPE;
  if (z_dtype != TORQ_F32 && z_dtype != TORQ_BF16) return TORQ_ERR_SHAPE;
  if (!aligned16(Z) || !aligned16(out_codes) || !aligned16(out_scales)) return TORQ_ERR_ALIGN;
  DeviceState* st = device_state();
  if (!st) return TORQ_ERR_LAUNCH;
  if (!st->arch_ok) return TORQ_ERR_ARCH;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int64_t kb4 = (d / 16 + 3) / 4;
  const int64_t items = ((M + 127) / 128 * 128) * ((kb4 * 64 + 255) / 256);   // warps
  const int grid = ew_grid(items, 8, st->sm_count);
  if (z_dtype == TORQ_F32)
    nv_quantize_kernel<float><<<grid, 256, 0, s>>>(static_cast<const float*>(Z), M, d, tensor_scale,
                                                   static_cast<uint8_t*>(out_codes), static_cast<uint8_t*>(out_scales));
  else
    nv_quantize_kernel<__nv_bfloat16><<<grid, 256, 0, s>>>(static_cast<const __nv_bfloat16*>(Z), M, d, tensor_scale,
                                                           static_cast<uint8_t*>(out_codes),
                                                           static_cast<uint8_t*>(out_scales));
  return launch_status();
}

torq_status torq_rotate_quantize_nvfp4(const void* X, const void* R_inter, const void* R_intra32, int64_t M,
                                       int64_t d, float tensor_scale, void* out_codes, void* out_scales,
                                       void* stream) {
  if (!scale_ok(tensor_scale)) return TORQ_ERR_SHAPE;
  return rotate_quantize_impl(X, R_inter, R_intra32, M, d, out_codes, out_scales, nullptr, 0, stream, FMT_NVFP4,
                              tensor_scale);
}

torq_status torq_rotated_linear_nvfp4(const void* X, const void* R_inter, const void* R_intra32, float x_tensor_scale,
                                      const void* Wq, const void* Ws, float w_tensor_scale, int64_t M, int64_t d,
                                      int64_t N, void* Y, torq_dtype y_dtype, void* workspace, size_t workspace_bytes,
                                      void* dbg_codes, void* dbg_scales, void* stream) {
  if (!X || !R_inter || !Wq || !Ws || !Y) return TORQ_ERR_NULL;
  if (M < 1 || d < 128 || d % 128 != 0 || N < 8 || N % 8 != 0 || M > (1 << 30) || d > (1 << 24) ||
      !scale_ok(x_tensor_scale) || !scale_ok(w_tensor_scale))
    return TORQ_ERR_SHAPE;
  if (!workspace || workspace_bytes < torq_nvfp4_workspace_bytes(M, d, N)) return TORQ_ERR_WORKSPACE;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return TORQ_ERR_ALIGN;
  uint8_t* codes = static_cast<uint8_t*>(workspace);
  const size_t codes_bytes = (size_t)M * (size_t)(d / 2);
  uint8_t* scales = codes + (codes_bytes + 255) / 256 * 256;
  const size_t used = nvfp4_quantized_bytes(M, d);
  torq_status rc = rotate_quantize_impl(X, R_inter, R_intra32, M, d, codes, scales, codes + used,
                                        workspace_bytes - used, stream, FMT_NVFP4, x_tensor_scale);
  if (rc != TORQ_OK) return rc;
  rc = torq_nvfp4_gemm(codes, scales, x_tensor_scale, Wq, Ws, w_tensor_scale, M, N, d, Y, y_dtype, stream);
  if (rc != TORQ_OK) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (dbg_codes &&
      cudaMemcpyAsync(dbg_codes, codes, codes_bytes, cudaMemcpyDeviceToDevice, s) != cudaSuccess)
    return TORQ_ERR_LAUNCH;
  if (dbg_scales && cudaMemcpyAsync(dbg_scales, scales, torq_nvfp4_scales_bytes(M, d),
                                    cudaMemcpyDeviceToDevice, s) != cudaSuccess)
    return TORQ_ERR_LAUNCH;
  return TORQ_OK;
}

// ---- MXINT4 (format study of Section 6): integer codes, E8M0 scales, E4M3 operand bytes ----------

static size_t mxint4_quantized_bytes(int64_t M, int64_t d) {
  return ((size_t)M * (size_t)d + 255) / 256 * 256 + torq_scales_bytes(M, d);
}

size_t torq_mxint4_workspace_bytes(int64_t M, int64_t d, int64_t N) {
  (void)N;
  if (M <= 0 || d <= 0) return 0;
  return mxint4_quantized_bytes(M, d) + splitk_scratch_bytes(M, d, rotation_splits(M, d, 0));
}

torq_status torq_quantize_mxint4(const void* Z, torq_dtype z_dtype, int64_t M, int64_t d, int packed, void* out_codes,
                                 void* out_scales, void* stream) {
  if (!Z || !out_codes || !out_scales) return TORQ_ERR_NULL;
  if (M < 1 || d < 32 || d % 32 != 0 || M > (1 << 30) || d > (1 << 30)) return TORQ_ERR_SHAPE;
  if (z_dtype != TORQ_F32 && z_dtype != TORQ_BF16) return TORQ_ERR_SHAPE;
  if (!aligned16(Z) || !aligned16(out_codes) || !aligned16(out_scales)) return TORQ_ERR_ALIGN;
  DeviceState* st = device_state();
  if (!st) return TORQ_ERR_LAUNCH;
  if (!st->arch_ok) return TORQ_ERR_ARCH;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int64_t kb4 = (d / 32 + 3) / 4;
  const int64_t items = ((M + 127) / 128 * 128) * ((kb4 * 128 + 255) / 256);   // warps
  const int grid = ew_grid(items, 8, st->sm_count);
  uint8_t* c = static_cast<uint8_t*>(out_codes);
  uint8_t* sc = static_cast<uint8_t*>(out_scales);
  if (z_dtype == TORQ_F32) {
    const float* z = static_cast<const float*>(Z);
    if (packed) mxint4_quantize_kernel<float, true><<<grid, 256, 0, s>>>(z, M, d, c, sc);
    else mxint4_quantize_kernel<float, false><<<grid, 256, 0, s>>>(z, M, d, c, sc);
  } else {
    const __nv_bfloat16* z = static_cast<const __nv_bfloat16*>(Z);
    if (packed) mxint4_quantize_kernel<__nv_bfloat16, true><<<grid, 256, 0, s>>>(z, M, d, c, sc);
    else mxint4_quantize_kernel<__nv_bfloat16, false><<<grid, 256, 0, s>>>(z, M, d, c, sc);
  }
  return launch_status();
}

torq_status torq_mxint4_expand(const void* packed, int64_t rows, int64_t k, void* out_bytes, void* stream) {
  if (!packed || !out_bytes) return TORQ_ERR_NULL;
  if (rows < 1 || k < 32 || k % 32 != 0 || rows > (1 << 30) || k > (1 << 30)) return TORQ_ERR_SHAPE;
  if (!aligned16(packed) || !aligned16(out_bytes)) return TORQ_ERR_ALIGN;
  DeviceState* st = device_state();
  if (!st) return TORQ_ERR_LAUNCH;
  if (!st->arch_ok) return TORQ_ERR_ARCH;
  const int64_t words = rows * (k / 8);
  mxint4_expand_kernel<<<ew_grid(words, 256, st->sm_count), 256, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const uint32_t*>(packed), words, static_cast<uint2*>(out_bytes));
  return launch_status();
}

torq_status torq_rotate_quantize_mxint4(const void* X, const void* R_inter, const void* R_intra, int64_t M,
                                        int64_t d, void* out_bytes, void* out_scales, void* stream) {
  return rotate_quantize_impl(X, R_inter, R_intra, M, d, out_bytes, out_scales, nullptr, 0, stream, FMT_MXINT4,
                              0.0f);
}

torq_status torq_rotate_quantize_structured_mxint4(const void* X, const void* R_B, const void* R_intra, int64_t M,
                                                   int64_t d, void* out_bytes, void* out_scales, void* stream) {
  return rotate_structured_impl(X, R_B, R_intra, M, d, out_bytes, out_scales, stream, FMT_MXINT4, 0.0f);
}

torq_status torq_mxint4_gemm(const void* A8, const void* As, const void* W8, const void* Ws, int64_t M, int64_t N,
                             int64_t K, void* Y, torq_dtype y_dtype, void* stream) {
  return gemm_impl<FMT_MXINT4>(A8, As, W8, Ws, M, N, K, Y, y_dtype, 1.0f, stream);
}

torq_status torq_rotated_linear_mxint4(const void* X, const void* R_inter, const void* R_intra, const void* W8,
                                       const void* Ws, int64_t M, int64_t d, int64_t N, void* Y, torq_dtype y_dtype,
                                       void* workspace, size_t workspace_bytes, void* dbg_bytes, void* dbg_scales,
                                       void* stream) {
  if (!X || !R_inter || !W8 || !Ws || !Y) return TORQ_ERR_NULL;
  if (M < 1 || d < 128 || d % 128 != 0 || N < 8 || N % 8 != 0 || M > (1 << 30) || d > (1 << 24))
    return TORQ_ERR_SHAPE;
  if (!workspace || workspace_bytes < torq_mxint4_workspace_bytes(M, d, N)) return TORQ_ERR_WORKSPACE;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return TORQ_ERR_ALIGN;
  uint8_t* bytes = static_cast<uint8_t*>(workspace);
  const size_t n_bytes = (size_t)M * (size_t)d;
  uint8_t* scales = bytes + (n_bytes + 255) / 256 * 256;
  const size_t used = mxint4_quantized_bytes(M, d);
  torq_status rc = rotate_quantize_impl(X, R_inter, R_intra, M, d, bytes, scales, bytes + used, workspace_bytes - used,
                                        stream, FMT_MXINT4, 0.0f);
  if (rc != TORQ_OK) return rc;
  rc = torq_mxint4_gemm(bytes, scales, W8, Ws, M, N, d, Y, y_dtype, stream);
  if (rc != TORQ_OK) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (dbg_bytes && cudaMemcpyAsync(dbg_bytes, bytes, n_bytes, cudaMemcpyDeviceToDevice, s) != cudaSuccess)
    return TORQ_ERR_LAUNCH;
  if (dbg_scales &&
      cudaMemcpyAsync(dbg_scales, scales, torq_scales_bytes(M, d), cudaMemcpyDeviceToDevice, s) != cudaSuccess)
    return TORQ_ERR_LAUNCH;
  return TORQ_OK;
}

// Steps 1-5 with `workspace_bytes` >= quantized_bytes(M, d) already checked by the caller: codes,
// scales, then whatever is left as split-K scratch.
static torq_status rotated_linear_impl(const void* X, const void* R_inter, const void* R_intra, const void* Wq,
                                       const void* Ws, int64_t M, int64_t d, int64_t N, void* Y,
                                       torq_dtype y_dtype, void* workspace, size_t workspace_bytes,
                                       void* dbg_codes, void* dbg_scales, void* stream) {
  uint8_t* codes = static_cast<uint8_t*>(workspace);
  const size_t codes_bytes = (size_t)M * (size_t)(d / 2);
  uint8_t* scales = codes + (codes_bytes + 255) / 256 * 256;
  const size_t used = quantized_bytes(M, d);
  torq_status rc = rotate_quantize_impl(X, R_inter, R_intra, M, d, codes, scales, codes + used,
                                        workspace_bytes > used ? workspace_bytes - used : 0, stream);
  if (rc != TORQ_OK) return rc;
  rc = torq_mxfp4_gemm(codes, scales, Wq, Ws, M, N, d, Y, y_dtype, stream);
  if (rc != TORQ_OK) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (dbg_codes &&
      cudaMemcpyAsync(dbg_codes, codes, codes_bytes, cudaMemcpyDeviceToDevice, s) != cudaSuccess)
    return TORQ_ERR_LAUNCH;
  if (dbg_scales && cudaMemcpyAsync(dbg_scales, scales, torq_scales_bytes(M, d),
                                    cudaMemcpyDeviceToDevice, s) != cudaSuccess)
    return TORQ_ERR_LAUNCH;
  return TORQ_OK;
}

torq_status torq_rotated_linear(const void* X, const void* R_inter, const void* R_intra, const void* Wq,
                                const void* Ws, int64_t M, int64_t d, int64_t N, void* Y,
                                torq_dtype y_dtype, void* workspace, size_t workspace_bytes,
                                void* dbg_codes, void* dbg_scales, void* stream) {
  if (!X || !Wq || !Ws || !Y) return TORQ_ERR_NULL;
  if (M < 1 || d < 128 || d % 128 != 0 || N < 8 || N % 8 != 0) return TORQ_ERR_SHAPE;
  if (!workspace || workspace_bytes < torq_workspace_bytes(M, d, N)) return TORQ_ERR_WORKSPACE;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return TORQ_ERR_ALIGN;
  return rotated_linear_impl(X, R_inter, R_intra, Wq, Ws, M, d, N, Y, y_dtype, workspace, workspace_bytes,
                             dbg_codes, dbg_scales, stream);
}

torq_status torq_rotated_linear_structured(const void* X, const void* R_B, const void* R_intra, const void* Wq,
                                           const void* Ws, int64_t M, int64_t d, int64_t N, void* Y,
                                           torq_dtype y_dtype, void* workspace, size_t workspace_bytes,
                                           void* dbg_codes, void* dbg_scales, void* stream) {
  if (!X || !R_B || !Wq || !Ws || !Y) return TORQ_ERR_NULL;
  if (M < 1 || d < 256 || d % 256 != 0 || N < 8 || N % 8 != 0) return TORQ_ERR_SHAPE;
  if (!workspace || workspace_bytes < quantized_bytes(M, d)) return TORQ_ERR_WORKSPACE;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return TORQ_ERR_ALIGN;
  uint8_t* codes = static_cast<uint8_t*>(workspace);
  const size_t codes_bytes = (size_t)M * (size_t)(d / 2);
  uint8_t* scales = codes + (codes_bytes + 255) / 256 * 256;
  torq_status rc = torq_rotate_quantize_structured(X, R_B, R_intra, M, d, codes, scales, stream);
  if (rc != TORQ_OK) return rc;
  rc = torq_mxfp4_gemm(codes, scales, Wq, Ws, M, N, d, Y, y_dtype, stream);
  if (rc != TORQ_OK) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (dbg_codes &&
      cudaMemcpyAsync(dbg_codes, codes, codes_bytes, cudaMemcpyDeviceToDevice, s) != cudaSuccess)
    return TORQ_ERR_LAUNCH;
  if (dbg_scales && cudaMemcpyAsync(dbg_scales, scales, torq_scales_bytes(M, d),
                                    cudaMemcpyDeviceToDevice, s) != cudaSuccess)
    return TORQ_ERR_LAUNCH;
  return TORQ_OK;
}

// ---- the layer without any allocation -----------------------------------------------------------
// Scratch for torq_rotated_linear_static.  In host code this name is only a handle for the
// runtime's symbol table, not an address a kernel can use: the device address comes from
// cudaGetSymbolAddress, once per device, with that device current.
static __device__ __align__(256) uint8_t g_static_workspace[TORQ_STATIC_WORKSPACE_BYTES];
static void* g_static_workspace_addr[torq::kMaxDevices] = {};
static std::mutex g_static_workspace_mutex;

// Device address of the scratch array on the current device (nullptr when CUDA reports an error).
static void* static_workspace_address() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= torq::kMaxDevices) return nullptr;
  std::lock_guard<std::mutex> lock(g_static_workspace_mutex);
  if (!g_static_workspace_addr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_workspace) != cudaSuccess || p == nullptr) {
      cudaGetLastError();                    // leave no sticky-looking error behind for the caller
      return nullptr;
    }
    g_static_workspace_addr[dev] = p;
  }
  return g_static_workspace_addr[dev];
}

torq_status torq_rotated_linear_static(const void* X, const void* R_inter, const void* R_intra,
                                       const void* Wq, const void* Ws, int64_t M, int64_t d,
                                       int64_t N, void* Y, torq_dtype y_dtype, void* stream) {
  if (!X || !Wq || !Ws || !Y) return TORQ_ERR_NULL;
  if (M < 1 || d < 128 || d % 128 != 0 || N < 8 || N % 8 != 0 || M > (1 << 30) || d > (1 << 24))
    return TORQ_ERR_SHAPE;
  if (quantized_bytes(M, d) > (size_t)TORQ_STATIC_WORKSPACE_BYTES) return TORQ_ERR_WORKSPACE;
  DeviceState* st = device_state();                // architecture first: another device has no image of the array
  if (!st) return TORQ_ERR_LAUNCH;
  if (!st->arch_ok) return TORQ_ERR_ARCH;
  void* scratch = static_workspace_address();
  if (!scratch) return TORQ_ERR_LAUNCH;
  return rotated_linear_impl(X, R_inter, R_intra, Wq, Ws, M, d, N, Y, y_dtype, scratch,
                             (size_t)TORQ_STATIC_WORKSPACE_BYTES, nullptr, nullptr, stream);
}

torq_status torq_probe_fp4_peak(int groups, double* tflops, void* stream) {
  if (!tflops) return TORQ_ERR_NULL;
  if (groups < 1 || groups > (1 << 24)) return TORQ_ERR_SHAPE;
  DeviceState* st = device_state();
  if (!st) return TORQ_ERR_LAUNCH;
  if (!st->arch_ok) return TORQ_ERR_ARCH;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (!opt_in_smem(fp4_peak_probe_kernel, Fp4ProbeCfg::SMEM_BYTES)) return TORQ_ERR_LAUNCH;
  const int pairs = st->gemm_pairs;
  cudaEvent_t e0, e1;
  if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) return TORQ_ERR_LAUNCH;
  launch_tc(fp4_peak_probe_kernel, 2, 2 * pairs, Fp4ProbeCfg::THREADS, Fp4ProbeCfg::SMEM_BYTES, s, 64, st->err_word);
  cudaEventRecord(e0, s);
  launch_tc(fp4_peak_probe_kernel, 2, 2 * pairs, Fp4ProbeCfg::THREADS, Fp4ProbeCfg::SMEM_BYTES, s, groups, st->err_word);
  cudaEventRecord(e1, s);
  g_launches.fetch_add(2, std::memory_order_relaxed);
  float ms = 0.f;
  const bool ok = cudaEventSynchronize(e1) == cudaSuccess && cudaEventElapsedTime(&ms, e0, e1) == cudaSuccess &&
                  cudaGetLastError() == cudaSuccess && ms > 0.f;
  cudaEventDestroy(e0);
  cudaEventDestroy(e1);
  if (!ok) return TORQ_ERR_LAUNCH;
  *tflops = (double)pairs * groups * 4.0 * 2.0 * 256.0 * 256.0 * 64.0 / ((double)ms * 1e-3) / 1e12;
  return TORQ_OK;
}

torq_status torq_selftest_wait_timeout(uint64_t limit_ns, void* result_u64x3, void* stream) {
  if (!result_u64x3) return TORQ_ERR_NULL;
  if (limit_ns < 1000ull || limit_ns > 100000000ull) return TORQ_ERR_SHAPE;        // 1 us .. 100 ms
  if (!aligned16(result_u64x3)) return TORQ_ERR_ALIGN;
  DeviceState* st = device_state();
  if (!st) return TORQ_ERR_LAUNCH;
  if (!st->arch_ok) return TORQ_ERR_ARCH;
  wait_selftest_kernel<<<1, 64, 0, static_cast<cudaStream_t>(stream)>>>(
      (unsigned long long)limit_ns, st->err_word, static_cast<unsigned long long*>(result_u64x3));
  return launch_status();
}

torq_status torq_block_covariance(const void* X, int64_t T, int64_t d, void* Sigma_f64, void* stream) {
  if (!X || !Sigma_f64) return TORQ_ERR_NULL;
  if (T < 1 || d < 32 || d % 32 != 0 || T > (1 << 30) || d > (1 << 20)) return TORQ_ERR_SHAPE;
  if (!aligned16(X) || !aligned16(Sigma_f64)) return TORQ_ERR_ALIGN;
  DeviceState* st = device_state();
  if (!st) return TORQ_ERR_LAUNCH;
  if (!st->arch_ok) return TORQ_ERR_ARCH;
  const unsigned tiles = (unsigned)((d / 32 + 15) / 16);
  block_covariance_kernel<<<dim3(tiles, tiles, 1), 256, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const __nv_bfloat16*>(X), T, d, static_cast<double*>(Sigma_f64));
  return launch_status();
}

torq_status torq_givens_equalize(void* Sigma_f64, int64_t B, double eps, void* Q_f64, void* Q_bf16,
                                 void* n_rotations, void* stream) {
  if (!Sigma_f64 || !Q_f64) return TORQ_ERR_NULL;
  if (B < 1 || B > 32768 || !(eps >= 0.0)) return TORQ_ERR_SHAPE;
  if (!aligned16(Sigma_f64) || !aligned16(Q_f64) || (Q_bf16 && !aligned16(Q_bf16))) return TORQ_ERR_ALIGN;
  DeviceState* st = device_state();
  if (!st) return TORQ_ERR_LAUNCH;
  if (!st->arch_ok) return TORQ_ERR_ARCH;
  givens_equalize_kernel<<<1, 512, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<double*>(Sigma_f64), (int)B, eps, static_cast<double*>(Q_f64), static_cast<__nv_bfloat16*>(Q_bf16),
      static_cast<int*>(n_rotations), (int)(4 * B));
  return launch_status();
}

torq_status torq_swizzle_scales(const void* linear_scales, int64_t rows, int64_t k, void* out,
                                void* stream) {
  if (!linear_scales || !out) return TORQ_ERR_NULL;
  if (rows < 1 || k < 32 || k % 32 != 0) return TORQ_ERR_SHAPE;
  DeviceState* st = device_state();
  if (!st) return TORQ_ERR_LAUNCH;
  if (!st->arch_ok) return TORQ_ERR_ARCH;
  const int64_t items = ((rows + 127) / 128 * 128) * (((k / 32 + 3) / 4) * 4);
  swizzle_scales_kernel<<<ew_grid(items, 256, st->sm_count), 256, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const uint8_t*>(linear_scales), rows, k / 32, static_cast<uint8_t*>(out));
  return launch_status();
}

// ---- offline weight side (Algorithm 3 step 5, option B) ------------------------------------------
// Workspace: the three-term bf16 split of W^T [N, 3 d], then (256-byte aligned) W' as float32 [N, d].
static size_t prep_split_bytes(int64_t d, int64_t N) { return ((size_t)N * (size_t)d * 6 + 255) / 256 * 256; }

size_t torq_prepare_weights_workspace_bytes(int64_t d, int64_t N) {
  if (d <= 0 || N <= 0) return 0;
  return prep_split_bytes(d, N) + (size_t)N * (size_t)d * 4;
}

// W' (float32 [N, d]) into the workspace; returns its address in *wp.
static torq_status rotate_weights(const void* W, const void* R_inter, const void* R_intra, int64_t d, int64_t N,
                                  void* workspace, size_t workspace_bytes, void* stream, float** wp) {
  if (!W || !R_inter) return TORQ_ERR_NULL;
  if (d < 64 || d % 64 != 0 || N < 1 || N > (1 << 30) || d > (1 << 24)) return TORQ_ERR_SHAPE;
  if (!workspace || workspace_bytes < torq_prepare_weights_workspace_bytes(d, N)) return TORQ_ERR_WORKSPACE;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0 || !aligned16(W)) return TORQ_ERR_ALIGN;
  DeviceState* st = device_state();
  if (!st) return TORQ_ERR_LAUNCH;
  if (!st->arch_ok) return TORQ_ERR_ARCH;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  __nv_bfloat16* T = static_cast<__nv_bfloat16*>(workspace);
  *wp = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + prep_split_bytes(d, N));
  const int64_t tiles = ((N + 31) / 32) * ((d + 31) / 32);
  transpose_split3_kernel<<<ew_grid(tiles, 1, st->sm_count), 256, 0, s>>>(static_cast<const float*>(W), d, N, T);
  if (launch_status() != TORQ_OK) return TORQ_ERR_LAUNCH;
  return rotate_quantize_impl(T, R_inter, R_intra, N, d, *wp, nullptr, nullptr, 0, stream, FMT_F32OUT, 0.0f, 3);
}

torq_status torq_prepare_weights(const void* W, const void* R_inter, const void* R_intra, int64_t d, int64_t N,
                                 void* Wq, void* Ws, void* workspace, size_t workspace_bytes, void* stream) {
  if (!Wq || !Ws) return TORQ_ERR_NULL;
  float* wp = nullptr;
  const torq_status rc = rotate_weights(W, R_inter, R_intra, d, N, workspace, workspace_bytes, stream, &wp);
  if (rc != TORQ_OK) return rc;
  return torq_quantize_mxfp4(wp, TORQ_F32, N, d, Wq, Ws, stream);
}

torq_status torq_prepare_weights_nvfp4(const void* W, const void* R_inter, const void* R_intra32, int64_t d,
                                       int64_t N, void* Wq, void* Ws, float* tensor_scale, void* workspace,
                                       size_t workspace_bytes, void* stream) {
  if (!Wq || !Ws || !tensor_scale) return TORQ_ERR_NULL;
  float* wp = nullptr;
  torq_status rc = rotate_weights(W, R_inter, R_intra32, d, N, workspace, workspace_bytes, stream, &wp);
  if (rc != TORQ_OK) return rc;
  DeviceState* st = device_state();
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // the split of W^T is no longer needed: its first word holds the running maximum
  unsigned int* amax_bits = static_cast<unsigned int*>(workspace);
  if (cudaMemsetAsync(amax_bits, 0, sizeof(unsigned int), s) != cudaSuccess) return TORQ_ERR_LAUNCH;
  absmax_kernel<<<ew_grid(N * d, 1024, st->sm_count), 256, 0, s>>>(wp, N * d, amax_bits);
  if (launch_status() != TORQ_OK) return TORQ_ERR_LAUNCH;
  float amax = 0.f;
  if (cudaMemcpyAsync(&amax, amax_bits, sizeof(float), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
      cudaStreamSynchronize(s) != cudaSuccess)
    return TORQ_ERR_LAUNCH;
  const float ts = amax / 2688.0f;                       // amax / (6 * 448), one float32 division
  if (!scale_ok(ts)) return TORQ_ERR_SHAPE;              // an all-zero (or non-finite) W' has no scale
  *tensor_scale = ts;
  return torq_quantize_nvfp4(wp, TORQ_F32, N, d, ts, Wq, Ws, stream);
}

torq_status torq_prepare_weights_mxint4(const void* W, const void* R_inter, const void* R_intra, int64_t d,
                                        int64_t N, void* Wn, void* W8, void* Ws, void* workspace,
                                        size_t workspace_bytes, void* stream) {
  if ((!Wn && !W8) || !Ws) return TORQ_ERR_NULL;
  float* wp = nullptr;
  torq_status rc = rotate_weights(W, R_inter, R_intra, d, N, workspace, workspace_bytes, stream, &wp);
  if (rc != TORQ_OK) return rc;
  if (Wn) {
    rc = torq_quantize_mxint4(wp, TORQ_F32, N, d, 1, Wn, Ws, stream);
    if (rc != TORQ_OK) return rc;
  }
  if (W8) return torq_quantize_mxint4(wp, TORQ_F32, N, d, 0, W8, Ws, stream);
  return TORQ_OK;
}

torq_status torq_merge_rotations_bf16(const void* R_inter, const void* R_intra, int64_t d, void* R_merged_bf16,
                                      void* stream) {
  if (!R_inter || !R_intra || !R_merged_bf16) return TORQ_ERR_NULL;
  if (d < 32 || d % 32 != 0 || d > (1 << 24)) return TORQ_ERR_SHAPE;
  DeviceState* st = device_state();
  if (!st) return TORQ_ERR_LAUNCH;
  if (!st->arch_ok) return TORQ_ERR_ARCH;
  merge_rotations_kernel<__nv_bfloat16><<<ew_grid(d * d, 256, st->sm_count), 256, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const __nv_bfloat16*>(R_inter), static_cast<const __nv_bfloat16*>(R_intra), d,
      static_cast<__nv_bfloat16*>(R_merged_bf16));
  return launch_status();
}

torq_status torq_merge_rotations(const void* R_inter, const void* R_intra, int64_t d, void* R_merged_f32,
                                 void* stream) {
  if (!R_inter || !R_intra || !R_merged_f32) return TORQ_ERR_NULL;
  if (d < 32 || d % 32 != 0 || d > (1 << 24)) return TORQ_ERR_SHAPE;
  DeviceState* st = device_state();
  if (!st) return TORQ_ERR_LAUNCH;
  if (!st->arch_ok) return TORQ_ERR_ARCH;
  merge_rotations_kernel<float><<<ew_grid(d * d, 256, st->sm_count), 256, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const __nv_bfloat16*>(R_inter), static_cast<const __nv_bfloat16*>(R_intra), d,
      static_cast<float*>(R_merged_f32));
  return launch_status();
}

}  // extern "C"
