// C ABI of the SGEMM-cube library (declarations and contracts: include/sgemm_cube.h).
// Host side only validates arguments, builds TMA descriptors and launches; every step of the
// computation runs in the kernels of this directory.
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>

#include <cuda.h>
#include <cuda_runtime.h>

#include "../../include/sgemm_cube.h"
#include "gemm_tc.cuh"
#include "split_kernel.cuh"

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct DeviceGuard {
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
    if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
  }
  ~DeviceGuard() {
    if (prev >= 0) cudaSetDevice(prev);
  }
};

inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

struct sgemm_cube_ctx {
  int device = 0;
  int sm_count = 0;
  unsigned int* err_dev = nullptr;   // [0] error word; [4..13] scratch of sgemm_cube_exponent_window;
                                     // [16..19] clocks and nanoseconds of the last timed tensor-core kernel
  bool err_dev_has_clock = false;    // false for the static entry point's single error word
  void* ws = nullptr;          // unfused path: FP16 words of A and B, D_hh, D_x
  size_t ws_bytes = 0;
  void* part_ws = nullptr;     // split-K partial sums
  size_t part_ws_bytes = 0;
  int split_k = 1;             // 1: split the k range of few-tile problems over idle SMs; 0: never
  void* host_ws = nullptr;     // host-buffer path: device copies of A, B, C
  size_t host_ws_bytes = 0;
  long long launches = 0;
  int kblock_termwise = 128;
  int kblock_elementwise = 64;
  int cta_pair = 2;            // 0/1: never/always 2-CTA clusters (cta_group::2); 2: see use_pair
  int strategy = 0;            // sgemm_cube: 0 auto, 1 fused kernel, 2 split kernel + 3-product kernel
  int time_kernel = 0;         // record events around the tensor-core kernel of sgemm_cube
  static constexpr int kTimedCalls = 128;           // event pairs kept (most recent calls)
  cudaEvent_t ev_ring[2 * kTimedCalls] = {};
  long long ev_calls = 0;      // timed calls since timing was switched on or last averaged
  // host-buffer path: copy streams and events of the panel pipeline (created on first use)
  static constexpr int kMaxPanels = 32;
  cudaStream_t s_in = nullptr, s_out = nullptr;
  cudaEvent_t ev_start = nullptr, ev_b = nullptr, ev_out = nullptr;
  cudaEvent_t ev_a[kMaxPanels] = {}, ev_c[kMaxPanels] = {};
  int max_pair_clusters[3] = {0, 0, 0};   // co-resident 2-CTA clusters: <1,false>, <3,false>, <3,true>
  EncodeTiledFn encode = nullptr;
  bool attrs_set = false;
};

namespace {

int grow(void** buf, size_t* have, size_t want) {
  if (*have >= want) return SGEMM_CUBE_OK;
  if (*buf) {
    if (cudaFree(*buf) != cudaSuccess) return SGEMM_CUBE_CUDA_ERROR;
    *buf = nullptr;
    *have = 0;
  }
  if (cudaMalloc(buf, want) != cudaSuccess) {
    cudaGetLastError();
    *buf = nullptr;
    return SGEMM_CUBE_ALLOC_FAILED;
  }
  *have = want;
  return SGEMM_CUBE_OK;
}

// 2-D tensor map over a row-major matrix: dims {inner, outer}, row pitch in bytes.
int make_map(sgemm_cube_ctx* h, CUtensorMap* map, CUtensorMapDataType dt, size_t elem, const void* base,
             uint64_t inner, uint64_t outer, uint64_t ld_elems, uint32_t box_inner,
             uint32_t box_outer, CUtensorMapSwizzle swz) {
  cuuint64_t dims[2] = {inner, outer};
  cuuint64_t strides[1] = {ld_elems * elem};
  cuuint32_t box[2] = {box_inner, box_outer};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = h->encode(map, dt, 2, const_cast<void*>(base), dims, strides, box, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? SGEMM_CUBE_OK : SGEMM_CUBE_CUDA_ERROR;
}

int set_kernel_attrs(sgemm_cube_ctx* h) {
  if (h->attrs_set) return SGEMM_CUBE_OK;
  const cudaFuncAttribute attr = cudaFuncAttributeMaxDynamicSharedMemorySize;
  if (cudaFuncSetAttribute(sgc::tc_gemm_kernel<1, false, false>, attr, (int)sgc::TcCfg<1, false>::SMEM_BYTES) != cudaSuccess ||
      cudaFuncSetAttribute(sgc::tc_gemm_kernel<3, false, false>, attr, (int)sgc::TcCfg<3, false>::SMEM_BYTES) != cudaSuccess ||
      cudaFuncSetAttribute(sgc::tc_gemm_kernel<3, true, false>, attr, (int)sgc::TcCfg<3, false, true>::SMEM_BYTES) != cudaSuccess ||
      cudaFuncSetAttribute(sgc::tc_gemm_kernel<1, false, true>, attr, (int)sgc::TcCfg<1, true>::SMEM_BYTES) != cudaSuccess ||
      cudaFuncSetAttribute(sgc::tc_gemm_kernel<3, false, true>, attr, (int)sgc::TcCfg<3, true>::SMEM_BYTES) != cudaSuccess ||
      cudaFuncSetAttribute(sgc::tc_gemm_kernel<3, true, true>, attr, (int)sgc::TcCfg<3, true, true>::SMEM_BYTES) != cudaSuccess ||
      cudaFuncSetAttribute(sgc::tc_gemm_kernel<3, false, false, true>, attr, (int)sgc::TcCfg<3, false>::SMEM_BYTES) != cudaSuccess ||
      cudaFuncSetAttribute(sgc::tc_gemm_kernel<3, true, false, true>, attr, (int)sgc::TcCfg<3, false, true>::SMEM_BYTES) != cudaSuccess ||
      cudaFuncSetAttribute(sgc::tc_gemm_kernel<3, false, true, true>, attr, (int)sgc::TcCfg<3, true>::SMEM_BYTES) != cudaSuccess ||
      cudaFuncSetAttribute(sgc::tc_gemm_kernel<3, true, true, true>, attr, (int)sgc::TcCfg<3, true, true>::SMEM_BYTES) != cudaSuccess) {
    cudaGetLastError();
    return SGEMM_CUBE_CUDA_ERROR;
  }
  h->attrs_set = true;
  return SGEMM_CUBE_OK;
}

// 2-CTA clusters (each CTA loads half of the B tile: two thirds of the L2 -> SM traffic of single
// CTAs, and two thirds of the tensor core's shared-memory reads) measured faster than single CTAs
// from 512^3 up (e.g. 8192^3: 458 against 439 TFLOP/s from FP16 words, 374 against 270 for the
// fused converter kernel); by default they are used whenever the problem has more than one 128-row
// block.
bool use_pair(const sgemm_cube_ctx* h, int M, int N, bool fused) {
  (void)N;
  (void)fused;
  if (h->cta_pair != 2) return h->cta_pair == 1;
  return M > sgc::kBM;
}

// Launch one tensor-core kernel: a persistent grid of single CTAs, or of 2-CTA clusters (PAIR).
template <int NTERMS, bool FUSED, bool PAIR, bool REORD>
int launch_tc_kernel_impl(sgemm_cube_ctx* h, int M, int N, const CUtensorMap& tmA0, const CUtensorMap& tmA1,
                          const CUtensorMap& tmB0, const CUtensorMap& tmB1, const sgc::TcGemmParams& p,
                          cudaStream_t st) {
  using Cfg = sgc::TcCfg<NTERMS, PAIR, FUSED>;
  auto kernel = sgc::tc_gemm_kernel<NTERMS, FUSED, PAIR, REORD>;
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.blockDim = dim3(FUSED ? sgc::kFusedThreads : sgc::kTcThreads, 1, 1);
  cfg.dynamicSmemBytes = Cfg::SMEM_BYTES;
  cfg.stream = st;
  cudaLaunchAttribute attrs[1];
  const int tiles_n = (N + sgc::kBN - 1) / sgc::kBN;
  if (PAIR) {
    attrs[0].id = cudaLaunchAttributeClusterDimension;
    attrs[0].val.clusterDim.x = 2;
    attrs[0].val.clusterDim.y = 1;
    attrs[0].val.clusterDim.z = 1;
    cfg.attrs = attrs;
    cfg.numAttrs = 1;
    int& cached = h->max_pair_clusters[FUSED ? 2 : (NTERMS == 3 ? 1 : 0)];
    if (cached == 0) {
      cfg.gridDim = dim3(2 * h->sm_count, 1, 1);
      int n = 0;
      if (cudaOccupancyMaxActiveClusters(&n, kernel, &cfg) != cudaSuccess || n < 1) {
        cudaGetLastError();
        return SGEMM_CUBE_CUDA_ERROR;
      }
      cached = n;
    }
    const int units = ((M + 2 * sgc::kBM - 1) / (2 * sgc::kBM)) * tiles_n;
    cfg.gridDim = dim3(2 * (units < cached ? units : cached), 1, 1);
  } else {
    const int units = ((M + sgc::kBM - 1) / sgc::kBM) * tiles_n * (p.ksplit > 1 ? p.ksplit : 1);
    cfg.gridDim = dim3(units < h->sm_count ? units : h->sm_count, 1, 1);
  }
  h->launches++;
  return cudaLaunchKernelEx(&cfg, kernel, tmA0, tmA1, tmB0, tmB1, p) == cudaSuccess
             ? SGEMM_CUBE_OK : (cudaGetLastError(), SGEMM_CUBE_CUDA_ERROR);
}

// The reordered elementwise order (p.order == 2) runs its own instantiation of the kernel.
template <int NTERMS, bool FUSED, bool PAIR>
int launch_tc_kernel(sgemm_cube_ctx* h, int M, int N, const CUtensorMap& tmA0, const CUtensorMap& tmA1,
                     const CUtensorMap& tmB0, const CUtensorMap& tmB1, const sgc::TcGemmParams& p,
                     cudaStream_t st) {
  if constexpr (NTERMS == 3) {
    if (p.order == SGEMM_CUBE_ELEMENTWISE_REORDERED)
      return launch_tc_kernel_impl<NTERMS, FUSED, PAIR, true>(h, M, N, tmA0, tmA1, tmB0, tmB1, p, st);
  }
  return launch_tc_kernel_impl<NTERMS, FUSED, PAIR, false>(h, M, N, tmA0, tmA1, tmB0, tmB1, p, st);
}

// Dimensions may be zero (an empty operand may then be a null pointer); negative ones are errors.
int check_gemm_dims(int M, int N, int K, int64_t lda, int64_t ldb, int64_t ldc) {
  if (M < 0 || N < 0 || K < 0) return SGEMM_CUBE_INVALID_ARG;
  if (lda < K || ldb < N || ldc < N) return SGEMM_CUBE_INVALID_ARG;
  return SGEMM_CUBE_OK;
}
bool missing_operand(int M, int N, int K, const void* A, const void* A2, const void* B, const void* B2,
                     const void* C) {
  return ((!A || !A2) && M > 0 && K > 0) || ((!B || !B2) && K > 0 && N > 0) || (!C && M > 0 && N > 0);
}
// Empty problems: nothing to do when C has no elements; an empty inner dimension leaves the empty
// sum, C = 0 (unless the call accumulates into C).  Returns true when the call is complete.
bool empty_problem(int M, int N, int K, float* C, int64_t ldc, cudaStream_t st, bool c_on_host,
                   bool keep_c, int* status) {
  if (M > 0 && N > 0 && K > 0) return false;
  *status = SGEMM_CUBE_OK;
  if (M == 0 || N == 0 || keep_c) return true;
  if (c_on_host) {
    for (int i = 0; i < M; ++i) memset(C + (size_t)i * ldc, 0, (size_t)N * sizeof(float));
  } else if (cudaMemset2DAsync(C, (size_t)ldc * sizeof(float), 0, (size_t)N * sizeof(float), M, st) !=
             cudaSuccess) {
    cudaGetLastError();
    *status = SGEMM_CUBE_CUDA_ERROR;
  }
  return true;
}

int launch_split(sgemm_cube_ctx* h, int rows, int cols, const float* X, int64_t ldx, uint16_t* hi,
                 uint16_t* lo, int64_t ldh, int s, cudaStream_t st, float pre = 1.0f) {
  const bool vec = (cols % 8 == 0) && aligned16(X) && (ldx % 4 == 0) && aligned16(hi) &&
                   aligned16(lo) && (ldh % 8 == 0);
  const long long items = vec ? (long long)rows * (cols / 8) : (long long)rows * cols;
  long long blocks = (items + 255) / 256;
  const long long cap = (long long)h->sm_count * 16;
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  if (vec)
    sgc::split_vec8_kernel<<<(unsigned)blocks, 256, 0, st>>>(rows, cols, X, ldx, hi, lo, ldh, s, pre);
  else
    sgc::split_scalar_kernel<<<(unsigned)blocks, 256, 0, st>>>(rows, cols, X, ldx, hi, lo, ldh, s, pre);
  h->launches++;
  return cudaGetLastError() == cudaSuccess ? SGEMM_CUBE_OK : SGEMM_CUBE_CUDA_ERROR;
}

// Split A (M x K) and B (K x N) of one product: one launch when both take the vector path.
int launch_split_pair(sgemm_cube_ctx* h, int M, int N, int K, const float* A, int64_t lda, uint16_t* Ahi,
                      uint16_t* Alo, int64_t ldA16, const float* B, int64_t ldb, uint16_t* Bhi,
                      uint16_t* Blo, int64_t ldB16, int s, cudaStream_t st, float pre_a = 1.0f,
                      float pre_b = 1.0f) {
  const bool vec_a = (K % 8 == 0) && aligned16(A) && (lda % 4 == 0) && aligned16(Ahi) && aligned16(Alo) &&
                     (ldA16 % 8 == 0);
  const bool vec_b = (N % 8 == 0) && aligned16(B) && (ldb % 4 == 0) && aligned16(Bhi) && aligned16(Blo) &&
                     (ldB16 % 8 == 0);
  if (!vec_a || !vec_b) {
    int rc = launch_split(h, M, K, A, lda, Ahi, Alo, ldA16, s, st, pre_a);
    if (rc) return rc;
    return launch_split(h, K, N, B, ldb, Bhi, Blo, ldB16, s, st, pre_b);
  }
  const long long items_a = (long long)M * (K / 8), items_b = (long long)K * (N / 8);
  long long blocks = (items_a + items_b + 255) / 256;
  const long long cap = (long long)h->sm_count * 16;
  if (blocks > cap) blocks = cap;
  if (blocks < 2) blocks = 2;
  long long blocks_a = (long long)((double)blocks * (double)items_a / (double)(items_a + items_b) + 0.5);
  if (blocks_a < 1) blocks_a = 1;
  if (blocks_a > blocks - 1) blocks_a = blocks - 1;
  const sgc::SplitOperand a{M, K, A, lda, Ahi, Alo, ldA16, pre_a};
  const sgc::SplitOperand b{K, N, B, ldb, Bhi, Blo, ldB16, pre_b};
  sgc::split2_vec8_kernel<<<(unsigned)blocks, 256, 0, st>>>(a, b, s, (unsigned)blocks_a);
  h->launches++;
  return cudaGetLastError() == cudaSuccess ? SGEMM_CUBE_OK : SGEMM_CUBE_CUDA_ERROR;
}

// FP16-operand tensor-core GEMM launch, NTERMS = 1 (lo pointers unused) or 3.
template <int NTERMS>
int launch_tc_gemm(sgemm_cube_ctx* h, int M, int N, int K, const uint16_t* Ahi, const uint16_t* Alo,
                   int64_t lda16, const uint16_t* Bhi, const uint16_t* Blo, int64_t ldb16, float* D,
                   int64_t ldd, int accumulate, int order, int kblock, float inv_scale,
                   cudaStream_t st, const float* Dll = nullptr, int64_t ldll = 0) {
  // Dll (NTERMS == 3, termwise only): a finished low-low product lo_A lo_B.  The kernel then
  // writes its raw sums to the partial-sum workspace even with a single k slice and the reduction
  // kernel forms the four-term result.
  using Cfg = sgc::TcCfg<NTERMS, false>;      // BK and the A swizzle do not depend on PAIR
  int rc = set_kernel_attrs(h);
  if (rc) return rc;
  CUtensorMap tmA0, tmA1, tmB0, tmB1;
  const CUtensorMapSwizzle a_swz =
      (Cfg::A_ROW_BYTES == 128) ? CU_TENSOR_MAP_SWIZZLE_128B
      : (Cfg::A_ROW_BYTES == 64) ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B;
  rc = make_map(h, &tmA0, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, Ahi, K, M, lda16, Cfg::BK, sgc::kBM, a_swz);
  if (rc) return rc;
  rc = make_map(h, &tmB0, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, Bhi, N, K, ldb16, 64, Cfg::BK,
                CU_TENSOR_MAP_SWIZZLE_128B);
  if (rc) return rc;
  if (NTERMS == 3) {
    rc = make_map(h, &tmA1, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, Alo, K, M, lda16, Cfg::BK, sgc::kBM, a_swz);
    if (rc) return rc;
    rc = make_map(h, &tmB1, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, Blo, N, K, ldb16, 64, Cfg::BK,
                  CU_TENSOR_MAP_SWIZZLE_128B);
    if (rc) return rc;
  } else {
    tmA1 = tmA0;
    tmB1 = tmB0;
  }
  sgc::TcGemmParams p;
  p.M = M; p.N = N; p.K = K;
  p.D = D; p.ldd = ldd;
  p.accumulate = accumulate;
  p.order = order;
  p.kchunk_blocks = kblock / Cfg::BK;
  if (p.kchunk_blocks < 1) p.kchunk_blocks = 1;
  p.inv_scale = inv_scale;
  p.err = h->err_dev;
  p.scale = 1.f;
  p.ksplit = 1; p.kslice_blocks = 0; p.Phh = nullptr; p.Px = nullptr; p.pstride = 0; p.ldp = 0;
  p.kclock = (NTERMS == 3 && h->time_kernel && h->err_dev_has_clock)
                 ? reinterpret_cast<unsigned long long*>(h->err_dev + 16) : nullptr;
  // Split-K: when the tiles would leave more than half of the SMs idle and k is long, cut the k
  // range into slices (whole k-blocks) so that tiles x slices fills the machine; a reduction
  // kernel adds the slices' sums.
  bool pair = use_pair(h, M, N, false);
  // Split-K runs on single CTAs; with the pair mode left to the library it takes precedence.
  if (NTERMS == 3 && h->split_k && (!pair || h->cta_pair == 2)) {
    const int tiles = ((M + sgc::kBM - 1) / sgc::kBM) * ((N + sgc::kBN - 1) / sgc::kBN);
    const int num_kb = (K + Cfg::BK - 1) / Cfg::BK;
    const int chunks = (num_kb + p.kchunk_blocks - 1) / p.kchunk_blocks;
    int want = h->sm_count / tiles;
    if (want > 16) want = 16;
    if (want > K / 1024) want = K / 1024;       // a slice shorter than 1024 costs more than it saves
    if (want >= 2 && chunks >= 2 * want) {
      const int chunks_per_slice = (chunks + want - 1) / want;
      const int slices = (chunks + chunks_per_slice - 1) / chunks_per_slice;
      const size_t ldp = round_up((size_t)N, 4);
      const size_t pstride = round_up((size_t)M * ldp, 64);
      const size_t need = (size_t)slices * pstride * 4 * (order == SGEMM_CUBE_TERMWISE ? 2 : 1);
      if (slices >= 2 && grow(&h->part_ws, &h->part_ws_bytes, need) == SGEMM_CUBE_OK) {
        pair = false;
        p.ksplit = slices;
        p.kslice_blocks = chunks_per_slice * p.kchunk_blocks;
        p.Phh = static_cast<float*>(h->part_ws);
        p.Px = p.Phh + (size_t)slices * pstride;
        p.pstride = (long long)pstride;
        p.ldp = (long long)ldp;
      }
    }
  }
  if (Dll && !p.Phh) {
    const size_t ldp = round_up((size_t)N, 4);
    const size_t pstride = round_up((size_t)M * ldp, 64);
    if ((rc = grow(&h->part_ws, &h->part_ws_bytes, 2 * pstride * 4))) return rc;
    p.Phh = static_cast<float*>(h->part_ws);
    p.Px = p.Phh + pstride;
    p.pstride = (long long)pstride;
    p.ldp = (long long)ldp;
  }
  if (p.Phh) {
    // raw sums to the workspace: k slices on single CTAs, or (four-term path, one slice) pairs
    rc = (pair && p.ksplit == 1) ? launch_tc_kernel<NTERMS, false, true>(h, M, N, tmA0, tmA1, tmB0, tmB1, p, st)
                                 : launch_tc_kernel<NTERMS, false, false>(h, M, N, tmA0, tmA1, tmB0, tmB1, p, st);
    if (rc) return rc;
    const long long total = (long long)M * N;
    long long blocks = (total + 255) / 256;
    const long long cap = (long long)h->sm_count * 16;
    if (blocks > cap) blocks = cap;
    sgc::splitk_reduce_kernel<<<(unsigned)blocks, 256, 0, st>>>(M, N, p.ksplit, p.Phh, p.Px, p.pstride, p.ldp,
                                                                 D, ldd, inv_scale,
                                                                 order == SGEMM_CUBE_TERMWISE ? 1 : 0, Dll,
                                                                 (long long)ldll);
    h->launches++;
    return cudaGetLastError() == cudaSuccess ? SGEMM_CUBE_OK : SGEMM_CUBE_CUDA_ERROR;
  }
  if (pair) {
    rc = launch_tc_kernel<NTERMS, false, true>(h, M, N, tmA0, tmA1, tmB0, tmB1, p, st);
    // Clusters that cannot be scheduled (a partitioned or partly occupied device): when the pair
    // mode was the library's own choice, single CTAs compute the same bits.
    if (rc != SGEMM_CUBE_CUDA_ERROR || h->cta_pair != 2) return rc;
  }
  return launch_tc_kernel<NTERMS, false, false>(h, M, N, tmA0, tmA1, tmB0, tmB1, p, st);
}

int launch_fused(sgemm_cube_ctx* h, int M, int N, int K, const float* A, int64_t lda, const float* B,
                 int64_t ldb, float* C, int64_t ldc, int s, int order, cudaStream_t st) {
  using Cfg = sgc::TcCfg<3, false, true>;
  int rc = set_kernel_attrs(h);
  if (rc) return rc;
  sgc::TcGemmParams p;
  p.M = M; p.N = N; p.K = K;
  p.D = C; p.ldd = ldc;
  p.accumulate = 0;
  p.order = order;
  const int kblock = (order == SGEMM_CUBE_TERMWISE) ? h->kblock_termwise : h->kblock_elementwise;
  p.kchunk_blocks = kblock / Cfg::BK;
  if (p.kchunk_blocks < 1) p.kchunk_blocks = 1;
  p.inv_scale = ldexpf(1.0f, -s);
  p.err = h->err_dev;
  p.scale = ldexpf(1.0f, s);
  p.ksplit = 1; p.kslice_blocks = 0; p.Phh = nullptr; p.Px = nullptr; p.pstride = 0; p.ldp = 0;
  p.kclock = (h->time_kernel && h->err_dev_has_clock)
                 ? reinterpret_cast<unsigned long long*>(h->err_dev + 16) : nullptr;
  // FP32 tiles as TMA stages them for the converter warps: A in boxes of {BK k, 128 rows}, B in
  // boxes of {32 columns, BK k-rows}, both with the 128-byte swizzle (rows of 128 bytes).
  CUtensorMap tmA, tmB;
  rc = make_map(h, &tmA, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, A, K, M, lda, Cfg::BK, sgc::kBM,
                CU_TENSOR_MAP_SWIZZLE_128B);
  if (rc) return rc;
  rc = make_map(h, &tmB, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, B, N, K, ldb, 32, Cfg::BK,
                CU_TENSOR_MAP_SWIZZLE_128B);
  if (rc) return rc;
  if (use_pair(h, M, N, true)) {
    rc = launch_tc_kernel<3, true, true>(h, M, N, tmA, tmA, tmB, tmB, p, st);
    // Clusters that cannot be scheduled: when the pair mode was the library's own choice, single
    // CTAs compute the same bits.
    if (rc != SGEMM_CUBE_CUDA_ERROR || h->cta_pair != 2) return rc;
  }
  return launch_tc_kernel<3, true, false>(h, M, N, tmA, tmA, tmB, tmB, p, st);
}

// sgemm_cube, strategy "two-phase": split both operands once into the handle's workspace, then one
// three-product kernel on the FP16 words.  Same arithmetic and bracketing as the fused kernel.
int launch_two_phase(sgemm_cube_ctx* h, int M, int N, int K, const float* A, int64_t lda, const float* B,
                     int64_t ldb, float* C, int64_t ldc, int s, int order, cudaStream_t st,
                     float pre_a = 1.0f, float pre_b = 1.0f) {
  const size_t ldA16 = round_up((size_t)K, 8), ldB16 = round_up((size_t)N, 8);
  const size_t szA = round_up((size_t)M * ldA16 * 2, 256), szB = round_up((size_t)K * ldB16 * 2, 256);
  int rc = grow(&h->ws, &h->ws_bytes, 2 * szA + 2 * szB);
  if (rc) return rc;
  uint8_t* w = static_cast<uint8_t*>(h->ws);
  uint16_t* Ahi = reinterpret_cast<uint16_t*>(w);
  uint16_t* Alo = reinterpret_cast<uint16_t*>(w + szA);
  uint16_t* Bhi = reinterpret_cast<uint16_t*>(w + 2 * szA);
  uint16_t* Blo = reinterpret_cast<uint16_t*>(w + 2 * szA + szB);
  if ((rc = launch_split_pair(h, M, N, K, A, lda, Ahi, Alo, (int64_t)ldA16, B, ldb, Bhi, Blo, (int64_t)ldB16, s,
                              st, pre_a, pre_b)))
    return rc;
  const int kblock = (order == SGEMM_CUBE_TERMWISE) ? h->kblock_termwise : h->kblock_elementwise;
  const int slot = (int)(h->ev_calls % sgemm_cube_ctx::kTimedCalls);
  if (h->time_kernel) cudaEventRecord(h->ev_ring[2 * slot], st);
  rc = launch_tc_gemm<3>(h, M, N, K, Ahi, Alo, (int64_t)ldA16, Bhi, Blo, (int64_t)ldB16, C, ldc, 0, order,
                         kblock, ldexpf(1.0f, -s), st);
  if (h->time_kernel) { cudaEventRecord(h->ev_ring[2 * slot + 1], st); h->ev_calls++; }
  return rc;
}

// The entry point's strategy choice.  The fused kernel re-splits every operand tile once per
// output tile, and its staging and conversion traffic shares the shared-memory pipe with the
// tensor core's operand reads, which keeps the tensor pipe about 60 % busy on large problems
// against 90 % when the split is done once up front.  Small problems keep the single launch.
int launch_sgemm_cube(sgemm_cube_ctx* h, int M, int N, int K, const float* A, int64_t lda, const float* B,
                      int64_t ldb, float* C, int64_t ldc, int s, int order, cudaStream_t st) {
  bool two_phase = (h->strategy == 2) ||
                   (h->strategy == 0 && (double)M * (double)N * (double)K >= 512.0 * 512.0 * 512.0);
  if (two_phase) {
    int rc = launch_two_phase(h, M, N, K, A, lda, B, ldb, C, ldc, s, order, st);
    if (rc != SGEMM_CUBE_ALLOC_FAILED || h->strategy == 2) return rc;
    // no room for the FP16 words: the fused kernel needs no workspace
  }
  const int slot = (int)(h->ev_calls % sgemm_cube_ctx::kTimedCalls);
  if (h->time_kernel) cudaEventRecord(h->ev_ring[2 * slot], st);
  int rc = launch_fused(h, M, N, K, A, lda, B, ldb, C, ldc, s, order, st);
  if (h->time_kernel) { cudaEventRecord(h->ev_ring[2 * slot + 1], st); h->ev_calls++; }
  return rc;
}

int host_pipelined(sgemm_cube_ctx* h, int M, int N, int K, const float* A_host, int64_t lda,
                   const float* B_host, int64_t ldb, float* C_host, int64_t ldc, int s, int order,
                   cudaStream_t st, float* dA, size_t ldA, float* dB, size_t ldB, float* dC, size_t ldC);

}  // namespace

extern "C" {

int sgemm_cube_version(void) { return 100; }

const char* sgemm_cube_status_string(int status) {
  switch (status) {
    case SGEMM_CUBE_OK: return "success";
    case SGEMM_CUBE_INVALID_ARG: return "invalid argument";
    case SGEMM_CUBE_MISALIGNED: return "pointer or leading dimension violates an alignment rule";
    case SGEMM_CUBE_CUDA_ERROR: return "CUDA runtime or driver call failed";
    case SGEMM_CUBE_DEVICE_TIMEOUT: return "a kernel gave up on a bounded wait";
    case SGEMM_CUBE_UNSUPPORTED_ARCH: return "device is not compute capability 10.x (sm_100)";
    case SGEMM_CUBE_ALLOC_FAILED: return "workspace allocation failed";
    case SGEMM_CUBE_TOO_LARGE: return "problem does not fit the fixed scratch of sgemm_cube_unfused_static";
    default: return "unknown status";
  }
}

int sgemm_cube_create(sgemm_cube_handle* out, int device) {
  if (!out) return SGEMM_CUBE_INVALID_ARG;
  *out = nullptr;
  int count = 0;
  if (cudaGetDeviceCount(&count) != cudaSuccess) { cudaGetLastError(); return SGEMM_CUBE_CUDA_ERROR; }
  if (device < 0 || device >= count) return SGEMM_CUBE_INVALID_ARG;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return SGEMM_CUBE_CUDA_ERROR;
  if (prop.major != 10) return SGEMM_CUBE_UNSUPPORTED_ARCH;
  DeviceGuard g(device);
  if (!g.ok) return SGEMM_CUBE_CUDA_ERROR;
  sgemm_cube_ctx* h = new (std::nothrow) sgemm_cube_ctx();
  if (!h) return SGEMM_CUBE_ALLOC_FAILED;
  h->device = device;
  h->sm_count = prop.multiProcessorCount;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess || !fn) {
    cudaGetLastError();
    delete h;
    return SGEMM_CUBE_CUDA_ERROR;
  }
  h->encode = reinterpret_cast<EncodeTiledFn>(fn);
  if (cudaMalloc(reinterpret_cast<void**>(&h->err_dev), 32 * sizeof(unsigned int)) != cudaSuccess) {
    cudaGetLastError();
    delete h;
    return SGEMM_CUBE_ALLOC_FAILED;
  }
  if (cudaMemset(h->err_dev, 0, 32 * sizeof(unsigned int)) != cudaSuccess) {
    cudaFree(h->err_dev);
    delete h;
    return SGEMM_CUBE_CUDA_ERROR;
  }
  h->err_dev_has_clock = true;
  *out = h;
  return SGEMM_CUBE_OK;
}

int sgemm_cube_destroy(sgemm_cube_handle h) {
  if (!h) return SGEMM_CUBE_INVALID_ARG;
  DeviceGuard g(h->device);
  int rc = SGEMM_CUBE_OK;
  if (cudaDeviceSynchronize() != cudaSuccess) rc = SGEMM_CUBE_CUDA_ERROR;
  unsigned int e = 0;
  if (rc == SGEMM_CUBE_OK && cudaMemcpy(&e, h->err_dev, sizeof(e), cudaMemcpyDeviceToHost) == cudaSuccess && e)
    rc = SGEMM_CUBE_DEVICE_TIMEOUT;
  if (h->ws) cudaFree(h->ws);
  if (h->host_ws) cudaFree(h->host_ws);
  if (h->part_ws) cudaFree(h->part_ws);
  for (cudaEvent_t e : h->ev_ring)
    if (e) cudaEventDestroy(e);
  if (h->s_in) cudaStreamDestroy(h->s_in);
  if (h->s_out) cudaStreamDestroy(h->s_out);
  if (h->ev_start) cudaEventDestroy(h->ev_start);
  if (h->ev_b) cudaEventDestroy(h->ev_b);
  if (h->ev_out) cudaEventDestroy(h->ev_out);
  for (int i = 0; i < sgemm_cube_ctx::kMaxPanels; ++i) {
    if (h->ev_a[i]) cudaEventDestroy(h->ev_a[i]);
    if (h->ev_c[i]) cudaEventDestroy(h->ev_c[i]);
  }
  cudaFree(h->err_dev);
  delete h;
  return rc;
}

int sgemm_cube_set_option(sgemm_cube_handle h, int option, int64_t value) {
  if (!h) return SGEMM_CUBE_INVALID_ARG;
  if (option == SGEMM_CUBE_OPT_CTA_PAIR) {
    if (value < 0 || value > 2) return SGEMM_CUBE_INVALID_ARG;
    h->cta_pair = (int)value;
    return SGEMM_CUBE_OK;
  }
  if (option == SGEMM_CUBE_OPT_SPLIT_K) {
    if (value != 0 && value != 1) return SGEMM_CUBE_INVALID_ARG;
    h->split_k = (int)value;
    return SGEMM_CUBE_OK;
  }
  if (option == SGEMM_CUBE_OPT_STRATEGY) {
    if (value < 0 || value > 2) return SGEMM_CUBE_INVALID_ARG;
    h->strategy = (int)value;
    return SGEMM_CUBE_OK;
  }
  if (option == SGEMM_CUBE_OPT_TIME_KERNEL) {
    if (value != 0 && value != 1) return SGEMM_CUBE_INVALID_ARG;
    DeviceGuard g(h->device);
    if (value && !h->ev_ring[0]) {
      for (cudaEvent_t& e : h->ev_ring) {
        if (cudaEventCreate(&e) != cudaSuccess) {
          cudaGetLastError();
          for (cudaEvent_t& d : h->ev_ring) {
            if (d) cudaEventDestroy(d);
            d = nullptr;
          }
          return SGEMM_CUBE_CUDA_ERROR;
        }
      }
    }
    h->time_kernel = (int)value;
    h->ev_calls = 0;
    return SGEMM_CUBE_OK;
  }
  if (value < 64 || value % 64 != 0 || value > (1 << 24)) return SGEMM_CUBE_INVALID_ARG;
  if (option == SGEMM_CUBE_OPT_TERMWISE_K_BLOCK) h->kblock_termwise = (int)value;
  else if (option == SGEMM_CUBE_OPT_ELEMENTWISE_K_BLOCK) h->kblock_elementwise = (int)value;
  else return SGEMM_CUBE_INVALID_ARG;
  return SGEMM_CUBE_OK;
}

int sgemm_cube_split(sgemm_cube_handle h, int rows, int cols, const float* X, int64_t ldx,
                     uint16_t* hi, uint16_t* lo, int64_t ldh, int scale_exp, void* stream) {
  if (!h) return SGEMM_CUBE_INVALID_ARG;
  if (rows < 0 || cols < 0 || ldx < cols || ldh < cols) return SGEMM_CUBE_INVALID_ARG;
  if (scale_exp < 0 || scale_exp > 24) return SGEMM_CUBE_INVALID_ARG;
  if (rows == 0 || cols == 0) return SGEMM_CUBE_OK;
  if (!X || !hi || !lo) return SGEMM_CUBE_INVALID_ARG;
  DeviceGuard g(h->device);
  if (!g.ok) return SGEMM_CUBE_CUDA_ERROR;
  return launch_split(h, rows, cols, X, ldx, hi, lo, ldh, scale_exp, static_cast<cudaStream_t>(stream));
}

int sgemm_cube(sgemm_cube_handle h, int M, int N, int K, const float* A, int64_t lda, const float* B,
               int64_t ldb, float* C, int64_t ldc, int scale_exp, int order, void* stream) {
  if (!h) return SGEMM_CUBE_INVALID_ARG;
  int rc = check_gemm_dims(M, N, K, lda, ldb, ldc);
  if (rc) return rc;
  if (missing_operand(M, N, K, A, A, B, B, C)) return SGEMM_CUBE_INVALID_ARG;
  if (scale_exp < 0 || scale_exp > 24) return SGEMM_CUBE_INVALID_ARG;
  if (order < SGEMM_CUBE_TERMWISE || order > SGEMM_CUBE_ELEMENTWISE_REORDERED) return SGEMM_CUBE_INVALID_ARG;
  DeviceGuard g(h->device);
  if (!g.ok) return SGEMM_CUBE_CUDA_ERROR;
  if (empty_problem(M, N, K, C, ldc, static_cast<cudaStream_t>(stream), false, false, &rc)) return rc;
  if (!aligned16(A) || !aligned16(B) || (lda % 4) || (ldb % 4)) return SGEMM_CUBE_MISALIGNED;
  return launch_sgemm_cube(h, M, N, K, A, lda, B, ldb, C, ldc, scale_exp, order,
                           static_cast<cudaStream_t>(stream));
}

int sgemm_cube_presplit(sgemm_cube_handle h, int M, int N, int K, const uint16_t* Ahi,
                        const uint16_t* Alo, int64_t lda16, const uint16_t* Bhi, const uint16_t* Blo,
                        int64_t ldb16, float* C, int64_t ldc, int scale_exp, int order, void* stream) {
  if (!h) return SGEMM_CUBE_INVALID_ARG;
  int rc = check_gemm_dims(M, N, K, lda16, ldb16, ldc);
  if (rc) return rc;
  if (missing_operand(M, N, K, Ahi, Alo, Bhi, Blo, C)) return SGEMM_CUBE_INVALID_ARG;
  if (scale_exp < 0 || scale_exp > 24) return SGEMM_CUBE_INVALID_ARG;
  if (order < SGEMM_CUBE_TERMWISE || order > SGEMM_CUBE_ELEMENTWISE_REORDERED) return SGEMM_CUBE_INVALID_ARG;
  DeviceGuard g(h->device);
  if (!g.ok) return SGEMM_CUBE_CUDA_ERROR;
  if (empty_problem(M, N, K, C, ldc, static_cast<cudaStream_t>(stream), false, false, &rc)) return rc;
  if (!aligned16(Ahi) || !aligned16(Alo) || !aligned16(Bhi) || !aligned16(Blo) || (lda16 % 8) ||
      (ldb16 % 8))
    return SGEMM_CUBE_MISALIGNED;
  const int kblock = (order == SGEMM_CUBE_TERMWISE) ? h->kblock_termwise : h->kblock_elementwise;
  return launch_tc_gemm<3>(h, M, N, K, Ahi, Alo, lda16, Bhi, Blo, ldb16, C, ldc, 0, order, kblock,
                           ldexpf(1.0f, -scale_exp), static_cast<cudaStream_t>(stream));
}

int sgemm_cube_hgemm(sgemm_cube_handle h, int M, int N, int K, const uint16_t* A16, int64_t lda16,
                     const uint16_t* B16, int64_t ldb16, float* D, int64_t ldd, int accumulate,
                     void* stream) {
  if (!h) return SGEMM_CUBE_INVALID_ARG;
  int rc = check_gemm_dims(M, N, K, lda16, ldb16, ldd);
  if (rc) return rc;
  if (missing_operand(M, N, K, A16, A16, B16, B16, D)) return SGEMM_CUBE_INVALID_ARG;
  DeviceGuard g(h->device);
  if (!g.ok) return SGEMM_CUBE_CUDA_ERROR;
  if (empty_problem(M, N, K, D, ldd, static_cast<cudaStream_t>(stream), false, accumulate != 0, &rc)) return rc;
  if (!aligned16(A16) || !aligned16(B16) || (lda16 % 8) || (ldb16 % 8)) return SGEMM_CUBE_MISALIGNED;
  return launch_tc_gemm<1>(h, M, N, K, A16, nullptr, lda16, B16, nullptr, ldb16, D, ldd,
                           accumulate ? 1 : 0, 0, h->kblock_termwise, 1.0f,
                           static_cast<cudaStream_t>(stream));
}

int sgemm_cube_unfused(sgemm_cube_handle h, int M, int N, int K, const float* A, int64_t lda,
                       const float* B, int64_t ldb, float* C, int64_t ldc, int scale_exp, int order,
                       void* stream) {
  if (!h) return SGEMM_CUBE_INVALID_ARG;
  int rc = check_gemm_dims(M, N, K, lda, ldb, ldc);
  if (rc) return rc;
  if (missing_operand(M, N, K, A, A, B, B, C)) return SGEMM_CUBE_INVALID_ARG;
  if (scale_exp < 0 || scale_exp > 24) return SGEMM_CUBE_INVALID_ARG;
  if (order != SGEMM_CUBE_TERMWISE) return SGEMM_CUBE_INVALID_ARG;
  DeviceGuard g(h->device);
  if (!g.ok) return SGEMM_CUBE_CUDA_ERROR;
  if (empty_problem(M, N, K, C, ldc, static_cast<cudaStream_t>(stream), false, false, &rc)) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // Workspace layout: A_hi, A_lo (M x ldA16), B_hi, B_lo (K x ldB16), D_hh, D_x (M x ldD).
  const size_t ldA16 = round_up((size_t)K, 8), ldB16 = round_up((size_t)N, 8);
  const size_t ldD = round_up((size_t)N, 4);
  const size_t szA = round_up((size_t)M * ldA16 * 2, 256), szB = round_up((size_t)K * ldB16 * 2, 256);
  const size_t szD = round_up((size_t)M * ldD * 4, 256);
  rc = grow(&h->ws, &h->ws_bytes, 2 * szA + 2 * szB + 2 * szD);
  if (rc) return rc;
  uint8_t* w = static_cast<uint8_t*>(h->ws);
  uint16_t* Ahi = reinterpret_cast<uint16_t*>(w);
  uint16_t* Alo = reinterpret_cast<uint16_t*>(w + szA);
  uint16_t* Bhi = reinterpret_cast<uint16_t*>(w + 2 * szA);
  uint16_t* Blo = reinterpret_cast<uint16_t*>(w + 2 * szA + szB);
  float* Dhh = reinterpret_cast<float*>(w + 2 * szA + 2 * szB);
  float* Dx = reinterpret_cast<float*>(w + 2 * szA + 2 * szB + szD);
  const float inv = ldexpf(1.0f, -scale_exp);
  const int kb = h->kblock_termwise;
  if ((rc = launch_split_pair(h, M, N, K, A, lda, Ahi, Alo, (int64_t)ldA16, B, ldb, Bhi, Blo, (int64_t)ldB16,
                              scale_exp, st)))
    return rc;
  if ((rc = launch_tc_gemm<1>(h, M, N, K, Ahi, nullptr, ldA16, Bhi, nullptr, ldB16, Dhh, ldD, 0, 0, kb, 1.f, st))) return rc;
  if ((rc = launch_tc_gemm<1>(h, M, N, K, Alo, nullptr, ldA16, Bhi, nullptr, ldB16, Dx, ldD, 0, 0, kb, 1.f, st))) return rc;
  if ((rc = launch_tc_gemm<1>(h, M, N, K, Ahi, nullptr, ldA16, Blo, nullptr, ldB16, Dx, ldD, 1, 0, kb, 1.f, st))) return rc;
  const long long total = (long long)M * N;
  long long blocks = (total + 255) / 256;
  const long long cap = (long long)h->sm_count * 16;
  if (blocks > cap) blocks = cap;
  sgc::combine_kernel<<<(unsigned)blocks, 256, 0, st>>>(M, N, Dhh, Dx, (long long)ldD, C, ldc, inv);
  h->launches++;
  return cudaGetLastError() == cudaSuccess ? SGEMM_CUBE_OK : SGEMM_CUBE_CUDA_ERROR;
}

int sgemm_cube_four_term(sgemm_cube_handle h, int M, int N, int K, const float* A, int64_t lda,
                         const float* B, int64_t ldb, float* C, int64_t ldc, int scale_exp,
                         void* stream) {
  if (!h) return SGEMM_CUBE_INVALID_ARG;
  int rc = check_gemm_dims(M, N, K, lda, ldb, ldc);
  if (rc) return rc;
  if (missing_operand(M, N, K, A, A, B, B, C)) return SGEMM_CUBE_INVALID_ARG;
  if (scale_exp < 0 || scale_exp > 24) return SGEMM_CUBE_INVALID_ARG;
  DeviceGuard g(h->device);
  if (!g.ok) return SGEMM_CUBE_CUDA_ERROR;
  if (empty_problem(M, N, K, C, ldc, static_cast<cudaStream_t>(stream), false, false, &rc)) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // Workspace layout: A_hi, A_lo (M x ldA16), B_hi, B_lo (K x ldB16), D_ll (M x ldD).
  const size_t ldA16 = round_up((size_t)K, 8), ldB16 = round_up((size_t)N, 8);
  const size_t ldD = round_up((size_t)N, 4);
  const size_t szA = round_up((size_t)M * ldA16 * 2, 256), szB = round_up((size_t)K * ldB16 * 2, 256);
  const size_t szD = round_up((size_t)M * ldD * 4, 256);
  rc = grow(&h->ws, &h->ws_bytes, 2 * szA + 2 * szB + szD);
  if (rc) return rc;
  uint8_t* w = static_cast<uint8_t*>(h->ws);
  uint16_t* Ahi = reinterpret_cast<uint16_t*>(w);
  uint16_t* Alo = reinterpret_cast<uint16_t*>(w + szA);
  uint16_t* Bhi = reinterpret_cast<uint16_t*>(w + 2 * szA);
  uint16_t* Blo = reinterpret_cast<uint16_t*>(w + 2 * szA + szB);
  float* Dll = reinterpret_cast<float*>(w + 2 * szA + 2 * szB);
  const int kb = h->kblock_termwise;
  if ((rc = launch_split_pair(h, M, N, K, A, lda, Ahi, Alo, (int64_t)ldA16, B, ldb, Bhi, Blo, (int64_t)ldB16,
                              scale_exp, st)))
    return rc;
  if ((rc = launch_tc_gemm<1>(h, M, N, K, Alo, nullptr, ldA16, Blo, nullptr, ldB16, Dll, ldD, 0, 0, kb, 1.f, st)))
    return rc;
  return launch_tc_gemm<3>(h, M, N, K, Ahi, Alo, (int64_t)ldA16, Bhi, Blo, (int64_t)ldB16, C, ldc, 0,
                           SGEMM_CUBE_TERMWISE, kb, ldexpf(1.0f, -scale_exp), st, Dll, (int64_t)ldD);
}

int sgemm_cube_host(sgemm_cube_handle h, int M, int N, int K, const float* A_host, int64_t lda,
                    const float* B_host, int64_t ldb, float* C_host, int64_t ldc, int scale_exp,
                    int order, void* stream) {
  if (!h) return SGEMM_CUBE_INVALID_ARG;
  int rc = check_gemm_dims(M, N, K, lda, ldb, ldc);
  if (rc) return rc;
  if (missing_operand(M, N, K, A_host, A_host, B_host, B_host, C_host)) return SGEMM_CUBE_INVALID_ARG;
  if (scale_exp < 0 || scale_exp > 24) return SGEMM_CUBE_INVALID_ARG;
  if (order < SGEMM_CUBE_TERMWISE || order > SGEMM_CUBE_ELEMENTWISE_REORDERED) return SGEMM_CUBE_INVALID_ARG;
  DeviceGuard g(h->device);
  if (!g.ok) return SGEMM_CUBE_CUDA_ERROR;
  if (empty_problem(M, N, K, C_host, ldc, static_cast<cudaStream_t>(stream), true, false, &rc)) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t ldA = round_up((size_t)K, 4), ldB = round_up((size_t)N, 4), ldC = ldB;
  const size_t szA = round_up((size_t)M * ldA * 4, 256), szB = round_up((size_t)K * ldB * 4, 256);
  const size_t szC = round_up((size_t)M * ldC * 4, 256);
  rc = grow(&h->host_ws, &h->host_ws_bytes, szA + szB + szC);
  if (rc) return rc;
  uint8_t* w = static_cast<uint8_t*>(h->host_ws);
  float* dA = reinterpret_cast<float*>(w);
  float* dB = reinterpret_cast<float*>(w + szA);
  float* dC = reinterpret_cast<float*>(w + szA + szB);
  if (h->strategy != SGEMM_CUBE_STRATEGY_FUSED && M >= 1024 &&
      (double)M * (double)N * (double)K >= 1024.0 * 1024.0 * 1024.0) {
    rc = host_pipelined(h, M, N, K, A_host, lda, B_host, ldb, C_host, ldc, scale_exp, order, st, dA, ldA,
                        dB, ldB, dC, ldC);
    if (rc == SGEMM_CUBE_OK) return sgemm_cube_check(h, stream, nullptr);
    if (rc != SGEMM_CUBE_ALLOC_FAILED) return rc;
    // no room for the FP16 words: fall through to the plain sequence below
  }
  if (cudaMemcpy2DAsync(dA, ldA * 4, A_host, (size_t)lda * 4, (size_t)K * 4, M, cudaMemcpyHostToDevice, st) != cudaSuccess ||
      cudaMemcpy2DAsync(dB, ldB * 4, B_host, (size_t)ldb * 4, (size_t)N * 4, K, cudaMemcpyHostToDevice, st) != cudaSuccess) {
    cudaGetLastError();
    return SGEMM_CUBE_CUDA_ERROR;
  }
  rc = launch_sgemm_cube(h, M, N, K, dA, (int64_t)ldA, dB, (int64_t)ldB, dC, (int64_t)ldC, scale_exp, order, st);
  if (rc) return rc;
  if (cudaMemcpy2DAsync(C_host, (size_t)ldc * 4, dC, ldC * 4, (size_t)N * 4, M, cudaMemcpyDeviceToHost, st) != cudaSuccess) {
    cudaGetLastError();
    return SGEMM_CUBE_CUDA_ERROR;
  }
  return sgemm_cube_check(h, stream, nullptr);
}

}  // extern "C"

namespace {

int host_pipeline_setup(sgemm_cube_ctx* h) {
  if (h->s_in) return SGEMM_CUBE_OK;
  bool ok = cudaStreamCreateWithFlags(&h->s_in, cudaStreamNonBlocking) == cudaSuccess &&
            cudaStreamCreateWithFlags(&h->s_out, cudaStreamNonBlocking) == cudaSuccess &&
            cudaEventCreateWithFlags(&h->ev_start, cudaEventDisableTiming) == cudaSuccess &&
            cudaEventCreateWithFlags(&h->ev_b, cudaEventDisableTiming) == cudaSuccess &&
            cudaEventCreateWithFlags(&h->ev_out, cudaEventDisableTiming) == cudaSuccess;
  for (int i = 0; ok && i < sgemm_cube_ctx::kMaxPanels; ++i)
    ok = cudaEventCreateWithFlags(&h->ev_a[i], cudaEventDisableTiming) == cudaSuccess &&
         cudaEventCreateWithFlags(&h->ev_c[i], cudaEventDisableTiming) == cudaSuccess;
  if (!ok) { cudaGetLastError(); return SGEMM_CUBE_CUDA_ERROR; }
  return SGEMM_CUBE_OK;
}

// Host-buffer path for large problems: B is copied and split once; A and C move in row panels so
// that the upload of panel p + 1, the products of panel p and the download of panel p - 1 overlap
// (one copy stream per direction besides the caller's stream).  Same kernels, same per-element
// arithmetic as sgemm_cube's two-phase strategy: a row panel of C depends on its rows of A only.
int host_pipelined(sgemm_cube_ctx* h, int M, int N, int K, const float* A_host, int64_t lda,
                   const float* B_host, int64_t ldb, float* C_host, int64_t ldc, int s, int order,
                   cudaStream_t st, float* dA, size_t ldA, float* dB, size_t ldB, float* dC, size_t ldC) {
  int rc = host_pipeline_setup(h);
  if (rc) return rc;
  const size_t ldA16 = round_up((size_t)K, 8), ldB16 = round_up((size_t)N, 8);
  const size_t szA = round_up((size_t)M * ldA16 * 2, 256), szB = round_up((size_t)K * ldB16 * 2, 256);
  rc = grow(&h->ws, &h->ws_bytes, 2 * szA + 2 * szB);
  if (rc) return rc;
  uint8_t* w = static_cast<uint8_t*>(h->ws);
  uint16_t* Ahi = reinterpret_cast<uint16_t*>(w);
  uint16_t* Alo = reinterpret_cast<uint16_t*>(w + szA);
  uint16_t* Bhi = reinterpret_cast<uint16_t*>(w + 2 * szA);
  uint16_t* Blo = reinterpret_cast<uint16_t*>(w + 2 * szA + szB);
  int panel = (int)round_up((size_t)(M + 7) / 8, 256);           // about eight panels
  while ((M + panel - 1) / panel > sgemm_cube_ctx::kMaxPanels) panel *= 2;
  const int panels = (M + panel - 1) / panel;
  const int kblock = (order == SGEMM_CUBE_TERMWISE) ? h->kblock_termwise : h->kblock_elementwise;
  const float inv = ldexpf(1.0f, -s);
  bool ok = true;
  // the copy streams start after whatever the caller's stream holds (earlier users of the buffers)
  ok = ok && cudaEventRecord(h->ev_start, st) == cudaSuccess;
  ok = ok && cudaStreamWaitEvent(h->s_in, h->ev_start, 0) == cudaSuccess;
  ok = ok && cudaStreamWaitEvent(h->s_out, h->ev_start, 0) == cudaSuccess;
  ok = ok && cudaMemcpy2DAsync(dB, ldB * 4, B_host, (size_t)ldb * 4, (size_t)N * 4, K,
                               cudaMemcpyHostToDevice, h->s_in) == cudaSuccess;
  ok = ok && cudaEventRecord(h->ev_b, h->s_in) == cudaSuccess;
  ok = ok && cudaStreamWaitEvent(st, h->ev_b, 0) == cudaSuccess;
  if (!ok) { cudaGetLastError(); return SGEMM_CUBE_CUDA_ERROR; }
  if ((rc = launch_split(h, K, N, dB, (int64_t)ldB, Bhi, Blo, (int64_t)ldB16, s, st))) return rc;
  for (int p = 0; p < panels; ++p) {
    const int r0 = p * panel;
    const int rows = (M - r0 < panel) ? (M - r0) : panel;
    ok = ok && cudaMemcpy2DAsync(dA + (size_t)r0 * ldA, ldA * 4, A_host + (size_t)r0 * lda, (size_t)lda * 4,
                                 (size_t)K * 4, rows, cudaMemcpyHostToDevice, h->s_in) == cudaSuccess;
    ok = ok && cudaEventRecord(h->ev_a[p], h->s_in) == cudaSuccess;
    ok = ok && cudaStreamWaitEvent(st, h->ev_a[p], 0) == cudaSuccess;
    if (!ok) { cudaGetLastError(); return SGEMM_CUBE_CUDA_ERROR; }
    if ((rc = launch_split(h, rows, K, dA + (size_t)r0 * ldA, (int64_t)ldA, Ahi + (size_t)r0 * ldA16,
                           Alo + (size_t)r0 * ldA16, (int64_t)ldA16, s, st))) return rc;
    if ((rc = launch_tc_gemm<3>(h, rows, N, K, Ahi + (size_t)r0 * ldA16, Alo + (size_t)r0 * ldA16,
                                (int64_t)ldA16, Bhi, Blo, (int64_t)ldB16, dC + (size_t)r0 * ldC, (int64_t)ldC,
                                0, order, kblock, inv, st))) return rc;
    ok = ok && cudaEventRecord(h->ev_c[p], st) == cudaSuccess;
    ok = ok && cudaStreamWaitEvent(h->s_out, h->ev_c[p], 0) == cudaSuccess;
    ok = ok && cudaMemcpy2DAsync(C_host + (size_t)r0 * ldc, (size_t)ldc * 4, dC + (size_t)r0 * ldC, ldC * 4,
                                 (size_t)N * 4, rows, cudaMemcpyDeviceToHost, h->s_out) == cudaSuccess;
    if (!ok) { cudaGetLastError(); return SGEMM_CUBE_CUDA_ERROR; }
  }
  ok = ok && cudaEventRecord(h->ev_out, h->s_out) == cudaSuccess;
  ok = ok && cudaStreamWaitEvent(st, h->ev_out, 0) == cudaSuccess;
  if (!ok) { cudaGetLastError(); return SGEMM_CUBE_CUDA_ERROR; }
  return SGEMM_CUBE_OK;
}

}  // namespace

extern "C" {

int sgemm_cube_check(sgemm_cube_handle h, void* stream, uint32_t* detail_out) {
  if (!h) return SGEMM_CUBE_INVALID_ARG;
  DeviceGuard g(h->device);
  if (!g.ok) return SGEMM_CUBE_CUDA_ERROR;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cudaStreamSynchronize(st) != cudaSuccess) { cudaGetLastError(); return SGEMM_CUBE_CUDA_ERROR; }
  unsigned int e = 0;
  if (cudaMemcpy(&e, h->err_dev, sizeof(e), cudaMemcpyDeviceToHost) != cudaSuccess) {
    cudaGetLastError();
    return SGEMM_CUBE_CUDA_ERROR;
  }
  if (detail_out) *detail_out = e;
  if (e) {
    cudaMemset(h->err_dev, 0, sizeof(e));
    return SGEMM_CUBE_DEVICE_TIMEOUT;
  }
  return SGEMM_CUBE_OK;
}

int sgemm_cube_exponent_window(sgemm_cube_handle h, int rows, int cols, const float* X, int64_t ldx,
                               int64_t* window_out, void* stream) {
  if (!h || !X || !window_out) return SGEMM_CUBE_INVALID_ARG;
  if (rows <= 0 || cols <= 0 || ldx < cols) return SGEMM_CUBE_INVALID_ARG;
  DeviceGuard g(h->device);
  if (!g.ok) return SGEMM_CUBE_CUDA_ERROR;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  long long* dev = reinterpret_cast<long long*>(h->err_dev + 4);
  const long long init[5] = {127, -127, 0, 0, 0};
  if (cudaMemcpyAsync(dev, init, sizeof(init), cudaMemcpyHostToDevice, st) != cudaSuccess) {
    cudaGetLastError();
    return SGEMM_CUBE_CUDA_ERROR;
  }
  const long long total = (long long)rows * cols;
  long long blocks = (total + 1023) / 1024;
  const long long cap = (long long)h->sm_count * 16;
  if (blocks > cap) blocks = cap;
  sgc::exponent_window_kernel<<<(unsigned)blocks, 256, 0, st>>>(rows, cols, X, ldx, dev);
  h->launches++;
  if (cudaGetLastError() != cudaSuccess) return SGEMM_CUBE_CUDA_ERROR;
  long long res[5];
  if (cudaMemcpyAsync(res, dev, sizeof(res), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess) {
    cudaGetLastError();
    return SGEMM_CUBE_CUDA_ERROR;
  }
  for (int i = 0; i < 5; ++i) window_out[i] = res[i];
  return SGEMM_CUBE_OK;
}

int sgemm_cube_hi_exponent_range(sgemm_cube_handle h, int rows, int cols, const float* X, int64_t ldx,
                                 int64_t* range_out, void* stream) {
  if (!h || !X || !range_out) return SGEMM_CUBE_INVALID_ARG;
  if (rows <= 0 || cols <= 0 || ldx < cols) return SGEMM_CUBE_INVALID_ARG;
  DeviceGuard g(h->device);
  if (!g.ok) return SGEMM_CUBE_CUDA_ERROR;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  long long* dev = reinterpret_cast<long long*>(h->err_dev + 4);
  const long long init[3] = {127, -127, 0};
  if (cudaMemcpyAsync(dev, init, sizeof(init), cudaMemcpyHostToDevice, st) != cudaSuccess) {
    cudaGetLastError();
    return SGEMM_CUBE_CUDA_ERROR;
  }
  const long long total = (long long)rows * cols;
  long long blocks = (total + 1023) / 1024;
  const long long cap = (long long)h->sm_count * 16;
  if (blocks > cap) blocks = cap;
  sgc::hi_exponent_range_kernel<<<(unsigned)blocks, 256, 0, st>>>(rows, cols, X, ldx, dev);
  h->launches++;
  if (cudaGetLastError() != cudaSuccess) return SGEMM_CUBE_CUDA_ERROR;
  long long res[3];
  if (cudaMemcpyAsync(res, dev, sizeof(res), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess) {
    cudaGetLastError();
    return SGEMM_CUBE_CUDA_ERROR;
  }
  for (int i = 0; i < 3; ++i) range_out[i] = res[i];
  return SGEMM_CUBE_OK;
}

int sgemm_cube_choose_input_scaling(const int64_t* range_a, const int64_t* range_b, int* p_a_out,
                                    int* p_b_out, int* scale_exp_out, int* protected_out) {
  if (!range_a || !range_b || !p_a_out || !p_b_out || !scale_exp_out) return SGEMM_CUBE_INVALID_ARG;
  bool ok = true;
  const int64_t* rs[2] = {range_a, range_b};
  int* ps[2] = {p_a_out, p_b_out};
  for (int i = 0; i < 2; ++i) {
    const int64_t e_min = rs[i][0], e_max = rs[i][1];
    int p = 0;
    if (e_max >= e_min) {                        // the operand has a non-zero finite entry
      int64_t q = 15 - e_max;                    // largest high word into the top normal binade
      if (q > 126) q = 126;
      if (q < -126) q = -126;
      p = (int)q;
      ok = ok && (e_min + p >= -14) && (e_max + p <= 15);
    }
    ok = ok && rs[i][2] == 0;
    *ps[i] = p;
  }
  *scale_exp_out = 11;                           // Eq. sf_bounds for the whole normal window
  if (protected_out) *protected_out = ok ? 1 : 0;
  return SGEMM_CUBE_OK;
}

int sgemm_cube_scaled(sgemm_cube_handle h, int M, int N, int K, const float* A, int64_t lda,
                      const float* B, int64_t ldb, float* C, int64_t ldc, int p_a, int p_b,
                      int scale_exp, int order, void* stream) {
  if (!h) return SGEMM_CUBE_INVALID_ARG;
  int rc = check_gemm_dims(M, N, K, lda, ldb, ldc);
  if (rc) return rc;
  if (missing_operand(M, N, K, A, A, B, B, C)) return SGEMM_CUBE_INVALID_ARG;
  if (scale_exp < 0 || scale_exp > 24) return SGEMM_CUBE_INVALID_ARG;
  if (order < SGEMM_CUBE_TERMWISE || order > SGEMM_CUBE_ELEMENTWISE_REORDERED) return SGEMM_CUBE_INVALID_ARG;
  if (p_a < -126 || p_a > 126 || p_b < -126 || p_b > 126) return SGEMM_CUBE_INVALID_ARG;
  DeviceGuard g(h->device);
  if (!g.ok) return SGEMM_CUBE_CUDA_ERROR;
  if (empty_problem(M, N, K, C, ldc, static_cast<cudaStream_t>(stream), false, false, &rc)) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  rc = launch_two_phase(h, M, N, K, A, lda, B, ldb, C, ldc, scale_exp, order, st, ldexpf(1.0f, p_a),
                        ldexpf(1.0f, p_b));
  if (rc) return rc;
  if (p_a + p_b != 0) {
    const long long total = (long long)M * N;
    long long blocks = (total + 255) / 256;
    const long long cap = (long long)h->sm_count * 16;
    if (blocks > cap) blocks = cap;
    sgc::scale_pow2_kernel<<<(unsigned)blocks, 256, 0, st>>>(M, N, C, ldc, -(p_a + p_b));
    h->launches++;
    if (cudaGetLastError() != cudaSuccess) return SGEMM_CUBE_CUDA_ERROR;
  }
  return SGEMM_CUBE_OK;
}

int sgemm_cube_auto_scaled(sgemm_cube_handle h, int M, int N, int K, const float* A, int64_t lda,
                           const float* B, int64_t ldb, float* C, int64_t ldc, int order, void* stream,
                           int* chosen_out) {
  if (!h) return SGEMM_CUBE_INVALID_ARG;
  int rc = check_gemm_dims(M, N, K, lda, ldb, ldc);
  if (rc) return rc;
  if (missing_operand(M, N, K, A, A, B, B, C)) return SGEMM_CUBE_INVALID_ARG;
  if (M == 0 || N == 0 || K == 0)
    return sgemm_cube_scaled(h, M, N, K, A, lda, B, ldb, C, ldc, 0, 0, 11, order, stream);
  int64_t ra[3], rb[3];
  if ((rc = sgemm_cube_hi_exponent_range(h, M, K, A, lda, ra, stream))) return rc;
  if ((rc = sgemm_cube_hi_exponent_range(h, K, N, B, ldb, rb, stream))) return rc;
  int p_a = 0, p_b = 0, s = 11, prot = 0;
  if ((rc = sgemm_cube_choose_input_scaling(ra, rb, &p_a, &p_b, &s, &prot))) return rc;
  if (chosen_out) { chosen_out[0] = p_a; chosen_out[1] = p_b; chosen_out[2] = s; chosen_out[3] = prot; }
  return sgemm_cube_scaled(h, M, N, K, A, lda, B, ldb, C, ldc, p_a, p_b, s, order, stream);
}

int sgemm_cube_residual_overflow_count(sgemm_cube_handle h, int rows, int cols, const uint16_t* hi,
                                       const uint16_t* lo, int64_t ldh, int64_t* count_out, void* stream) {
  if (!h || !count_out) return SGEMM_CUBE_INVALID_ARG;
  if (rows < 0 || cols < 0 || ldh < cols) return SGEMM_CUBE_INVALID_ARG;
  *count_out = 0;
  if (rows == 0 || cols == 0) return SGEMM_CUBE_OK;
  if (!hi || !lo) return SGEMM_CUBE_INVALID_ARG;
  DeviceGuard g(h->device);
  if (!g.ok) return SGEMM_CUBE_CUDA_ERROR;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  unsigned long long* dev = reinterpret_cast<unsigned long long*>(h->err_dev + 4);
  if (cudaMemsetAsync(dev, 0, sizeof(unsigned long long), st) != cudaSuccess) {
    cudaGetLastError();
    return SGEMM_CUBE_CUDA_ERROR;
  }
  const long long total = (long long)rows * cols;
  long long blocks = (total + 1023) / 1024;
  const long long cap = (long long)h->sm_count * 16;
  if (blocks > cap) blocks = cap;
  sgc::residual_overflow_kernel<<<(unsigned)blocks, 256, 0, st>>>(rows, cols, hi, lo, ldh, dev);
  h->launches++;
  if (cudaGetLastError() != cudaSuccess) return SGEMM_CUBE_CUDA_ERROR;
  unsigned long long res = 0;
  if (cudaMemcpyAsync(&res, dev, sizeof(res), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess) {
    cudaGetLastError();
    return SGEMM_CUBE_CUDA_ERROR;
  }
  *count_out = (int64_t)res;
  return SGEMM_CUBE_OK;
}

int sgemm_cube_choose_scale_exp(const int64_t* window_a, const int64_t* window_b, int* scale_exp_out,
                                int* protected_out) {
  if (!window_a || !window_b || !scale_exp_out) return SGEMM_CUBE_INVALID_ARG;
  const bool any_a = window_a[1] >= window_a[0], any_b = window_b[1] >= window_b[0];
  int e_max = -127, e_min = 127;
  if (any_a) { e_max = (int)window_a[1]; e_min = (int)window_a[0]; }
  if (any_b) {
    e_max = (int)window_b[1] > e_max ? (int)window_b[1] : e_max;
    e_min = (int)window_b[0] < e_min ? (int)window_b[0] : e_min;
  }
  int s = 15;                                  // nothing normal and finite: any scale will do
  if (any_a || any_b) {
    s = 26 - e_max;                            // Rule 2 / upper end of Eq. sf_bounds
    if (s > 15) s = 15;
    if (s < 0) s = 0;
  }
  *scale_exp_out = s;
  if (protected_out) {
    const bool clean = window_a[2] == 0 && window_a[3] == 0 && window_b[2] == 0 && window_b[3] == 0;
    const bool lower_ok = !(any_a || any_b) || s >= -3 - e_min;    // lower end of Eq. sf_bounds
    *protected_out = (clean && lower_ok) ? 1 : 0;
  }
  return SGEMM_CUBE_OK;
}

int64_t sgemm_cube_launch_count(sgemm_cube_handle h) { return h ? h->launches : -1; }

int sgemm_cube_last_kernel_ms(sgemm_cube_handle h, float* ms_out) {
  if (!h || !ms_out || !h->time_kernel || h->ev_calls == 0) return SGEMM_CUBE_INVALID_ARG;
  DeviceGuard g(h->device);
  const int slot = (int)((h->ev_calls - 1) % sgemm_cube_ctx::kTimedCalls);
  if (cudaEventSynchronize(h->ev_ring[2 * slot + 1]) != cudaSuccess ||
      cudaEventElapsedTime(ms_out, h->ev_ring[2 * slot], h->ev_ring[2 * slot + 1]) != cudaSuccess) {
    cudaGetLastError();
    return SGEMM_CUBE_CUDA_ERROR;
  }
  return SGEMM_CUBE_OK;
}

int sgemm_cube_mean_kernel_ms(sgemm_cube_handle h, float* mean_ms_out, int* calls_out) {
  if (!h || !mean_ms_out || !h->time_kernel || h->ev_calls == 0) return SGEMM_CUBE_INVALID_ARG;
  DeviceGuard g(h->device);
  const long long n = h->ev_calls < sgemm_cube_ctx::kTimedCalls ? h->ev_calls : sgemm_cube_ctx::kTimedCalls;
  double sum = 0.0;
  for (long long i = 0; i < n; ++i) {
    const int slot = (int)((h->ev_calls - 1 - i) % sgemm_cube_ctx::kTimedCalls);
    float ms = 0.f;
    if (cudaEventSynchronize(h->ev_ring[2 * slot + 1]) != cudaSuccess ||
        cudaEventElapsedTime(&ms, h->ev_ring[2 * slot], h->ev_ring[2 * slot + 1]) != cudaSuccess) {
      cudaGetLastError();
      return SGEMM_CUBE_CUDA_ERROR;
    }
    sum += ms;
  }
  *mean_ms_out = (float)(sum / (double)n);
  if (calls_out) *calls_out = (int)n;
  h->ev_calls = 0;
  return SGEMM_CUBE_OK;
}

int sgemm_cube_last_kernel_clock(sgemm_cube_handle h, uint64_t* sm_cycles_out, uint64_t* ns_out) {
  if (!h || !sm_cycles_out || !ns_out || !h->time_kernel || !h->err_dev_has_clock) return SGEMM_CUBE_INVALID_ARG;
  DeviceGuard g(h->device);
  if (!g.ok) return SGEMM_CUBE_CUDA_ERROR;
  unsigned long long v[2] = {0, 0};
  if (cudaDeviceSynchronize() != cudaSuccess ||
      cudaMemcpy(v, h->err_dev + 16, sizeof(v), cudaMemcpyDeviceToHost) != cudaSuccess) {
    cudaGetLastError();
    return SGEMM_CUBE_CUDA_ERROR;
  }
  *sm_cycles_out = v[0];
  *ns_out = v[1];
  return SGEMM_CUBE_OK;
}

int sgemm_cube_debug_inject_error(sgemm_cube_handle h, uint32_t code) {
  if (!h) return SGEMM_CUBE_INVALID_ARG;
  DeviceGuard g(h->device);
  if (!g.ok) return SGEMM_CUBE_CUDA_ERROR;
  if (cudaDeviceSynchronize() != cudaSuccess ||
      cudaMemcpy(h->err_dev, &code, sizeof(code), cudaMemcpyHostToDevice) != cudaSuccess) {
    cudaGetLastError();
    return SGEMM_CUBE_CUDA_ERROR;
  }
  return SGEMM_CUBE_OK;
}

int sgemm_cube_debug_wait_timeout(sgemm_cube_handle h, int64_t limit_clocks, void* stream) {
  if (!h || limit_clocks < 1 || limit_clocks > 100000000) return SGEMM_CUBE_INVALID_ARG;
  DeviceGuard g(h->device);
  if (!g.ok) return SGEMM_CUBE_CUDA_ERROR;
  sgc::wait_timeout_probe_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(h->err_dev,
                                                                                (long long)limit_clocks);
  h->launches++;
  return cudaGetLastError() == cudaSuccess ? SGEMM_CUBE_OK : SGEMM_CUBE_CUDA_ERROR;
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------
// sgemm_cube_unfused_static: the unfused path for callers that must not allocate.
//
// Its scratch (the FP16 words of A and B and the two FP32 partial-result matrices) is a fixed
// array in the library's device image instead of a cudaMalloc'd workspace.  In host code the
// array's name is only a stand-in: the device address is looked up once per device with
// cudaGetSymbolAddress while that device is current, and that pointer is what the kernels get.
namespace {

static __device__ __align__(256) unsigned char g_static_scratch[SGEMM_CUBE_STATIC_SCRATCH_BYTES];
static __device__ unsigned int g_static_err;

constexpr int kMaxStaticDevices = 64;

struct StaticDeviceState {
  bool ready = false;
  unsigned char* scratch = nullptr;   // device address of g_static_scratch on this device
  sgemm_cube_ctx ctx;                 // host-side launch state; owns no device memory
};

StaticDeviceState g_static_state[kMaxStaticDevices];
std::mutex g_static_mutex;

// First call on a device: resolve the device addresses of the scratch array and of the error
// word, fetch the descriptor encoder and raise the kernels' shared-memory limit.  Allocates nothing.
int static_setup(int device, StaticDeviceState** out) {
  if (device < 0 || device >= kMaxStaticDevices) return SGEMM_CUBE_INVALID_ARG;
  std::lock_guard<std::mutex> lock(g_static_mutex);
  StaticDeviceState& s = g_static_state[device];
  if (!s.ready) {
    int major = 0, sms = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) {
      cudaGetLastError();
      return SGEMM_CUBE_CUDA_ERROR;
    }
    if (major != 10) return SGEMM_CUBE_UNSUPPORTED_ARCH;
    void* scratch = nullptr;
    void* err = nullptr;
    if (cudaGetSymbolAddress(&scratch, g_static_scratch) != cudaSuccess ||
        cudaGetSymbolAddress(&err, g_static_err) != cudaSuccess || !scratch || !err) {
      cudaGetLastError();
      return SGEMM_CUBE_CUDA_ERROR;
    }
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess || !fn) {
      cudaGetLastError();
      return SGEMM_CUBE_CUDA_ERROR;
    }
    s.scratch = static_cast<unsigned char*>(scratch);
    s.ctx.device = device;
    s.ctx.sm_count = sms;
    s.ctx.err_dev = static_cast<unsigned int*>(err);
    s.ctx.encode = reinterpret_cast<EncodeTiledFn>(fn);
    int rc = set_kernel_attrs(&s.ctx);
    if (rc) return rc;
    s.ready = true;
  }
  *out = &s;
  return SGEMM_CUBE_OK;
}

}  // namespace

extern "C" int sgemm_cube_unfused_static(int M, int N, int K, const float* A, int64_t lda,
                                         const float* B, int64_t ldb, float* C, int64_t ldc,
                                         int scale_exp, void* stream) {
  int rc = check_gemm_dims(M, N, K, lda, ldb, ldc);
  if (rc) return rc;
  if (missing_operand(M, N, K, A, A, B, B, C)) return SGEMM_CUBE_INVALID_ARG;
  if (scale_exp < 0 || scale_exp > 24) return SGEMM_CUBE_INVALID_ARG;
  if (empty_problem(M, N, K, C, ldc, static_cast<cudaStream_t>(stream), false, false, &rc)) return rc;
  // Same layout as the workspace of sgemm_cube_unfused, carved out of the fixed array.
  const size_t ldA16 = round_up((size_t)K, 8), ldB16 = round_up((size_t)N, 8);
  const size_t ldD = round_up((size_t)N, 4);
  const size_t szA = round_up((size_t)M * ldA16 * 2, 256), szB = round_up((size_t)K * ldB16 * 2, 256);
  const size_t szD = round_up((size_t)M * ldD * 4, 256);
  if (2 * szA + 2 * szB + 2 * szD > (size_t)SGEMM_CUBE_STATIC_SCRATCH_BYTES) return SGEMM_CUBE_TOO_LARGE;
  int device = -1;
  if (cudaGetDevice(&device) != cudaSuccess) { cudaGetLastError(); return SGEMM_CUBE_CUDA_ERROR; }
  StaticDeviceState* s = nullptr;
  rc = static_setup(device, &s);
  if (rc) return rc;
  sgemm_cube_ctx* h = &s->ctx;
  // The per-device launch state is shared by every caller of this entry point: host threads
  // enqueue one at a time (the GPU work itself is ordered by the caller's streams).
  std::lock_guard<std::mutex> lock(g_static_mutex);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  unsigned char* w = s->scratch;
  uint16_t* Ahi = reinterpret_cast<uint16_t*>(w);
  uint16_t* Alo = reinterpret_cast<uint16_t*>(w + szA);
  uint16_t* Bhi = reinterpret_cast<uint16_t*>(w + 2 * szA);
  uint16_t* Blo = reinterpret_cast<uint16_t*>(w + 2 * szA + szB);
  float* Dhh = reinterpret_cast<float*>(w + 2 * szA + 2 * szB);
  float* Dx = reinterpret_cast<float*>(w + 2 * szA + 2 * szB + szD);
  const float inv = ldexpf(1.0f, -scale_exp);
  const int kb = h->kblock_termwise;
  // Every region used below is fully overwritten before it is read (D_x by the second pass before
  // the third adds to it), so nothing left by an earlier call can leak into this one.
  if ((rc = launch_split(h, M, K, A, lda, Ahi, Alo, (int64_t)ldA16, scale_exp, st))) return rc;
  if ((rc = launch_split(h, K, N, B, ldb, Bhi, Blo, (int64_t)ldB16, scale_exp, st))) return rc;
  if ((rc = launch_tc_gemm<1>(h, M, N, K, Ahi, nullptr, ldA16, Bhi, nullptr, ldB16, Dhh, ldD, 0, 0, kb, 1.f, st))) return rc;
  if ((rc = launch_tc_gemm<1>(h, M, N, K, Alo, nullptr, ldA16, Bhi, nullptr, ldB16, Dx, ldD, 0, 0, kb, 1.f, st))) return rc;
  if ((rc = launch_tc_gemm<1>(h, M, N, K, Ahi, nullptr, ldA16, Blo, nullptr, ldB16, Dx, ldD, 1, 0, kb, 1.f, st))) return rc;
  const long long total = (long long)M * N;
  long long blocks = (total + 255) / 256;
  const long long cap = (long long)h->sm_count * 16;
  if (blocks > cap) blocks = cap;
  sgc::combine_kernel<<<(unsigned)blocks, 256, 0, st>>>(M, N, Dhh, Dx, (long long)ldD, C, ldc, inv);
  return cudaGetLastError() == cudaSuccess ? SGEMM_CUBE_OK : SGEMM_CUBE_CUDA_ERROR;
}

#ifdef SGC_ROLE_TIMING
// Debug builds only: read and clear the role-timing table of tc_gemm_kernel.
extern "C" int sgemm_cube_debug_role_timing(unsigned long long* out16) {
  if (cudaDeviceSynchronize() != cudaSuccess) return SGEMM_CUBE_CUDA_ERROR;
  if (cudaMemcpyFromSymbol(out16, sgc::g_role_timing, 16 * sizeof(unsigned long long)) != cudaSuccess)
    return SGEMM_CUBE_CUDA_ERROR;
  unsigned long long z[16] = {0};
  cudaMemcpyToSymbol(sgc::g_role_timing, z, sizeof(z));
  return SGEMM_CUBE_OK;
}
#endif
