// kdkl_logz_noalloc: the per-token log-normaliser log Z = logsumexp_v(h W^T / tau) computed with
// no device allocation anywhere - not by the caller, not by this library.
//
// Who needs this: code that runs inside someone else's process and may not call cudaMalloc. A
// plugin loaded by an inference server whose memory pool already owns the whole device gets an
// out-of-memory error from cudaMalloc however small the request; a callback on a latency-critical
// path must not enter the driver's allocator, which can serialise with other work on the device.
// Such callers can still pass their inputs and an output buffer, but have nowhere to put the
// per-vocab-tile partial results the tensor-core sweep produces. Here that scratch lives in a
// fixed array compiled into the library.
//
// The scratch is a file-scope __device__ array (about 8 MiB, see kScratchBytes): every GPU on
// which this library is loaded holds that much until the process exits. In host code the array's
// name is only a handle; the device address is obtained once per device with
// cudaGetSymbolAddress() and that pointer is what the kernels receive.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdio.h>
#include <string.h>

#include <mutex>

#include "../../include/kdkl.h"
#include "gemm_tcgen05.cuh"

namespace {

using namespace kdkl;

constexpr long long kMaxV = 262144;                  // largest vocabulary accepted
constexpr int kPassRows = 1024;                      // tokens per internal pass
constexpr long long kMaxTiles = kMaxV / BN;          // vocab tiles of the GEMM at kMaxV
constexpr size_t kOffStatus = 0;                     // int[2]: {code, site} of an expired wait
constexpr size_t kOffNvalid = 256;                   // int[kPassRows], all zero: no teacher entries
constexpr size_t kOffPartM = kOffNvalid + sizeof(int) * kPassRows;
constexpr size_t kOffPartS = kOffPartM + sizeof(float) * kMaxTiles * kPassRows;
constexpr size_t kScratchBytes = kOffPartS + sizeof(float) * kMaxTiles * kPassRows;   // 8 MiB + 4.25 KiB
constexpr size_t kClearBytes = kOffPartM;            // what must start at zero on every call

static __device__ __align__(256) unsigned char g_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
struct PerDevice { bool ready = false; unsigned char* scratch = nullptr; int sm_count = 0; };
static PerDevice g_dev[kMaxDevices];
static std::mutex g_mu;
static thread_local char g_text[256] = "";

// Merge the (max, sum) partials of one pass into log Z; a recorded wait expiry poisons the output
// with NaN instead of letting a wrong value through.
__global__ void __launch_bounds__(256)
logz_combine_kernel(const float* __restrict__ part_m, const float* __restrict__ part_s, int n_tiles, int rows,
                    const int* __restrict__ status, float* __restrict__ logz_out) {
  __shared__ float sm_m[8][32], sm_s[8][32];
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const int r = blockIdx.x * 32 + tx;
  float m = -INFINITY, s = 0.f;
  if (r < rows) {
    for (int nt = ty; nt < n_tiles; nt += 8) {
      const float pm = part_m[(long long)nt * kPassRows + r];
      const float ps = part_s[(long long)nt * kPassRows + r];
      const float mn = fmaxf(m, pm);
      s = s * exp2f(m - mn) + ps * exp2f(pm - mn);
      m = mn;
    }
  }
  sm_m[ty][tx] = m; sm_s[ty][tx] = s;
  __syncthreads();
  if (ty == 0 && r < rows) {
    float mm = sm_m[0][tx], ss = sm_s[0][tx];
    for (int i = 1; i < 8; ++i) {
      const float pm = sm_m[i][tx], ps = sm_s[i][tx];
      if (pm == -INFINITY) continue;
      const float mn = fmaxf(mm, pm);
      ss = ss * exp2f(mm - mn) + ps * exp2f(pm - mn);
      mm = mn;
    }
    const float lz = (mm + log2f(ss)) * 0.6931471805599453f;
    logz_out[r] = (*status == 0) ? lz : __int_as_float(0x7fc00000);
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

int encode_bf16_2d(CUtensorMap* m, const void* base, uint64_t inner, uint64_t outer, uint32_t box_outer) {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      return KDKL_ERR_CUDA;
    fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  cuuint64_t dims[2] = {inner, outer};
  cuuint64_t strides[1] = {inner * 2};
  cuuint32_t box[2] = {BK, box_outer};
  cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS ? KDKL_OK : KDKL_ERR_CUDA;
}

// Once per device, with that device current: resolve the scratch array's device address and raise
// the GEMM kernel's shared-memory limit. Neither call allocates device memory.
int setup_device(int dev, PerDevice** out) {
  if (dev < 0 || dev >= kMaxDevices) { snprintf(g_text, sizeof(g_text), "device ordinal %d not supported", dev); return KDKL_ERR_ARG; }
  std::lock_guard<std::mutex> lock(g_mu);
  PerDevice& d = g_dev[dev];
  if (!d.ready) {
    int major = 0;
    cudaError_t e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e == cudaSuccess && major != 10) return KDKL_ERR_ARCH;
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, dev);
    void* ptr = nullptr;
    if (e == cudaSuccess) e = cudaGetSymbolAddress(&ptr, g_scratch);
    if (e == cudaSuccess)
      e = cudaFuncSetAttribute(gemm_tcgen05_kernel<EPI_LSE, false, false, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               GemmCfg<1>::SMEM_BYTES);
    if (e != cudaSuccess) {
      snprintf(g_text, sizeof(g_text), "set-up on device %d failed: %s", dev, cudaGetErrorString(e));
      return KDKL_ERR_CUDA;
    }
    d.scratch = static_cast<unsigned char*>(ptr);
    d.ready = true;
  }
  *out = &d;
  return KDKL_OK;
}

}  // namespace

extern "C" int kdkl_logz_noalloc(const void* hidden_bf16, const void* weight_bf16, int64_t T, int64_t H, int64_t V,
                                 float temperature, float* logz_out, void* cuda_stream) {
  if (!hidden_bf16 || !weight_bf16 || !logz_out) return KDKL_ERR_NULL;
  if (T < 1 || H < 1 || V < 1 || (H % 8) != 0 || T >= (1ll << 31)) return KDKL_ERR_SHAPE;
  if (V > kMaxV) {
    snprintf(g_text, sizeof(g_text), "V = %lld exceeds the built-in scratch limit of %lld", (long long)V, kMaxV);
    fprintf(stderr, "kdkl_logz_noalloc: %s\n", g_text);
    return KDKL_ERR_WORKSPACE;
  }
  if (!(temperature > 0.f)) return KDKL_ERR_ARG;
  if (((uintptr_t)hidden_bf16 & 15) || ((uintptr_t)weight_bf16 & 15)) return KDKL_ERR_ALIGN;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return KDKL_ERR_CUDA;
  PerDevice* pd = nullptr;
  int rc = setup_device(dev, &pd);
  if (rc) return rc;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  unsigned char* sc = pd->scratch;                       // device address, not the host-side symbol
  // the array keeps the previous call's contents: the status words and the (empty) teacher counts
  // must start at zero; the partials are fully rewritten by every pass before they are read
  if (cudaMemsetAsync(sc, 0, kClearBytes, st) != cudaSuccess) return KDKL_ERR_CUDA;

  CUtensorMap tmW, tmA;
  if ((rc = encode_bf16_2d(&tmW, weight_bf16, (uint64_t)H, (uint64_t)V, BN))) return rc;
  const int n_tiles = (int)((V + BN - 1) / BN);
  for (int64_t s0 = 0; s0 < T; s0 += kPassRows) {
    const int rows = (int)((T - s0 < kPassRows) ? (T - s0) : kPassRows);
    const __nv_bfloat16* hA = reinterpret_cast<const __nv_bfloat16*>(hidden_bf16) + s0 * H;
    if ((rc = encode_bf16_2d(&tmA, hA, (uint64_t)H, (uint64_t)rows, BM))) return rc;
    GemmParams p;
    memset(&p, 0, sizeof(p));
    p.M = rows; p.N = (int)V; p.K = (int)H;
    p.m_tiles = (rows + BM - 1) / BM; p.n_tiles = n_tiles; p.m_inner = 1; p.k_splits = 1;
    p.status = reinterpret_cast<int*>(sc + kOffStatus);
    p.scale_log2 = 1.4426950408889634f / temperature;
    p.Ktop = 1;
    p.nvalid = reinterpret_cast<const int*>(sc + kOffNvalid);      // zeros: nothing to gather
    p.idx_sorted = reinterpret_cast<const int*>(sc + kOffNvalid);  // never dereferenced with zero counts
    p.part_m = reinterpret_cast<float*>(sc + kOffPartM);
    p.part_s = reinterpret_cast<float*>(sc + kOffPartS);
    p.part_stride = kPassRows;
    const int tiles = p.m_tiles * p.n_tiles;
    const int grid = tiles < pd->sm_count ? tiles : pd->sm_count;
    gemm_tcgen05_kernel<EPI_LSE, false, false, 1><<<grid, GEMM_THREADS, GemmCfg<1>::SMEM_BYTES, st>>>(tmA, tmW, tmA /*no output map*/, p);
    logz_combine_kernel<<<(rows + 31) / 32, 256, 0, st>>>(p.part_m, p.part_s, n_tiles, rows, p.status, logz_out + s0);
    if (cudaGetLastError() != cudaSuccess) return KDKL_ERR_CUDA;
  }
  return KDKL_OK;
}
