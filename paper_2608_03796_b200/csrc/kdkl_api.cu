// Host side of the C ABI: argument checks, workspace carving, tensor-map encoding and the
// per-chunk launch schedule of Algorithm 1. Enqueue-only: nothing here synchronises except
// kdkl_status() and the host-buffer entry point, which say so.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <vector>

#include "../../include/kdkl.h"
#include "aux_kernels.cuh"
#include "feature_kernels.cuh"
#include "gemm_tcgen05.cuh"

namespace kdkl {

static thread_local char g_err[512] = "";
static thread_local int64_t g_launches = 0;

static int cuda_fail(const char* what, cudaError_t e) {
  snprintf(g_err, sizeof(g_err), "%s: %s", what, cudaGetErrorString(e));
  return KDKL_ERR_CUDA;
}
#define KDKL_CUDA(call)                                   \
  do {                                                    \
    cudaError_t e__ = (call);                             \
    if (e__ != cudaSuccess) return cuda_fail(#call, e__); \
  } while (0)
#define KDKL_LAUNCHED(name)                               \
  do {                                                    \
    cudaError_t e__ = cudaGetLastError();                 \
    if (e__ != cudaSuccess) return cuda_fail(name, e__);  \
    ++g_launches;                                         \
  } while (0)

// ------------------------------------------------------------------ per-stage event timing
// Off unless kdkl_profile_stages() is running on this thread. When on, every launch site first
// records an event tagged with its stage; the time between consecutive events is charged to the
// earlier one's stage.
enum { ST_PREP = 0, ST_F1, ST_COMBINE, ST_REDUCE, ST_COEF, ST_B1, ST_B2, ST_B3, ST_END, ST_COUNT = ST_END };
struct StageTimer {
  bool on = false;
  std::vector<cudaEvent_t> ev;
  std::vector<int> stage;
};
static thread_local StageTimer g_timer;
static void stage_mark(int stage, cudaStream_t st) {
  if (!g_timer.on) return;
  cudaEvent_t e;
  if (cudaEventCreate(&e) != cudaSuccess) return;
  cudaEventRecord(e, st);
  g_timer.ev.push_back(e);
  g_timer.stage.push_back(stage);
}

static void stage_timer_start() {
  g_timer.on = true;
  g_timer.ev.clear();
  g_timer.stage.clear();
}
// Closes the event list, waits for the stream and adds the time between consecutive events to the earlier one's stage.
static int stage_timer_finish(int rc, cudaStream_t st, float* stage_ms, int32_t* stage_launches) {
  stage_mark(ST_END, st);
  g_timer.on = false;
  cudaError_t e = cudaStreamSynchronize(st);
  for (int i = 0; i < ST_COUNT; ++i) { stage_ms[i] = 0.f; stage_launches[i] = 0; }
  for (size_t i = 0; e == cudaSuccess && i + 1 < g_timer.ev.size(); ++i) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, g_timer.ev[i], g_timer.ev[i + 1]) == cudaSuccess) {
      stage_ms[g_timer.stage[i]] += ms;
      stage_launches[g_timer.stage[i]] += 1;
    }
  }
  for (cudaEvent_t ev : g_timer.ev) cudaEventDestroy(ev);
  g_timer.ev.clear();
  g_timer.stage.clear();
  if (e != cudaSuccess) return cuda_fail("cudaStreamSynchronize", e);
  return rc;
}

// ------------------------------------------------------------------ host-buffer pipeline
// Set (per thread) only while kdkl_forward_backward_host runs its two calls: the hidden rows of chunk i arrive on a
// copy stream (the forward sweep of chunk i waits for in_ready[i]), and chunk i's dhidden rows leave on it as soon
// as they are final (dh_ready[i] is recorded after the chunk's dH kernels). Everything else stays on the caller's
// stream. Events and the copy stream are host-side objects: no device memory is allocated.
struct HostPipe {
  cudaStream_t side = nullptr;
  std::vector<cudaEvent_t> in_ready, dh_ready;
};
static thread_local HostPipe* g_pipe = nullptr;

// ------------------------------------------------------------------ tensor maps
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn) return fn;
  void* p = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess)
    return nullptr;
  fn = reinterpret_cast<EncodeTiledFn>(p);
  return fn;
}

// 2-D bf16 tensor, `inner` contiguous elements per row, `outer` rows of `pitch_bytes`;
// boxes of box_inner x box_outer written to shared memory with the 128-byte swizzle;
// out-of-bounds elements read as zero.
static int make_tmap(CUtensorMap* m, CUtensorMapDataType dtype, const void* base, uint64_t inner, uint64_t outer,
                     uint64_t pitch_bytes, uint32_t box_inner, uint32_t box_outer) {
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) { snprintf(g_err, sizeof(g_err), "cuTensorMapEncodeTiled entry point not found"); return KDKL_ERR_CUDA; }
  cuuint64_t dims[2] = {inner, outer};
  cuuint64_t strides[1] = {pitch_bytes};
  cuuint32_t box[2] = {box_inner, box_outer};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(m, dtype, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    snprintf(g_err, sizeof(g_err), "cuTensorMapEncodeTiled failed (%d): inner=%llu outer=%llu pitch=%llu box=%ux%u",
             (int)r, (unsigned long long)inner, (unsigned long long)outer, (unsigned long long)pitch_bytes, box_inner,
             box_outer);
    return KDKL_ERR_CUDA;
  }
  return KDKL_OK;
}

static int make_tmap_bf16(CUtensorMap* m, const void* base, uint64_t inner, uint64_t outer, uint64_t pitch_bytes,
                          uint32_t box_inner, uint32_t box_outer) {
  return make_tmap(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, base, inner, outer, pitch_bytes, box_inner, box_outer);
}
// Output maps: the epilogue stores boxes of 32 rows x 128 bytes (32 fp32 or 64 bf16 columns).
static int make_tmap_out_f32(CUtensorMap* m, void* base, uint64_t cols, uint64_t rows, uint64_t ld_elems) {
  return make_tmap(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, base, cols, rows, ld_elems * 4, 32, 32);
}
static int make_tmap_out_bf16(CUtensorMap* m, void* base, uint64_t cols, uint64_t rows, uint64_t ld_elems) {
  return make_tmap(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, base, cols, rows, ld_elems * 2, 64, 32);
}

// ------------------------------------------------------------------ device / launch helpers
// All GEMMs of the loss run as CTA pairs (256 x 256 tile per pair, see GemmCfg).
constexpr int kNCTA = 2;
constexpr int kTileM = GemmCfg<kNCTA>::TILE_M;
constexpr int kBRows = GemmCfg<kNCTA>::B_ROWS;             // rows of a K-major B box (also per half of a WIDE tile)
constexpr int kWideN = GemmCfg<kNCTA, true>::TILE_N;
static_assert(GemmCfg<kNCTA, true>::B_ROWS / 2 == kBRows, "a WIDE tile's halves take the narrow tile's B boxes");
// The two output GEMMs (N = H) use WIDE tiles when rounding H up to whole 512-column tiles wastes at most a
// tenth of the tensor work (H = 4096, 3072, 1024, 1000 ...); narrow 256-column tiles otherwise.
// Row tiles per raster group of the two vocabulary sweeps (forward, recompute): as many as keep the group's hidden
// rows within 32 MiB, i.e. resident in either half of the L2 while the weight streams past (4096 tokens at H = 4096).
static int m_group_for(long long H) {
  const long long rows = (32ll << 20) / (H * 2);
  const long long g = rows / kTileM;
  return (int)(g < 1 ? 1 : g);
}
static bool use_wide(long long N) { return ((N + kWideN - 1) / kWideN) * kWideN * 10 <= N * 11; }
static long long n_tiles_for(long long N, bool wide) { return wide ? (N + kWideN - 1) / kWideN : (N + BN - 1) / BN; }
// What the library has learnt about each device, asked once per device and process (a benign race: two
// threads asking at the same time store the same values).
constexpr int kMaxDevices = 64;
struct DeviceInfo { int dev; int sm_count; int cc_major; };
struct DeviceCache { bool known; int sm_count; int cc_major; };
static DeviceCache g_devices[kMaxDevices];
static int device_info(DeviceInfo* di) {
  int dev = 0;
  KDKL_CUDA(cudaGetDevice(&dev));
  di->dev = dev;
  if (dev >= 0 && dev < kMaxDevices && g_devices[dev].known) {
    di->sm_count = g_devices[dev].sm_count; di->cc_major = g_devices[dev].cc_major;
    return KDKL_OK;
  }
  KDKL_CUDA(cudaDeviceGetAttribute(&di->sm_count, cudaDevAttrMultiProcessorCount, dev));
  KDKL_CUDA(cudaDeviceGetAttribute(&di->cc_major, cudaDevAttrComputeCapabilityMajor, dev));
  if (dev >= 0 && dev < kMaxDevices) {
    g_devices[dev].sm_count = di->sm_count; g_devices[dev].cc_major = di->cc_major; g_devices[dev].known = true;
  }
  return KDKL_OK;
}
// SM count of the current device for sizing decisions that are also taken where there may be no device
// (kdkl_workspace_bytes on a build machine): a B200's 148 then.
static int sm_count_or_default() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return 148; }
  if (dev >= 0 && dev < kMaxDevices && g_devices[dev].known) return g_devices[dev].sm_count;
  DeviceInfo di;
  if (device_info(&di) != KDKL_OK || di.sm_count < 2) { cudaGetLastError(); return 148; }
  return di.sm_count;
}

template <int EPI, bool A_MN, bool B_MN, bool WIDE = false>
static int launch_gemm(const CUtensorMap& ta, const CUtensorMap& tb, const CUtensorMap& tc, const GemmParams& p,
                       const DeviceInfo& di, cudaStream_t st) {
  auto kern = gemm_tcgen05_kernel<EPI, A_MN, B_MN, kNCTA, WIDE>;
  constexpr int smem = GemmCfg<kNCTA, WIDE>::SMEM_BYTES;
  static_assert(smem <= 227 * 1024, "shared memory per CTA");
  // The shared-memory limit belongs to the current device's copy of this instantiation: set once per device
  // (a process may drive several), not per launch.
  static bool attr_set[kMaxDevices];
  const int sm_count = di.sm_count;
  if (di.dev < 0 || di.dev >= kMaxDevices || !attr_set[di.dev]) {
    KDKL_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    if (di.dev >= 0 && di.dev < kMaxDevices) attr_set[di.dev] = true;
  }
  // persistent: one worker (a CTA, or a pair of CTAs on neighbouring SMs) per SM (pair), each walking
  // the work units with a stride of the worker count
  const int units = p.m_tiles * p.n_tiles * p.k_splits;
  const int max_workers = sm_count / kNCTA;
  const int workers = units < max_workers ? units : max_workers;
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3((unsigned)(workers * kNCTA), 1, 1);
  cfg.blockDim = dim3(GEMM_THREADS, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = kNCTA;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t e = cudaLaunchKernelEx(&cfg, kern, ta, tb, tc, p);
  if (e != cudaSuccess) return cuda_fail("gemm_tcgen05_kernel launch", e);
  KDKL_LAUNCHED("gemm_tcgen05_kernel");
  return KDKL_OK;
}

// ------------------------------------------------------------------ workspace
static inline size_t up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// How many work units to cut each output tile's contraction into so that the units fill whole
// waves of SMs: the smallest count (<= 4, each unit keeping >= 32 k-blocks) that reaches 95 %
// wave efficiency, else the most efficient one, for the device's count of workers (SMs / CTAs per tile).
static int choose_k_splits(long long tiles, long long kblocks, int sm_count) {
  const long long sms = (sm_count < kNCTA ? kNCTA : sm_count) / kNCTA;
  int best = 1;
  double best_eff = 0.0;
  for (int sp = 1; sp <= 4; ++sp) {
    if (sp > 1 && kblocks / sp < 32) break;
    const long long units = tiles * sp;
    const double eff = (double)units / (double)(((units + sms - 1) / sms) * sms);
    if (eff > best_eff + 1e-9) { best_eff = eff; best = sp; }
    if (eff >= 0.95) break;
  }
  return best;
}

struct WsLayout {
  long long C, Cpad, Vpad, n_tiles_v;
  int dh_splits;             // split-K factor of the dH GEMM at full chunks
  int dw_group;              // chunks whose G is kept so that one dW pass contracts over all of them (1 or 2)
  long long g_rows;          // rows of the G buffer
  size_t hdr, idx_sorted, p_sorted, perm, zg, colread, nvalid, M, Hent, lz2, logZ, loss_tok, coefA, coefB;
  size_t part_m, part_s, G, dh_part, live, rs, hs, total;
  static constexpr int kMaxSlabs = 24;
  int n_slabs;
  size_t slab_off[kMaxSlabs], slab_len[kMaxSlabs];   // every slab in layout order (for kdkl_workspace_layout)
  long long tiles_per_chunk, n_live;   // live-row-tile flags: one per kTileM rows of every chunk
};

// Debug aid: kdkl_debug_guard_bytes(n) puts n untouched bytes after every workspace slab (and makes the
// workspace that much larger), so that a test can pre-fill the workspace, run, and see whether any kernel
// wrote past the end of a slab (kdkl_workspace_layout gives the slab table). 0: the compact layout.
static size_t g_guard_bytes = 0;
static size_t ws_guard_bytes() { return g_guard_bytes; }

// chunks_per_pass: the caller's kdkl_options.dw_chunks_per_pass (0 = default).
static WsLayout ws_layout(long long T, long long H, long long V, int K, long long chunk, int chunks_per_pass) {
  WsLayout L;
  L.C = chunk <= 0 ? 4096 : chunk;
  if (L.C > T) L.C = T;
  L.Cpad = (long long)up((size_t)L.C, 128);
  L.Vpad = (long long)up((size_t)V, 64);
  L.n_tiles_v = (V + BN - 1) / BN;
  size_t o = 0;
  const size_t guard = ws_guard_bytes();
  L.n_slabs = 0;
  auto take = [&](size_t bytes) {
    size_t at = o;
    if (L.n_slabs < WsLayout::kMaxSlabs) { L.slab_off[L.n_slabs] = at; L.slab_len[L.n_slabs] = bytes; ++L.n_slabs; }
    o = up(o + bytes, 256) + guard;
    return at;
  };
  L.hdr = take(256);
  L.idx_sorted = take((size_t)T * K * 4);
  L.p_sorted = take((size_t)T * K * 4);
  L.perm = take((size_t)T * K * 2);
  L.zg = take((size_t)T * K * 4);
  L.colread = take((size_t)T * K * 4);
  L.nvalid = take((size_t)T * 4);
  L.M = take((size_t)T * 4);
  L.Hent = take((size_t)T * 4);
  L.lz2 = take((size_t)T * 4);
  L.logZ = take((size_t)T * 4);
  L.loss_tok = take((size_t)T * 4);
  L.coefA = take((size_t)T * 4);
  L.coefB = take((size_t)T * 4);
  L.part_m = take((size_t)L.n_tiles_v * L.Cpad * 4);
  L.part_s = take((size_t)L.n_tiles_v * L.Cpad * 4);
  // dW += G^T h is read-modify-write of the whole fp32 dW per pass, and every byte a GEMM stores costs its SM
  // load bandwidth: with the G of two consecutive chunks kept, one pass contracts over both and the dW traffic
  // halves (one more [chunk, V] bf16 buffer). Up to 8192 tokens per pass (the kernel's k-block skip list).
  L.dw_group = (T > L.C && 2 * L.C <= 8192 && chunks_per_pass != 1) ? 2 : 1;
  const long long g_tokens = (long long)L.dw_group * L.C < T ? (long long)L.dw_group * L.C : T;
  L.g_rows = (long long)up((size_t)g_tokens, 128);
  L.G = take((size_t)L.g_rows * L.Vpad * 2);
  L.dh_splits = choose_k_splits(((L.C + kTileM - 1) / kTileM) * n_tiles_for(H, use_wide(H)), (V + BK - 1) / BK,
                                sm_count_or_default());
  L.dh_part = take((size_t)L.dh_splits * L.Cpad * H * 4);    // at least one slab: the single-pass step always fixes up
  L.rs = take((size_t)T * 4);                                 // single-pass step: the row scales ...
  L.hs = take((size_t)L.g_rows * H * 2);                      // ... and the scaled hidden rows of the group in flight
  L.tiles_per_chunk = (L.C + kTileM - 1) / kTileM;
  L.n_live = ((T + L.C - 1) / L.C) * L.tiles_per_chunk;
  L.live = take((size_t)L.n_live);
  L.total = o;
  return L;
}

// Options of this or of an earlier struct size (without grad_loss_device; without dw_chunks_per_pass; without
// denom_device; without stored_exponentials) are accepted.
static int copy_options(const kdkl_options* opt, kdkl_options* eff) {
  memset(eff, 0, sizeof(*eff));
  if (!opt) return KDKL_OK;
  constexpr int32_t kSize1 = (int32_t)offsetof(kdkl_options, stored_exponentials);
  constexpr int32_t kSize2 = (int32_t)(offsetof(kdkl_options, stored_exponentials) + sizeof(int32_t));
  constexpr int32_t kSize3 = (int32_t)(offsetof(kdkl_options, denom_device) + sizeof(const double*));
  constexpr int32_t kSize4 = (int32_t)offsetof(kdkl_options, grad_loss_device);
  if (opt->struct_size != (int32_t)sizeof(kdkl_options) && opt->struct_size != kSize1 && opt->struct_size != kSize2 &&
      opt->struct_size != kSize3 && opt->struct_size != kSize4)
    return KDKL_ERR_ARG;
  memcpy(eff, opt, (size_t)opt->struct_size);
  eff->struct_size = (int32_t)sizeof(kdkl_options);
  if (eff->stored_exponentials < 0 || eff->stored_exponentials > 1) return KDKL_ERR_ARG;
  return KDKL_OK;
}

// dw_chunks_per_pass of an option struct as the caller passed it (older, shorter structs do not have the field).
static int chunks_per_pass_of(const kdkl_options* opt) {
  if (opt == nullptr) return 0;
  if (opt->struct_size < (int32_t)(offsetof(kdkl_options, dw_chunks_per_pass) + sizeof(int32_t))) return 0;
  return opt->dw_chunks_per_pass;
}

static int check_common(const void* hidden, const void* weight, long long T, long long H, long long V, int K,
                        long long chunk, float tau, const kdkl_options* opt, const void* ws, size_t ws_bytes,
                        kdkl_options* eff, WsLayout* L, DeviceInfo* di) {
  if (!hidden || !weight || !ws) return KDKL_ERR_NULL;
  if (T < 1 || H < 1 || V < 1 || K < 1 || K > KDKL_MAX_K || (H % 8) != 0 || V >= (1ll << 31) || T >= (1ll << 31))
    return KDKL_ERR_SHAPE;
  if (!(tau > 0.f) || chunk < 0) return KDKL_ERR_ARG;
  if (copy_options(opt, eff) != KDKL_OK) return KDKL_ERR_ARG;
  if (eff->teacher_mode < 0 || eff->teacher_mode > 1) return KDKL_ERR_ARG;
  if (eff->teacher_mode == 1 && tau != 1.0f) return KDKL_ERR_ARG;
  if (eff->dhidden_dtype < 0 || eff->dhidden_dtype > 1) return KDKL_ERR_ARG;
  if (((uintptr_t)hidden & 15) || ((uintptr_t)weight & 15) || ((uintptr_t)ws & 15)) return KDKL_ERR_ALIGN;
  if (eff->dw_chunks_per_pass < 0 || eff->dw_chunks_per_pass > 2) return KDKL_ERR_ARG;
  *L = ws_layout(T, H, V, K, chunk, eff->dw_chunks_per_pass);
  if (eff->stored_exponentials && T > L->C) return KDKL_ERR_ARG;   // needs one chunk over all tokens
  if (ws_bytes < L->total) return KDKL_ERR_WORKSPACE;
  int rc = device_info(di);
  if (rc) return rc;
  if (di->cc_major != 10) return KDKL_ERR_ARCH;
  return KDKL_OK;
}

template <typename Tp>
static Tp* at(void* ws, size_t off) { return reinterpret_cast<Tp*>(reinterpret_cast<uint8_t*>(ws) + off); }

static int next_pow2(int x) { int p = 2; while (p < x) p <<= 1; return p; }

// Header reset, teacher preparation and (with a mask) the live-row-tile flags: the common start of every forward.
// Returns the flags (nullptr without a mask) through *live.
static int launch_prep(const WsLayout& L, const kdkl_options& o, void* ws, const int32_t* topk_idx,
                       const float* topk_val, const float* teacher_lse, const uint8_t* loss_mask, long long T,
                       long long V, long long v0, long long V_total, int K, float inv_tau, const uint8_t** live,
                       cudaStream_t st) {
  WsHeader* hdr = at<WsHeader>(ws, L.hdr);
  stage_mark(ST_PREP, st);
  header_reset_kernel<<<1, 32, 0, st>>>(hdr);
  KDKL_LAUNCHED("header_reset_kernel");
  const int Kpad = next_pow2(K);
  const size_t prep_smem = (size_t)PREP_WARPS * Kpad * (8 + 4);   // (key, slot) words and probabilities
  prep_kernel<<<(unsigned)((T + PREP_WARPS - 1) / PREP_WARPS), PREP_WARPS * 32, prep_smem, st>>>(
      topk_idx, topk_val, teacher_lse, loss_mask, T, (int)V, (int)v0, (int)V_total, K, Kpad, inv_tau, o.teacher_mode,
      at<int>(ws, L.idx_sorted), at<float>(ws, L.p_sorted), at<uint16_t>(ws, L.perm), at<int>(ws, L.nvalid),
      at<float>(ws, L.M), at<float>(ws, L.Hent), hdr);
  KDKL_LAUNCHED("prep_kernel");
  // with a mask: which row tiles hold at least one counted token (the others are skipped by every GEMM,
  // forward and backward; the flags stay in the workspace for kdkl_backward)
  *live = nullptr;
  if (loss_mask != nullptr) {
    tile_live_kernel<<<(unsigned)((L.n_live + 7) / 8), 256, 0, st>>>(loss_mask, T, L.C, kTileM, (int)L.tiles_per_chunk,
                                                                    L.n_live, at<uint8_t>(ws, L.live));
    KDKL_LAUNCHED("tile_live_kernel");
    *live = at<uint8_t>(ws, L.live);
  }
  return KDKL_OK;
}

// Parameters of the forward sweep of the chunk that starts at token s0 (EPI_LSE and its storing variants).
static void fill_forward_params(GemmParams* p, const WsLayout& L, void* ws, long long s0, long long rows, long long H,
                                long long V, int K, float inv_tau, const uint8_t* live_c) {
  WsHeader* hdr = at<WsHeader>(ws, L.hdr);
  memset(p, 0, sizeof(*p));
  p->M = (int)rows; p->N = (int)V; p->K = (int)H;
  p->m_tiles = (int)((rows + kTileM - 1) / kTileM); p->n_tiles = (int)L.n_tiles_v; p->m_inner = 1; p->k_splits = 1;
  p->m_group = m_group_for(H);
  p->status = &hdr->status; p->go = nullptr;
  p->scale_log2 = kLog2e * inv_tau; p->Ktop = K;
  p->idx_sorted = at<int>(ws, L.idx_sorted) + s0 * K;
  p->nvalid = at<int>(ws, L.nvalid) + s0;
  p->part_m = at<float>(ws, L.part_m); p->part_s = at<float>(ws, L.part_s); p->part_stride = L.Cpad;
  p->zg = at<float>(ws, L.zg) + s0 * K;
  p->colread = at<int>(ws, L.colread) + s0 * K;
  p->m_live = (live_c && p->m_tiles <= MAX_LIVE_M) ? live_c : nullptr;
}

// The two output GEMMs, shared by kdkl_backward and kdkl_forward_backward. G holds the dlogits (bf16, rows of
// Vpad elements) of the chunk, or of the group of chunks one dW pass contracts over.
//   dH[chunk] = G W        (M = rows, N = H, K = V; split-K with a fixed-order fix-up when the tiles are few)
//   dW (+)= G^T h[group]   (M = V, N = H, K = rows of the group; both operands MN-major: G is [t, v] with v
//                           contiguous, h is [t, h] with h contiguous)
struct ChunkOut {
  const __nv_bfloat16* G; const __nv_bfloat16* hA; void* dhidden; long long s0, rows, H, V;
  const WsLayout* L; const kdkl_options* o; WsHeader* hdr; void* ws; const int* go;
  const uint8_t* live_m;   // row-tile flags for the dH GEMM (nullptr: none)
  const uint8_t* live_c;   // row-tile flags of the dW contraction (nullptr: none)
  int accumulate_dw;
  const float* row_scale;  // single-pass step: per-row scale applied by the dH fix-up (nullptr: none)
};
static int launch_dhidden(const ChunkOut& c, const CUtensorMap& tmWmn, const DeviceInfo& di, cudaStream_t st) {
  const WsLayout& L = *c.L;
  const long long rows = c.rows, H = c.H, V = c.V, s0 = c.s0;
  int rc;
  CUtensorMap tmG, tmdH;
  stage_mark(ST_B2, st);
  if ((rc = make_tmap_bf16(&tmG, c.G, (uint64_t)V, (uint64_t)rows, (uint64_t)L.Vpad * 2, BK, BM))) return rc;
  const bool wide = use_wide(H);
  GemmParams p2;
  memset(&p2, 0, sizeof(p2));
  p2.M = (int)rows; p2.N = (int)H; p2.K = (int)V;
  p2.m_tiles = (int)((rows + kTileM - 1) / kTileM); p2.n_tiles = (int)n_tiles_for(H, wide); p2.m_inner = 0;
  p2.status = &c.hdr->status; p2.go = c.go;
  p2.m_live = c.live_m;              // dead row tiles: their dH rows are written as zeros
  // a short last chunk may want a different split; never more than the workspace was sized for
  int sp = choose_k_splits((long long)p2.m_tiles * p2.n_tiles, (V + BK - 1) / BK, di.sm_count);
  if (sp > L.dh_splits) sp = L.dh_splits;
  p2.k_splits = sp;
  __nv_bfloat16* dh16 = c.o->dhidden_dtype == 0 ? reinterpret_cast<__nv_bfloat16*>(c.dhidden) + s0 * H : nullptr;
  float* dh32 = c.o->dhidden_dtype == 1 ? reinterpret_cast<float*>(c.dhidden) + s0 * H : nullptr;
  if (sp > 1 || c.row_scale != nullptr) {
    // partial sums of each split go to fp32 slabs [split][Cpad, H]; a fixed-order fix-up adds them
    float* part = at<float>(c.ws, L.dh_part);
    p2.split_rows = (int)L.Cpad;
    if ((rc = make_tmap_out_f32(&tmdH, part, (uint64_t)H, (uint64_t)sp * L.Cpad, (uint64_t)H))) return rc;
    rc = wide ? launch_gemm<EPI_STORE_F32, false, true, true>(tmG, tmWmn, tmdH, p2, di, st)
              : launch_gemm<EPI_STORE_F32, false, true, false>(tmG, tmWmn, tmdH, p2, di, st);
    if (rc) return rc;
    const long long n4 = rows * H / 4;
    splitk_fixup_kernel<<<(unsigned)((n4 + 255) / 256), 256, 0, st>>>(part, (long long)L.Cpad * H, sp, n4, dh16, dh32,
                                                                     c.go, c.row_scale, (int)(H / 4));
    KDKL_LAUNCHED("splitk_fixup_kernel");
    return KDKL_OK;
  }
  if (dh16 != nullptr) {
    if ((rc = make_tmap_out_bf16(&tmdH, dh16, (uint64_t)H, (uint64_t)rows, (uint64_t)H))) return rc;
    return wide ? launch_gemm<EPI_STORE_BF16, false, true, true>(tmG, tmWmn, tmdH, p2, di, st)
                : launch_gemm<EPI_STORE_BF16, false, true, false>(tmG, tmWmn, tmdH, p2, di, st);
  }
  if ((rc = make_tmap_out_f32(&tmdH, dh32, (uint64_t)H, (uint64_t)rows, (uint64_t)H))) return rc;
  return wide ? launch_gemm<EPI_STORE_F32, false, true, true>(tmG, tmWmn, tmdH, p2, di, st)
              : launch_gemm<EPI_STORE_F32, false, true, false>(tmG, tmWmn, tmdH, p2, di, st);
}

// c.G / c.hA / c.rows: the whole group (rows = tokens of all its chunks, contiguous in G and in hidden).
static int launch_dweight(const ChunkOut& c, const CUtensorMap& tmdW, const DeviceInfo& di, cudaStream_t st) {
  const WsLayout& L = *c.L;
  const long long rows = c.rows, H = c.H, V = c.V;
  int rc;
  CUtensorMap tmGmn, tmhmn;
  if ((rc = make_tmap_bf16(&tmGmn, c.G, (uint64_t)V, (uint64_t)rows, (uint64_t)L.Vpad * 2, 64, BK))) return rc;
  if ((rc = make_tmap_bf16(&tmhmn, c.hA, (uint64_t)H, (uint64_t)rows, (uint64_t)H * 2, 64, BK))) return rc;
  const bool wide = use_wide(H);
  GemmParams p3;
  memset(&p3, 0, sizeof(p3));
  p3.M = (int)V; p3.N = (int)H; p3.K = (int)rows;
  p3.m_tiles = (int)((V + kTileM - 1) / kTileM); p3.n_tiles = (int)n_tiles_for(H, wide); p3.m_inner = 0; p3.k_splits = 1;
  p3.status = &c.hdr->status; p3.go = c.go;
  p3.accumulate = c.accumulate_dw;
  // dead row tiles of G are zeros: they are left out of the contraction over tokens (the kernel takes up to 32 flags)
  p3.k_live = (rows <= 32ll * kTileM && (rows + BK - 1) / BK <= MAX_LIVE_KB) ? c.live_c : nullptr;
  stage_mark(ST_B3, st);
  return wide ? launch_gemm<EPI_STORE_F32, true, true, true>(tmGmn, tmhmn, tmdW, p3, di, st)
              : launch_gemm<EPI_STORE_F32, true, true, false>(tmGmn, tmhmn, tmdW, p3, di, st);
}

// Where chunk ci's G lives inside the group buffer, and whether a dW pass is due after it.
struct GroupPos { long long j, row0; bool last; };
static GroupPos group_pos(const WsLayout& L, long long ci, long long s0, long long rows, long long T) {
  GroupPos g;
  g.j = ci % L.dw_group;
  g.row0 = g.j * L.C;
  g.last = g.j == L.dw_group - 1 || s0 + rows >= T;
  return g;
}
// The row-tile flags of a group are those of its chunks one after the other; they line up with the group's
// 256-row tiles only when every chunk but the last is a whole number of tiles.
static const uint8_t* group_flags(const WsLayout& L, const uint8_t* live, long long ci_first) {
  if (live == nullptr) return nullptr;
  if (L.dw_group > 1 && (L.C % kTileM) != 0) return nullptr;
  return live + ci_first * L.tiles_per_chunk;
}

}  // namespace kdkl

using namespace kdkl;

extern "C" {

const char* kdkl_last_error(void) { return g_err; }
int64_t kdkl_last_launch_count(void) { return g_launches; }

int kdkl_workspace_layout(int64_t T, int64_t H, int64_t V, int32_t K, int64_t chunk, const kdkl_options* opt,
                          int64_t* offsets, int64_t* lengths, int32_t capacity) {
  if (T < 1 || H < 1 || V < 1 || K < 1 || !offsets || !lengths) return 0;
  const WsLayout L = ws_layout(T, H, V, K, chunk, chunks_per_pass_of(opt));
  const int n = L.n_slabs < capacity ? L.n_slabs : capacity;
  for (int i = 0; i < n; ++i) { offsets[i] = (int64_t)L.slab_off[i]; lengths[i] = (int64_t)L.slab_len[i]; }
  return L.n_slabs;
}

size_t kdkl_workspace_bytes(int64_t T, int64_t H, int64_t V, int32_t K, int64_t chunk, const kdkl_options* opt) {
  if (T < 1 || H < 1 || V < 1 || K < 1) return 0;
  return ws_layout(T, H, V, K, chunk, chunks_per_pass_of(opt)).total;
}

int64_t kdkl_debug_guard_bytes(int64_t n) {
  const int64_t before = (int64_t)g_guard_bytes;
  if (n < 0) n = 0;
  if (n > (1ll << 20)) n = 1ll << 20;
  g_guard_bytes = up((size_t)n, 256);
  return before;
}

int kdkl_count_tokens(const uint8_t* loss_mask, int64_t T, double* count_out, void* cuda_stream) {
  g_launches = 0;
  if (!count_out) return KDKL_ERR_NULL;
  if (T < 1 || T >= (1ll << 31)) return KDKL_ERR_SHAPE;
  if ((uintptr_t)count_out & 7) return KDKL_ERR_ALIGN;
  count_tokens_kernel<<<1, 1024, 0, reinterpret_cast<cudaStream_t>(cuda_stream)>>>(loss_mask, T, 0.f, nullptr, nullptr,
                                                                                  count_out);
  KDKL_LAUNCHED("count_tokens_kernel");
  return KDKL_OK;
}

// Forward over the vocabulary rows [v0, v0 + V) this caller holds. Unsharded: v0 = 0, V_total = V,
// shard_stats = NULL and the loss is finished here. Sharded: the per-token local normaliser and cross
// term go to shard_stats [2, T] and kdkl_forward_finish completes the loss after the gather.
static int forward_impl(const void* hidden, const void* weight, const int32_t* topk_idx, const float* topk_val,
                        const float* teacher_lse, const uint8_t* loss_mask, int64_t T, int64_t H, int64_t V,
                        int64_t v0, int64_t V_total, int32_t K, int64_t chunk, float tau, const kdkl_options* opt,
                        void* ws, size_t ws_bytes, float* shard_stats, float* loss_out, float* loss_per_token,
                        float* gathered_logits, int32_t* gathered_idx, void* cuda_stream) {
  g_launches = 0;
  if (!topk_idx || !topk_val || (!loss_out && !shard_stats)) return KDKL_ERR_NULL;
  kdkl_options o;
  WsLayout L;
  DeviceInfo di;
  int rc = check_common(hidden, weight, T, H, V, K, chunk, tau, opt, ws, ws_bytes, &o, &L, &di);
  if (rc) return rc;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  WsHeader* hdr = at<WsHeader>(ws, L.hdr);
  const float inv_tau = 1.0f / tau;

  const uint8_t* live = nullptr;
  if ((rc = launch_prep(L, o, ws, topk_idx, topk_val, teacher_lse, loss_mask, T, V, v0, V_total, K, inv_tau, &live, st)))
    return rc;

  CUtensorMap tmW;
  if ((rc = make_tmap_bf16(&tmW, weight, (uint64_t)H, (uint64_t)V, (uint64_t)H * 2, BK, kBRows))) return rc;

  long long fci = 0;
  for (long long s0 = 0; s0 < T; s0 += L.C, ++fci) {
    const long long rows = (T - s0 < L.C) ? (T - s0) : L.C;
    CUtensorMap tmA;
    const __nv_bfloat16* hA = reinterpret_cast<const __nv_bfloat16*>(hidden) + s0 * H;
    if ((rc = make_tmap_bf16(&tmA, hA, (uint64_t)H, (uint64_t)rows, (uint64_t)H * 2, BK, BM))) return rc;
    GemmParams p;
    fill_forward_params(&p, L, ws, s0, rows, H, V, K, inv_tau, live ? live + fci * L.tiles_per_chunk : nullptr);
    if (g_pipe != nullptr && fci < (long long)g_pipe->in_ready.size())
      KDKL_CUDA(cudaStreamWaitEvent(st, g_pipe->in_ready[fci], 0));   // this chunk's hidden rows have arrived
    stage_mark(ST_F1, st);
    if (o.stored_exponentials) {
      // one chunk covers all tokens: leave the exponentials in the G buffer for a backward without recompute
      CUtensorMap tmE;
      if ((rc = make_tmap_out_bf16(&tmE, at<__nv_bfloat16>(ws, L.G), (uint64_t)V, (uint64_t)rows, (uint64_t)L.Vpad)))
        return rc;
      if ((rc = launch_gemm<EPI_LSE_E, false, false>(tmA, tmW, tmE, p, di, st))) return rc;
    } else {
      if ((rc = launch_gemm<EPI_LSE, false, false>(tmA, tmW, tmA /*no output map*/, p, di, st))) return rc;
    }
    stage_mark(ST_COMBINE, st);

    combine_kernel<<<(unsigned)((rows + 31) / 32), COMBINE_WARPS * 32, 0, st>>>(
        at<float>(ws, L.part_m), at<float>(ws, L.part_s), L.Cpad, (int)L.n_tiles_v, (int)rows, s0, K, inv_tau,
        at<int>(ws, L.nvalid), at<float>(ws, L.p_sorted), at<uint16_t>(ws, L.perm), at<float>(ws, L.zg),
        at<int>(ws, L.colread), at<float>(ws, L.M), at<float>(ws, L.Hent), loss_mask, at<float>(ws, L.lz2),
        at<float>(ws, L.logZ), at<float>(ws, L.loss_tok), loss_per_token, gathered_logits, gathered_idx, (int)v0,
        shard_stats, T, hdr, o.stored_exponentials);
    KDKL_LAUNCHED("combine_kernel");
  }
  if (shard_stats != nullptr) return KDKL_OK;   // the loss is completed by kdkl_forward_finish
  stage_mark(ST_REDUCE, st);
  loss_reduce_kernel<<<1, 1024, 0, st>>>(at<float>(ws, L.loss_tok), loss_mask, T, o.denom_override, o.denom_device, tau,
                                         H, V, K, L.C, o.stored_exponentials ? G_EXPONENTIALS : G_NONE, loss_out, hdr);
  KDKL_LAUNCHED("loss_reduce_kernel");
  return KDKL_OK;
}

int kdkl_forward(const void* hidden, const void* weight, const int32_t* topk_idx, const float* topk_val,
                 const float* teacher_lse, const uint8_t* loss_mask, int64_t T, int64_t H, int64_t V, int32_t K,
                 int64_t chunk, float tau, const kdkl_options* opt, void* ws, size_t ws_bytes, float* loss_out,
                 float* loss_per_token, float* gathered_logits, int32_t* gathered_idx, void* cuda_stream) {
  if (!loss_out) return KDKL_ERR_NULL;
  return forward_impl(hidden, weight, topk_idx, topk_val, teacher_lse, loss_mask, T, H, V, 0, V, K, chunk, tau, opt, ws,
                      ws_bytes, nullptr, loss_out, loss_per_token, gathered_logits, gathered_idx, cuda_stream);
}

int kdkl_forward_shard(const void* hidden, const void* weight_local, const int32_t* topk_idx, const float* topk_val,
                       const float* teacher_lse, const uint8_t* loss_mask, int64_t T, int64_t H, int64_t V_local,
                       int64_t vocab_offset, int64_t V_total, int32_t K, int64_t chunk, float tau,
                       const kdkl_options* opt, void* ws, size_t ws_bytes, float* shard_stats, float* gathered_logits,
                       int32_t* gathered_idx, void* cuda_stream) {
  if (!shard_stats) return KDKL_ERR_NULL;
  if (vocab_offset < 0 || V_local < 1 || vocab_offset + V_local > V_total || V_total >= (1ll << 30)) return KDKL_ERR_SHAPE;
  return forward_impl(hidden, weight_local, topk_idx, topk_val, teacher_lse, loss_mask, T, H, V_local, vocab_offset,
                      V_total, K, chunk, tau, opt, ws, ws_bytes, shard_stats, nullptr, nullptr, gathered_logits,
                      gathered_idx, cuda_stream);
}

int kdkl_forward_finish(const float* all_stats, int32_t n_shards, const uint8_t* loss_mask, int64_t T, int64_t H,
                        int64_t V_local, int32_t K, int64_t chunk, float tau, const kdkl_options* opt, void* ws,
                        size_t ws_bytes, float* loss_out, float* loss_per_token, void* cuda_stream) {
  g_launches = 0;
  if (!all_stats || !loss_out || !ws) return KDKL_ERR_NULL;
  if (n_shards < 1 || T < 1 || H < 1 || V_local < 1 || K < 1) return KDKL_ERR_SHAPE;
  kdkl_options o;
  memset(&o, 0, sizeof(o));
  if (copy_options(opt, &o) != KDKL_OK) return KDKL_ERR_ARG;
  WsLayout L = ws_layout(T, H, V_local, K, chunk, o.dw_chunks_per_pass);
  if (ws_bytes < L.total) return KDKL_ERR_WORKSPACE;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  WsHeader* hdr = at<WsHeader>(ws, L.hdr);
  shard_finish_kernel<<<(unsigned)((T + 255) / 256), 256, 0, st>>>(all_stats, n_shards, T, at<float>(ws, L.M),
                                                                   at<float>(ws, L.Hent), loss_mask,
                                                                   at<float>(ws, L.lz2), at<float>(ws, L.logZ),
                                                                   at<float>(ws, L.loss_tok), loss_per_token, hdr);
  KDKL_LAUNCHED("shard_finish_kernel");
  loss_reduce_kernel<<<1, 1024, 0, st>>>(at<float>(ws, L.loss_tok), loss_mask, T, o.denom_override, o.denom_device, tau,
                                         H, V_local, K, L.C, o.stored_exponentials ? G_EXPONENTIALS : G_NONE, loss_out,
                                         hdr);
  KDKL_LAUNCHED("loss_reduce_kernel");
  return KDKL_OK;
}

int kdkl_backward(const void* hidden, const void* weight, const uint8_t* loss_mask, int64_t T, int64_t H,
                  int64_t V, int32_t K, int64_t chunk, float tau, const kdkl_options* opt, float grad_loss, void* ws,
                  size_t ws_bytes, void* dhidden, float* dweight, void* cuda_stream) {
  g_launches = 0;
  if (!dhidden || !dweight) return KDKL_ERR_NULL;
  if (((uintptr_t)dhidden & 15) || ((uintptr_t)dweight & 15)) return KDKL_ERR_ALIGN;
  kdkl_options o;
  WsLayout L;
  DeviceInfo di;
  int rc = check_common(hidden, weight, T, H, V, K, chunk, tau, opt, ws, ws_bytes, &o, &L, &di);
  if (rc) return rc;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  WsHeader* hdr = at<WsHeader>(ws, L.hdr);
  const int* go = &hdr->go;
  const float inv_tau = 1.0f / tau;

  stage_mark(ST_COEF, st);
  bwd_coef_kernel<<<(unsigned)((T + 255) / 256), 256, 0, st>>>(at<float>(ws, L.M), loss_mask, T, H, V, K, L.C, tau,
                                                               o.stored_exponentials, grad_loss,
                                                               o.grad_loss_device, inv_tau, at<float>(ws, L.coefA),
                                                               at<float>(ws, L.coefB), hdr);
  KDKL_LAUNCHED("bwd_coef_kernel");

  __nv_bfloat16* Gbuf = at<__nv_bfloat16>(ws, L.G);
  // W as the K-major B operand of the recompute GEMM, and as the MN-major B operand of dH = G W
  CUtensorMap tmW, tmWmn;
  if ((rc = make_tmap_bf16(&tmW, weight, (uint64_t)H, (uint64_t)V, (uint64_t)H * 2, BK, kBRows))) return rc;
  if ((rc = make_tmap_bf16(&tmWmn, weight, (uint64_t)H, (uint64_t)V, (uint64_t)H * 2, 64, BK))) return rc;

  CUtensorMap tmdW;
  if ((rc = make_tmap_out_f32(&tmdW, dweight, (uint64_t)H, (uint64_t)V, (uint64_t)H))) return rc;

  // live-row-tile flags written by the forward call (same mask)
  const uint8_t* live = loss_mask != nullptr ? at<uint8_t>(ws, L.live) : nullptr;
  long long ci = 0;
  for (long long s0 = 0; s0 < T; s0 += L.C, ++ci) {
    const long long rows = (T - s0 < L.C) ? (T - s0) : L.C;
    const uint8_t* live_c = live ? live + ci * L.tiles_per_chunk : nullptr;
    const __nv_bfloat16* hA = reinterpret_cast<const __nv_bfloat16*>(hidden) + s0 * H;
    const GroupPos gp = group_pos(L, ci, s0, rows, T);
    __nv_bfloat16* G = Gbuf + gp.row0 * L.Vpad;            // this chunk's rows inside the group buffer
    CUtensorMap tmA;
    if ((rc = make_tmap_bf16(&tmA, hA, (uint64_t)H, (uint64_t)rows, (uint64_t)H * 2, BK, BM))) return rc;

    // B1: recompute logits, G = coefA * q - coefB * p
    GemmParams p;
    memset(&p, 0, sizeof(p));
    p.M = (int)rows; p.N = (int)V; p.K = (int)H;
    p.m_tiles = (int)((rows + kTileM - 1) / kTileM); p.n_tiles = (int)L.n_tiles_v; p.m_inner = 1; p.k_splits = 1;
    p.m_group = m_group_for(H);
    p.status = &hdr->status; p.go = go;
    p.scale_log2 = kLog2e * inv_tau; p.Ktop = K;
    p.idx_sorted = at<int>(ws, L.idx_sorted) + s0 * K;
    p.nvalid = at<int>(ws, L.nvalid) + s0;
    p.p_sorted = at<float>(ws, L.p_sorted) + s0 * K;
    p.lz2 = at<float>(ws, L.lz2) + s0;
    p.coefA = at<float>(ws, L.coefA) + s0;
    p.coefB = at<float>(ws, L.coefB) + s0;
    p.neg_a = &hdr->neg_grad;          // written by bwd_coef_kernel above
    // dead row tiles of G are written as zeros without being computed (up to MAX_LIVE_M row tiles per chunk)
    const uint8_t* live_m = (live_c && p.m_tiles <= MAX_LIVE_M) ? live_c : nullptr;
    p.m_live = live_m;
    CUtensorMap tmGout;
    if ((rc = make_tmap_out_bf16(&tmGout, G, (uint64_t)V, (uint64_t)rows, (uint64_t)L.Vpad))) return rc;
    stage_mark(ST_B1, st);
    if (o.stored_exponentials) {
      // the forward call left the exponentials of this (only) chunk in G: no second projection
      const int n_cols = (int)(((V + 7) / 8) * 8);
      const int n_seg = (n_cols + E2G_SEG - 1) / E2G_SEG;
      if ((long long)rows * n_seg > 2147483647ll) return KDKL_ERR_SHAPE;   // one block per (row, segment)
      e_to_g_kernel<<<(unsigned)(rows * n_seg), 256, 0, st>>>(
          G, L.Vpad, n_cols, (int)V, at<float>(ws, L.coefA) + s0, at<float>(ws, L.coefB) + s0,
          at<float>(ws, L.lz2) + s0, at<int>(ws, L.idx_sorted) + s0 * K, at<float>(ws, L.p_sorted) + s0 * K,
          at<int>(ws, L.nvalid) + s0, K, kExpBias, n_seg, hdr, go);
      KDKL_LAUNCHED("e_to_g_kernel");
    } else {
      if ((rc = launch_gemm<EPI_DLOGITS, false, false>(tmA, tmW, tmGout, p, di, st))) return rc;
    }

    ChunkOut co{G, hA, dhidden, s0, rows, H, V, &L, &o, hdr, ws, go, live_m, live_c, 0, nullptr};
    if ((rc = launch_dhidden(co, tmWmn, di, st))) return rc;
    if (g_pipe != nullptr && ci < (long long)g_pipe->dh_ready.size())
      KDKL_CUDA(cudaEventRecord(g_pipe->dh_ready[ci], st));            // this chunk's dhidden rows are final
    if (gp.last) {
      // one dW pass over the group that ends here: its chunks' G rows and hidden rows are contiguous
      const long long ci0 = ci - gp.j, g_s0 = s0 - gp.row0;
      ChunkOut cg{Gbuf, reinterpret_cast<const __nv_bfloat16*>(hidden) + g_s0 * H, nullptr, g_s0, gp.row0 + rows, H, V,
                  &L, &o, hdr, ws, go, nullptr, group_flags(L, live, ci0), (ci0 > 0 || o.accumulate_dweight) ? 1 : 0,
                  nullptr};
      if ((rc = launch_dweight(cg, tmdW, di, st))) return rc;
    }
  }
  return KDKL_OK;
}

// ------------------------------------------------------------------ single-pass forward + backward
// Same results as kdkl_forward followed by kdkl_backward (up to one more bf16 rounding inside G), with three
// projections instead of four: the forward sweep of a chunk also stores the unnormalised exponentials of its
// logits in the chunk's G buffer, and once the chunk's log Z is known they are turned into G in place.
int kdkl_forward_backward(const void* hidden, const void* weight, const int32_t* topk_idx, const float* topk_val,
                          const float* teacher_lse, const uint8_t* loss_mask, int64_t T, int64_t H, int64_t V, int32_t K,
                          int64_t chunk, float tau, const kdkl_options* opt, float grad_loss, void* ws, size_t ws_bytes,
                          float* loss_out, float* loss_per_token, void* dhidden, float* dweight, void* cuda_stream) {
  g_launches = 0;
  if (!topk_idx || !topk_val || !loss_out || !dhidden || !dweight) return KDKL_ERR_NULL;
  if (((uintptr_t)dhidden & 15) || ((uintptr_t)dweight & 15)) return KDKL_ERR_ALIGN;
  kdkl_options o;
  WsLayout L;
  DeviceInfo di;
  int rc = check_common(hidden, weight, T, H, V, K, chunk, tau, opt, ws, ws_bytes, &o, &L, &di);
  if (rc) return rc;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  WsHeader* hdr = at<WsHeader>(ws, L.hdr);
  const float inv_tau = 1.0f / tau;

  const uint8_t* live = nullptr;
  if ((rc = launch_prep(L, o, ws, topk_idx, topk_val, teacher_lse, loss_mask, T, V, 0, V, K, inv_tau, &live, st)))
    return rc;
  // the divisor of the mean and the per-token gradient coefficients are needed before the first chunk here
  count_tokens_kernel<<<1, 1024, 0, st>>>(loss_mask, T, o.denom_override, o.denom_device, hdr, nullptr);
  KDKL_LAUNCHED("count_tokens_kernel");
  step_coef_kernel<<<(unsigned)((T + 255) / 256), 256, 0, st>>>(at<float>(ws, L.M), loss_mask, T, grad_loss,
                                                                o.grad_loss_device, inv_tau, at<float>(ws, L.coefA),
                                                                at<float>(ws, L.coefB), hdr);
  KDKL_LAUNCHED("step_coef_kernel");

  __nv_bfloat16* Gbuf = at<__nv_bfloat16>(ws, L.G);
  CUtensorMap tmW, tmWmn, tmdW;
  if ((rc = make_tmap_bf16(&tmW, weight, (uint64_t)H, (uint64_t)V, (uint64_t)H * 2, BK, kBRows))) return rc;
  if ((rc = make_tmap_bf16(&tmWmn, weight, (uint64_t)H, (uint64_t)V, (uint64_t)H * 2, 64, BK))) return rc;
  if ((rc = make_tmap_out_f32(&tmdW, dweight, (uint64_t)H, (uint64_t)V, (uint64_t)H))) return rc;

  long long ci = 0;
  for (long long s0 = 0; s0 < T; s0 += L.C, ++ci) {
    const long long rows = (T - s0 < L.C) ? (T - s0) : L.C;
    const uint8_t* live_c = live ? live + ci * L.tiles_per_chunk : nullptr;
    const __nv_bfloat16* hA = reinterpret_cast<const __nv_bfloat16*>(hidden) + s0 * H;
    const GroupPos gp = group_pos(L, ci, s0, rows, T);
    __nv_bfloat16* G = Gbuf + gp.row0 * L.Vpad;
    CUtensorMap tmA, tmGout;
    if ((rc = make_tmap_bf16(&tmA, hA, (uint64_t)H, (uint64_t)rows, (uint64_t)H * 2, BK, BM))) return rc;
    if ((rc = make_tmap_out_bf16(&tmGout, G, (uint64_t)V, (uint64_t)rows, (uint64_t)L.Vpad))) return rc;

    // F1': logits tile by tile -> online log-sum-exp partials, gathered teacher logits, and e = 2^(s - bias) into G
    GemmParams p;
    fill_forward_params(&p, L, ws, s0, rows, H, V, K, inv_tau, live_c);
    p.coefA = at<float>(ws, L.coefA) + s0;         // rows without gradient store zeros instead of exponentials
    p.row_base = s0;
    const uint8_t* live_m = p.m_live;
    stage_mark(ST_F1, st);
    if ((rc = launch_gemm<EPI_LSE_E, false, false>(tmA, tmW, tmGout, p, di, st))) return rc;
    stage_mark(ST_COMBINE, st);
    combine_kernel<<<(unsigned)((rows + 31) / 32), COMBINE_WARPS * 32, 0, st>>>(
        at<float>(ws, L.part_m), at<float>(ws, L.part_s), L.Cpad, (int)L.n_tiles_v, (int)rows, s0, K, inv_tau,
        at<int>(ws, L.nvalid), at<float>(ws, L.p_sorted), at<uint16_t>(ws, L.perm), at<float>(ws, L.zg),
        at<int>(ws, L.colread), at<float>(ws, L.M), at<float>(ws, L.Hent), loss_mask, at<float>(ws, L.lz2),
        at<float>(ws, L.logZ), at<float>(ws, L.loss_tok), loss_per_token, nullptr, nullptr, 0, nullptr, T, hdr, 1);
    KDKL_LAUNCHED("combine_kernel");

    // With the chunk's log Z known: G = s_t e - b_t p. The row scale s_t leaves the contractions (the dH fix-up
    // multiplies by it, the dW pass reads hidden rows scaled by it) and only the <= K support entries per row
    // are patched in place: no pass over the [chunk, V] buffer.
    stage_mark(ST_B1, st);
    float* rs = at<float>(ws, L.rs) + s0;
    __nv_bfloat16* hs_group = at<__nv_bfloat16>(ws, L.hs);
    sp_scale_kernel<<<(unsigned)rows, 256, 0, st>>>(reinterpret_cast<const uint4*>(hA), (int)(H / 8),
                                                    at<float>(ws, L.coefA) + s0, at<float>(ws, L.lz2) + s0, kExpBias, rs,
                                                    reinterpret_cast<uint4*>(hs_group + gp.row0 * H));
    KDKL_LAUNCHED("sp_scale_kernel");
    sp_patch_kernel<<<(unsigned)((rows + 7) / 8), 256, 0, st>>>(
        G, L.Vpad, rows, rs, at<float>(ws, L.coefB) + s0, at<int>(ws, L.idx_sorted) + s0 * K,
        at<float>(ws, L.p_sorted) + s0 * K, at<int>(ws, L.nvalid) + s0, K);
    KDKL_LAUNCHED("sp_patch_kernel");

    // dH[chunk] = s (e' W) and dW (+)= e'^T (s h): the kernels of kdkl_backward, the scale applied outside them
    ChunkOut co{G, hA, dhidden, s0, rows, H, V, &L, &o, hdr, ws, nullptr, live_m, live_c, 0, rs};
    if ((rc = launch_dhidden(co, tmWmn, di, st))) return rc;
    if (gp.last) {
      const long long ci0 = ci - gp.j, g_s0 = s0 - gp.row0;
      ChunkOut cg{Gbuf, hs_group, nullptr, g_s0, gp.row0 + rows, H, V,
                  &L, &o, hdr, ws, nullptr, nullptr, group_flags(L, live, ci0), (ci0 > 0 || o.accumulate_dweight) ? 1 : 0,
                  nullptr};
      if ((rc = launch_dweight(cg, tmdW, di, st))) return rc;
    }
  }
  stage_mark(ST_REDUCE, st);
  loss_reduce_kernel<<<1, 1024, 0, st>>>(at<float>(ws, L.loss_tok), loss_mask, T, o.denom_override, o.denom_device, tau,
                                         H, V, K, L.C, G_NONE, loss_out, hdr);
  KDKL_LAUNCHED("loss_reduce_kernel");
  return KDKL_OK;
}

int kdkl_status(const void* ws, void* cuda_stream, int32_t* code, int64_t* detail) {
  if (!ws || !code) return KDKL_ERR_NULL;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  WsHeader h;
  KDKL_CUDA(cudaMemcpyAsync(&h, ws, sizeof(h), cudaMemcpyDeviceToHost, st));
  KDKL_CUDA(cudaStreamSynchronize(st));
  *code = h.status;
  if (detail) { detail[0] = h.where; detail[1] = h.n_tokens; detail[2] = h.n_bad_idx; }
  return KDKL_OK;
}

int kdkl_saved_state(void* ws, int64_t T, int64_t H, int64_t V, int32_t K, int64_t chunk, const kdkl_options* opt,
                     const float** logZ, const float** mass) {
  if (!ws) return KDKL_ERR_NULL;
  if (T < 1 || H < 1 || V < 1 || K < 1) return KDKL_ERR_SHAPE;
  WsLayout L = ws_layout(T, H, V, K, chunk, chunks_per_pass_of(opt));
  if (logZ) *logZ = at<float>(ws, L.logZ);
  if (mass) *mass = at<float>(ws, L.M);
  return KDKL_OK;
}

// ------------------------------------------------------------------ host-buffer entry point
struct ArenaLayout { size_t hidden, weight, idx, val, lse, mask, loss, dh, dw, ws, total; };
static ArenaLayout arena_layout(long long T, long long H, long long V, int K, long long chunk, int dh_fp32,
                                int chunks_per_pass) {
  ArenaLayout A;
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o = up(o + bytes, 256); return at; };
  A.hidden = take((size_t)T * H * 2);
  A.weight = take((size_t)V * H * 2);
  A.idx = take((size_t)T * K * 4);
  A.val = take((size_t)T * K * 4);
  A.lse = take((size_t)T * 4);
  A.mask = take((size_t)T);
  A.loss = take(256);
  A.dh = take((size_t)T * H * (dh_fp32 ? 4 : 2));
  A.dw = take((size_t)V * H * 4);
  A.ws = take(ws_layout(T, H, V, K, chunk, chunks_per_pass).total);
  A.total = o;
  return A;
}

size_t kdkl_host_arena_bytes(int64_t T, int64_t H, int64_t V, int32_t K, int64_t chunk, const kdkl_options* opt) {
  if (T < 1 || H < 1 || V < 1 || K < 1) return 0;
  return arena_layout(T, H, V, K, chunk, opt ? opt->dhidden_dtype : 0, chunks_per_pass_of(opt)).total;
}

int kdkl_forward_backward_host(const void* hidden, const void* weight, const int32_t* topk_idx, const float* topk_val,
                               const float* teacher_lse, const uint8_t* loss_mask, int64_t T, int64_t H, int64_t V,
                               int32_t K, int64_t chunk, float tau, const kdkl_options* opt, float grad_loss,
                               void* arena, size_t arena_bytes, float* loss_out, void* dhidden_out,
                               float* dweight_out, void* cuda_stream) {
  if (!hidden || !weight || !topk_idx || !topk_val || !arena || !loss_out) return KDKL_ERR_NULL;
  if (T < 1 || H < 1 || V < 1 || K < 1) return KDKL_ERR_SHAPE;
  if ((uintptr_t)arena & 255) return KDKL_ERR_ALIGN;
  const int dh32 = opt ? opt->dhidden_dtype : 0;
  ArenaLayout A = arena_layout(T, H, V, K, chunk, dh32, chunks_per_pass_of(opt));
  if (arena_bytes < A.total) return KDKL_ERR_WORKSPACE;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  uint8_t* d = reinterpret_cast<uint8_t*>(arena);
  const long long C = ws_layout(T, H, V, K, chunk, chunks_per_pass_of(opt)).C;
  const long long n_chunks = (T + C - 1) / C;
  const size_t dh_elem = dh32 ? 4 : 2;

  // Copies that overlap the chunk loop go over a second stream: the hidden rows of chunk i upstream while the
  // forward sweeps of earlier chunks run, the dhidden rows of chunk i downstream while later chunks are still
  // being differentiated. With one chunk there is nothing to overlap and everything stays on the caller's stream.
  HostPipe pipe;
  const bool piped = n_chunks > 1;
  auto cleanup = [&]() {
    for (cudaEvent_t e : pipe.in_ready) cudaEventDestroy(e);
    for (cudaEvent_t e : pipe.dh_ready) cudaEventDestroy(e);
    if (pipe.side) cudaStreamDestroy(pipe.side);
    g_pipe = nullptr;
  };
#define KDKL_PIPE(call)                                                          \
  do {                                                                           \
    cudaError_t e__ = (call);                                                    \
    if (e__ != cudaSuccess) { cleanup(); return cuda_fail(#call, e__); }         \
  } while (0)
  if (piped) {
    cudaEvent_t start;
    KDKL_PIPE(cudaStreamCreateWithFlags(&pipe.side, cudaStreamNonBlocking));
    KDKL_PIPE(cudaEventCreateWithFlags(&start, cudaEventDisableTiming));
    pipe.in_ready.push_back(start);                       // slot 0 doubles as "the caller's stream has reached this call"
    for (long long i = 0; i < n_chunks; ++i) {
      cudaEvent_t a, b;
      KDKL_PIPE(cudaEventCreateWithFlags(&a, cudaEventDisableTiming));
      pipe.in_ready.push_back(a);
      KDKL_PIPE(cudaEventCreateWithFlags(&b, cudaEventDisableTiming));
      pipe.dh_ready.push_back(b);
    }
    // the copy stream starts where the caller's stream stands (earlier work on the arena has finished by then)
    KDKL_PIPE(cudaEventRecord(pipe.in_ready[0], st));
    KDKL_PIPE(cudaStreamWaitEvent(pipe.side, pipe.in_ready[0], 0));
    cudaEventDestroy(pipe.in_ready[0]);
    pipe.in_ready.erase(pipe.in_ready.begin());
  }
  KDKL_PIPE(cudaMemcpyAsync(d + A.weight, weight, (size_t)V * H * 2, cudaMemcpyHostToDevice, st));
  KDKL_PIPE(cudaMemcpyAsync(d + A.idx, topk_idx, (size_t)T * K * 4, cudaMemcpyHostToDevice, st));
  KDKL_PIPE(cudaMemcpyAsync(d + A.val, topk_val, (size_t)T * K * 4, cudaMemcpyHostToDevice, st));
  if (teacher_lse) KDKL_PIPE(cudaMemcpyAsync(d + A.lse, teacher_lse, (size_t)T * 4, cudaMemcpyHostToDevice, st));
  if (loss_mask) KDKL_PIPE(cudaMemcpyAsync(d + A.mask, loss_mask, (size_t)T, cudaMemcpyHostToDevice, st));
  if (piped) {
    for (long long i = 0; i < n_chunks; ++i) {
      const long long s0 = i * C, rows = (T - s0 < C) ? (T - s0) : C;
      KDKL_PIPE(cudaMemcpyAsync(d + A.hidden + (size_t)s0 * H * 2, reinterpret_cast<const uint8_t*>(hidden) + (size_t)s0 * H * 2,
                                (size_t)rows * H * 2, cudaMemcpyHostToDevice, pipe.side));
      KDKL_PIPE(cudaEventRecord(pipe.in_ready[i], pipe.side));
    }
    g_pipe = &pipe;
  } else {
    KDKL_PIPE(cudaMemcpyAsync(d + A.hidden, hidden, (size_t)T * H * 2, cudaMemcpyHostToDevice, st));
  }
  const size_t ws_bytes = ws_layout(T, H, V, K, chunk, chunks_per_pass_of(opt)).total;
  int rc = kdkl_forward(d + A.hidden, d + A.weight, reinterpret_cast<int32_t*>(d + A.idx),
                        reinterpret_cast<float*>(d + A.val), teacher_lse ? reinterpret_cast<float*>(d + A.lse) : nullptr,
                        loss_mask ? d + A.mask : nullptr, T, H, V, K, chunk, tau, opt, d + A.ws, ws_bytes,
                        reinterpret_cast<float*>(d + A.loss), nullptr, nullptr, nullptr, cuda_stream);
  if (rc) { cleanup(); return rc; }
  const int64_t fl = g_launches;
  rc = kdkl_backward(d + A.hidden, d + A.weight, loss_mask ? d + A.mask : nullptr, T, H, V, K, chunk, tau, opt,
                     grad_loss, d + A.ws, ws_bytes, d + A.dh, reinterpret_cast<float*>(d + A.dw), cuda_stream);
  g_pipe = nullptr;
  if (rc) { cleanup(); return rc; }
  g_launches += fl;
  KDKL_PIPE(cudaMemcpyAsync(loss_out, d + A.loss, 4, cudaMemcpyDeviceToHost, st));
  if (dhidden_out) {
    if (piped) {
      // every dh_ready event has been recorded (enqueued) by kdkl_backward above, so these waits bind to them
      for (long long i = 0; i < n_chunks; ++i) {
        const long long s0 = i * C, rows = (T - s0 < C) ? (T - s0) : C;
        KDKL_PIPE(cudaStreamWaitEvent(pipe.side, pipe.dh_ready[i], 0));
        KDKL_PIPE(cudaMemcpyAsync(reinterpret_cast<uint8_t*>(dhidden_out) + (size_t)s0 * H * dh_elem,
                                  d + A.dh + (size_t)s0 * H * dh_elem, (size_t)rows * H * dh_elem,
                                  cudaMemcpyDeviceToHost, pipe.side));
      }
    } else {
      KDKL_PIPE(cudaMemcpyAsync(dhidden_out, d + A.dh, (size_t)T * H * dh_elem, cudaMemcpyDeviceToHost, st));
    }
  }
  if (dweight_out) KDKL_PIPE(cudaMemcpyAsync(dweight_out, d + A.dw, (size_t)V * H * 4, cudaMemcpyDeviceToHost, st));
  KDKL_PIPE(cudaStreamSynchronize(st));
  if (piped) KDKL_PIPE(cudaStreamSynchronize(pipe.side));
#undef KDKL_PIPE
  cleanup();
  return KDKL_OK;
}

// ------------------------------------------------------------------ step with the teacher record on the host
struct StagingLayout { size_t idx, val, lse, mask, loss, total; };
static StagingLayout staging_layout(long long T, int K) {
  StagingLayout S;
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o = up(o + bytes, 256); return at; };
  S.idx = take((size_t)T * K * 4);
  S.val = take((size_t)T * K * 4);
  S.lse = take((size_t)T * 4);
  S.mask = take((size_t)T);
  S.loss = take(256);
  S.total = o;
  return S;
}

size_t kdkl_record_staging_bytes(int64_t T, int32_t K) {
  if (T < 1 || K < 1) return 0;
  return staging_layout(T, K).total;
}

int kdkl_step_host_record(const void* hidden, const void* weight, const int32_t* topk_idx_host,
                          const float* topk_val_host, const float* teacher_lse_host, const uint8_t* loss_mask_host,
                          int64_t T, int64_t H, int64_t V, int32_t K, int64_t chunk, float tau, const kdkl_options* opt,
                          float grad_loss, void* staging, size_t staging_bytes, void* ws, size_t ws_bytes,
                          float* loss_out_host, void* dhidden, float* dweight, void* cuda_stream) {
  if (!topk_idx_host || !topk_val_host || !staging || !loss_out_host) return KDKL_ERR_NULL;
  if (T < 1 || K < 1) return KDKL_ERR_SHAPE;
  if ((uintptr_t)staging & 255) return KDKL_ERR_ALIGN;
  const StagingLayout S = staging_layout(T, K);
  if (staging_bytes < S.total) return KDKL_ERR_WORKSPACE;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  uint8_t* d = reinterpret_cast<uint8_t*>(staging);
  KDKL_CUDA(cudaMemcpyAsync(d + S.idx, topk_idx_host, (size_t)T * K * 4, cudaMemcpyHostToDevice, st));
  KDKL_CUDA(cudaMemcpyAsync(d + S.val, topk_val_host, (size_t)T * K * 4, cudaMemcpyHostToDevice, st));
  if (teacher_lse_host)
    KDKL_CUDA(cudaMemcpyAsync(d + S.lse, teacher_lse_host, (size_t)T * 4, cudaMemcpyHostToDevice, st));
  if (loss_mask_host) KDKL_CUDA(cudaMemcpyAsync(d + S.mask, loss_mask_host, (size_t)T, cudaMemcpyHostToDevice, st));
  const uint8_t* mask_d = loss_mask_host ? d + S.mask : nullptr;
  int rc = kdkl_forward(hidden, weight, reinterpret_cast<int32_t*>(d + S.idx), reinterpret_cast<float*>(d + S.val),
                        teacher_lse_host ? reinterpret_cast<float*>(d + S.lse) : nullptr, mask_d, T, H, V, K, chunk, tau,
                        opt, ws, ws_bytes, reinterpret_cast<float*>(d + S.loss), nullptr, nullptr, nullptr, cuda_stream);
  if (rc) return rc;
  const int64_t fl = g_launches;
  rc = kdkl_backward(hidden, weight, mask_d, T, H, V, K, chunk, tau, opt, grad_loss, ws, ws_bytes, dhidden, dweight,
                     cuda_stream);
  if (rc) return rc;
  g_launches += fl;
  KDKL_CUDA(cudaMemcpyAsync(loss_out_host, d + S.loss, 4, cudaMemcpyDeviceToHost, st));
  KDKL_CUDA(cudaStreamSynchronize(st));
  return KDKL_OK;
}

// ------------------------------------------------------------------ per-stage profile
int kdkl_profile_stages(const void* hidden, const void* weight, const int32_t* topk_idx, const float* topk_val,
                        const float* teacher_lse, const uint8_t* loss_mask, int64_t T, int64_t H, int64_t V, int32_t K,
                        int64_t chunk, float tau, const kdkl_options* opt, float grad_loss, void* ws, size_t ws_bytes,
                        float* loss_out, void* dhidden, float* dweight, void* cuda_stream, float* stage_ms,
                        int32_t* stage_launches) {
  if (!stage_ms || !stage_launches) return KDKL_ERR_NULL;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  stage_timer_start();
  int rc = kdkl_forward(hidden, weight, topk_idx, topk_val, teacher_lse, loss_mask, T, H, V, K, chunk, tau, opt, ws,
                        ws_bytes, loss_out, nullptr, nullptr, nullptr, cuda_stream);
  const int64_t fl = g_launches;
  if (rc == KDKL_OK)
    rc = kdkl_backward(hidden, weight, loss_mask, T, H, V, K, chunk, tau, opt, grad_loss, ws, ws_bytes, dhidden,
                       dweight, cuda_stream);
  g_launches += fl;
  return stage_timer_finish(rc, st, stage_ms, stage_launches);
}

// Same measurement for the single-pass step. Stage 5 is the in-place conversion of the stored exponentials
// (the place the recompute GEMM has in the two-call step).
int kdkl_profile_single_pass(const void* hidden, const void* weight, const int32_t* topk_idx, const float* topk_val,
                             const float* teacher_lse, const uint8_t* loss_mask, int64_t T, int64_t H, int64_t V,
                             int32_t K, int64_t chunk, float tau, const kdkl_options* opt, float grad_loss, void* ws,
                             size_t ws_bytes, float* loss_out, void* dhidden, float* dweight, void* cuda_stream,
                             float* stage_ms, int32_t* stage_launches) {
  if (!stage_ms || !stage_launches) return KDKL_ERR_NULL;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  stage_timer_start();
  int rc = kdkl_forward_backward(hidden, weight, topk_idx, topk_val, teacher_lse, loss_mask, T, H, V, K, chunk, tau,
                                 opt, grad_loss, ws, ws_bytes, loss_out, nullptr, dhidden, dweight, cuda_stream);
  return stage_timer_finish(rc, st, stage_ms, stage_launches);
}

// ------------------------------------------------------------------ teacher top-K cache record
constexpr long long kTopkTakeAllMaxV = 8192;
constexpr int kTopkRounds = 4;      // tightening rounds per pass: a list of 4 K slots then copes with 4 K * 4^4 candidates
struct TopkLayout {
  long long C, Cpad, n_tiles, ldz;
  int npad, cap, cpad;
  size_t hdr, flags, zeros, part_m, part_s, thr, cnt, cidx, cval, z, total;
  long long n_pass;
};
static int pow2_at_least(long long x) { int p = 32; while (p < x) p <<= 1; return p; }
static TopkLayout topk_layout(long long T, long long V, int K, bool stored = false) {
  TopkLayout L;
  L.C = T < 4096 ? T : 4096;
  L.Cpad = (long long)up((size_t)L.C, 128);
  L.n_tiles = (V + BN - 1) / BN;
  L.npad = pow2_at_least(L.n_tiles);
  // With at least K vocabulary tiles the threshold admits few more than K logits. With fewer tiles it says nothing
  // and every logit is a candidate: small vocabularies get a list that holds them all; larger ones start from
  // the standard list and rely on the tightening rounds (each keeps about K / cap of the candidates).
  long long cap = 4ll * K > 256 ? 4ll * K : 256;
  if (cap > 1024) cap = 1024;
  if (L.n_tiles < K && V <= kTopkTakeAllMaxV) cap = V;
  if (cap > V) cap = V;
  L.cap = (int)cap;
  L.cpad = pow2_at_least(L.cap);
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o = up(o + bytes, 256); return at; };
  L.hdr = take(256);
  L.n_pass = (T + L.C - 1) / L.C;
  L.flags = take((size_t)L.n_pass * kTopkRounds * 4);      // per pass: "rescan wanted" of each tightening round
  L.zeros = take((size_t)L.Cpad * 4);
  L.part_m = take((size_t)L.n_tiles * L.Cpad * 4);
  L.part_s = take((size_t)L.n_tiles * L.Cpad * 4);
  L.thr = take((size_t)L.Cpad * 4);
  L.cnt = take((size_t)L.Cpad * 4);
  L.cidx = take((size_t)L.Cpad * L.cap * 4);
  L.cval = take((size_t)L.Cpad * L.cap * 4);
  L.ldz = (long long)up((size_t)V, 32);                    // fp32 logits of one pass, when they are stored
  L.z = take(stored ? (size_t)L.Cpad * L.ldz * 4 : 0);
  L.total = o;
  return L;
}

size_t kdkl_teacher_topk_workspace_bytes(int64_t T, int64_t H, int64_t V, int32_t K) {
  if (T < 1 || H < 1 || V < 1 || K < 1) return 0;
  return topk_layout(T, V, K).total;
}

size_t kdkl_teacher_topk_stored_workspace_bytes(int64_t T, int64_t H, int64_t V, int32_t K) {
  if (T < 1 || H < 1 || V < 1 || K < 1) return 0;
  return topk_layout(T, V, K, true).total;
}

static int teacher_topk_impl(const void* hidden, const void* weight, int64_t T, int64_t H, int64_t V, int32_t K,
                             float tau, void* ws, size_t ws_bytes, int32_t* topk_idx, float* topk_val, float* lse,
                             void* cuda_stream, bool stored) {
  g_launches = 0;
  if (!hidden || !weight || !ws || !topk_idx || !topk_val || !lse) return KDKL_ERR_NULL;
  if (T < 1 || H < 1 || V < 1 || K < 1 || K > 256 || K > V || (H % 8) != 0 || V > (1ll << 20) || T >= (1ll << 31))
    return KDKL_ERR_SHAPE;
  if (!(tau > 0.f)) return KDKL_ERR_ARG;
  if (((uintptr_t)hidden & 15) || ((uintptr_t)weight & 15) || ((uintptr_t)ws & 15)) return KDKL_ERR_ALIGN;
  const TopkLayout L = topk_layout(T, V, K, stored);
  if (ws_bytes < L.total) return KDKL_ERR_WORKSPACE;
  DeviceInfo di;
  int rc = device_info(&di);
  if (rc) return rc;
  if (di.cc_major != 10) return KDKL_ERR_ARCH;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  int* status = at<int>(ws, L.hdr);
  KDKL_CUDA(cudaMemsetAsync(at<uint8_t>(ws, L.hdr), 0, L.zeros + (size_t)L.Cpad * 4 - L.hdr, st));   // header + zero counts

  CUtensorMap tmW;
  if ((rc = make_tmap_bf16(&tmW, weight, (uint64_t)H, (uint64_t)V, (uint64_t)H * 2, BK, kBRows))) return rc;
  long long pass = 0;
  for (long long s0 = 0; s0 < T; s0 += L.C, ++pass) {
    const long long rows = (T - s0 < L.C) ? (T - s0) : L.C;
    CUtensorMap tmA;
    const __nv_bfloat16* hA = reinterpret_cast<const __nv_bfloat16*>(hidden) + s0 * H;
    if ((rc = make_tmap_bf16(&tmA, hA, (uint64_t)H, (uint64_t)rows, (uint64_t)H * 2, BK, BM))) return rc;
    GemmParams p;
    memset(&p, 0, sizeof(p));
    p.M = (int)rows; p.N = (int)V; p.K = (int)H;
    p.m_tiles = (int)((rows + kTileM - 1) / kTileM); p.n_tiles = (int)L.n_tiles; p.m_inner = 1; p.k_splits = 1;
    p.status = status;
    p.scale_log2 = kLog2e / tau; p.Ktop = 1;
    p.nvalid = at<int>(ws, L.zeros); p.idx_sorted = at<int>(ws, L.zeros);     // no teacher entries to gather
    p.part_m = at<float>(ws, L.part_m); p.part_s = at<float>(ws, L.part_s); p.part_stride = L.Cpad;
    // sweep 1: per-tile maxima and sum-exp (and, in the stored form, the fp32 logits themselves)
    if (stored) {
      CUtensorMap tmZ;
      if ((rc = make_tmap_out_f32(&tmZ, at<float>(ws, L.z), (uint64_t)V, (uint64_t)rows, (uint64_t)L.ldz))) return rc;
      if ((rc = launch_gemm<EPI_LSE_Z, false, false>(tmA, tmW, tmZ, p, di, st))) return rc;
    } else {
      if ((rc = launch_gemm<EPI_LSE, false, false>(tmA, tmW, tmA, p, di, st))) return rc;
    }
    topk_threshold_kernel<<<(unsigned)rows, 32, (size_t)L.npad * 4, st>>>(
        at<float>(ws, L.part_m), at<float>(ws, L.part_s), L.Cpad, (int)L.n_tiles, L.npad, K, at<float>(ws, L.thr),
        at<int>(ws, L.cnt), lse + s0);
    KDKL_LAUNCHED("topk_threshold_kernel");
    if (stored) {
      // collect everything at or above the row's threshold from the stored logits
      const int n_seg = (int)((V + COLLECT_SEG - 1) / COLLECT_SEG);
      topk_collect_kernel<<<(unsigned)(rows * n_seg), 256, 0, st>>>(
          at<float>(ws, L.z), L.ldz, (int)V, p.scale_log2, at<float>(ws, L.thr), at<int>(ws, L.cnt),
          at<int>(ws, L.cidx), at<float>(ws, L.cval), L.cap, n_seg, nullptr);
      KDKL_LAUNCHED("topk_collect_kernel");
    } else {
      // sweep 2: recompute, emit everything at or above the row's threshold
      p.thr = at<float>(ws, L.thr); p.cand_cnt = at<int>(ws, L.cnt);
      p.cand_idx = at<int>(ws, L.cidx); p.cand_val = at<float>(ws, L.cval); p.cand_cap = L.cap;
      if ((rc = launch_gemm<EPI_TOPK, false, false>(tmA, tmW, tmA, p, di, st))) return rc;
    }
    // Lists that overflowed (more logits at or above the tile-maxima threshold than slots): rounds of a tighter
    // threshold and a new scan, each skipped on the device when no row of this pass asked for it.
    if (L.cap < V) {
      int* flags = at<int>(ws, L.flags) + kTopkRounds * pass;
      KDKL_CUDA(cudaFuncSetAttribute(topk_retighten_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, L.cpad * 4));
      for (int round = 0; round < kTopkRounds; ++round) {
        topk_retighten_kernel<<<(unsigned)rows, 32, (size_t)L.cpad * 4, st>>>(
            at<int>(ws, L.cnt), at<float>(ws, L.cval), L.cap, L.cpad, K, p.scale_log2, at<float>(ws, L.thr),
            flags + round, round == 0 ? nullptr : flags + round - 1);
        KDKL_LAUNCHED("topk_retighten_kernel");
        if (stored) {
          const int n_seg = (int)((V + COLLECT_SEG - 1) / COLLECT_SEG);
          topk_collect_kernel<<<(unsigned)(rows * n_seg), 256, 0, st>>>(
              at<float>(ws, L.z), L.ldz, (int)V, p.scale_log2, at<float>(ws, L.thr), at<int>(ws, L.cnt),
              at<int>(ws, L.cidx), at<float>(ws, L.cval), L.cap, n_seg, flags + round);
          KDKL_LAUNCHED("topk_collect_kernel");
        } else {
          p.thr = at<float>(ws, L.thr); p.cand_cnt = at<int>(ws, L.cnt);
          p.cand_idx = at<int>(ws, L.cidx); p.cand_val = at<float>(ws, L.cval); p.cand_cap = L.cap;
          p.go = flags + round;
          if ((rc = launch_gemm<EPI_TOPK, false, false>(tmA, tmW, tmA, p, di, st))) return rc;
          p.go = nullptr;
        }
      }
    }
    KDKL_CUDA(cudaFuncSetAttribute(topk_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, L.cpad * 8));
    topk_select_kernel<<<(unsigned)rows, 32, (size_t)L.cpad * 8, st>>>(
        at<int>(ws, L.cnt), at<int>(ws, L.cidx), at<float>(ws, L.cval), L.cap, L.cpad, K, topk_idx, topk_val, s0,
        status);
    KDKL_LAUNCHED("topk_select_kernel");
  }
  return KDKL_OK;
}

int kdkl_teacher_topk(const void* hidden, const void* weight, int64_t T, int64_t H, int64_t V, int32_t K, float tau,
                      void* ws, size_t ws_bytes, int32_t* topk_idx, float* topk_val, float* lse, void* cuda_stream) {
  return teacher_topk_impl(hidden, weight, T, H, V, K, tau, ws, ws_bytes, topk_idx, topk_val, lse, cuda_stream, false);
}

int kdkl_teacher_topk_stored(const void* hidden, const void* weight, int64_t T, int64_t H, int64_t V, int32_t K,
                             float tau, void* ws, size_t ws_bytes, int32_t* topk_idx, float* topk_val, float* lse,
                             void* cuda_stream) {
  return teacher_topk_impl(hidden, weight, T, H, V, K, tau, ws, ws_bytes, topk_idx, topk_val, lse, cuda_stream, true);
}

// ------------------------------------------------------------------ hidden-state feature loss
static size_t feature_ws_bytes(long long T) { return up(256 + sizeof(float) * (size_t)(T > 0 ? T : 0), 256); }

size_t kdkl_feature_loss_workspace_bytes(int64_t T) { return feature_ws_bytes(T); }

}  // extern "C"

// grad_dev: the upstream gradient on the device (then grad_loss is ignored), or nullptr.
static int feature_loss_impl(const void* student, const void* teacher, const uint8_t* loss_mask, int64_t T, int64_t H,
                             int32_t kind, float weight, float grad_loss, const float* grad_dev, float denom_override,
                             int32_t accumulate, void* workspace, size_t workspace_bytes, float* loss_out,
                             float* loss_per_token, void* dstudent, void* cuda_stream) {
  g_launches = 0;
  if (grad_dev != nullptr) grad_loss = 1.0f;
  if (!student || !teacher || !workspace || !loss_out) return KDKL_ERR_NULL;
  if (T < 1 || H < 1 || (H % 8) != 0 || T >= (1ll << 31) || H >= (1ll << 31)) return KDKL_ERR_SHAPE;
  if (kind != KDKL_FEATURE_MSE && kind != KDKL_FEATURE_COSINE) return KDKL_ERR_ARG;
  if (!isfinite(weight) || !isfinite(grad_loss) || (accumulate != 0 && accumulate != 1)) return KDKL_ERR_ARG;
  if (((uintptr_t)student & 15) || ((uintptr_t)teacher & 15) || ((uintptr_t)workspace & 15) ||
      ((uintptr_t)dstudent & 15))
    return KDKL_ERR_ALIGN;
  if (workspace_bytes < feature_ws_bytes(T)) return KDKL_ERR_WORKSPACE;
  DeviceInfo di;
  int rc = device_info(&di);
  if (rc) return rc;
  if (di.cc_major != 10) return KDKL_ERR_ARCH;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  float* tok = loss_per_token ? loss_per_token : at<float>(workspace, 256);
  // With a mask, N is counted on the device into the workspace header; without one N = T (or the
  // override) is known here and travels as a kernel argument, which saves a launch.
  const FeatHeader* hdr = nullptr;
  FeatHeader direct;
  memset(&direct, 0, sizeof(direct));
  if (loss_mask || grad_dev) {
    hdr = at<FeatHeader>(workspace, 0);
    feature_count_kernel<<<1, 1024, 0, st>>>(loss_mask, T, weight, grad_loss, grad_dev, denom_override,
                                             at<FeatHeader>(workspace, 0));
    KDKL_LAUNCHED("feature_count_kernel");
  } else {
    const float denom = denom_override > 0.f ? denom_override : (float)T;
    direct.n_counted = T;
    direct.g = grad_loss * weight / denom;
    direct.loss_scale = weight / denom;
  }
  const int nvec = (int)(H / 8);
  const uint4* S = reinterpret_cast<const uint4*>(student);
  const uint4* R = reinterpret_cast<const uint4*>(teacher);
  uint4* dS = reinterpret_cast<uint4*>(dstudent);
  // Threads per row: one warp up to 1024 columns; 128 threads (two rows per block, up to four 16-byte
  // vectors of each operand per thread in flight) up to 4096 columns; the whole block beyond. The grid
  // is capped at 16 blocks per SM and walks the rows with a stride. Measured at H = 4096 on one box:
  // 128 threads per row with this cap reaches 0.96-0.99 of the copy bandwidth, 256 threads per row
  // with a cap of 8 blocks per SM 0.79-0.87.
  const int group = nvec <= 128 ? 32 : (nvec <= 512 ? 128 : 256);
  const int nv = (nvec + group - 1) / group;
  const long long blocks_needed = (T + (256 / group) - 1) / (256 / group);
  const long long cap = (long long)di.sm_count * 16;
  const int grid = (int)(blocks_needed < cap ? blocks_needed : cap);
#define KDKL_FEAT_ROWS(KIND_, GROUP_) \
  launch_feature_rows<KIND_, GROUP_>(nv, grid, st, S, R, loss_mask, T, nvec, hdr, direct, accumulate, tok, dS)
  if (kind == KDKL_FEATURE_MSE) {
    if (group == 32) KDKL_FEAT_ROWS(0, 32); else if (group == 128) KDKL_FEAT_ROWS(0, 128); else KDKL_FEAT_ROWS(0, 256);
  } else {
    if (group == 32) KDKL_FEAT_ROWS(1, 32); else if (group == 128) KDKL_FEAT_ROWS(1, 128); else KDKL_FEAT_ROWS(1, 256);
  }
#undef KDKL_FEAT_ROWS
  KDKL_LAUNCHED("feature_rows_kernel");
  feature_reduce_kernel<<<1, 1024, 0, st>>>(tok, T, hdr, direct, loss_out);
  KDKL_LAUNCHED("feature_reduce_kernel");
  return KDKL_OK;
}

extern "C" {

int kdkl_feature_loss(const void* student, const void* teacher, const uint8_t* loss_mask, int64_t T, int64_t H,
                      int32_t kind, float weight, float grad_loss, float denom_override, int32_t accumulate,
                      void* workspace, size_t workspace_bytes, float* loss_out, float* loss_per_token, void* dstudent,
                      void* cuda_stream) {
  return feature_loss_impl(student, teacher, loss_mask, T, H, kind, weight, grad_loss, nullptr, denom_override,
                           accumulate, workspace, workspace_bytes, loss_out, loss_per_token, dstudent, cuda_stream);
}

int kdkl_feature_loss_device_grad(const void* student, const void* teacher, const uint8_t* loss_mask, int64_t T,
                                  int64_t H, int32_t kind, float weight, const float* grad_loss_device,
                                  float denom_override, int32_t accumulate, void* workspace, size_t workspace_bytes,
                                  float* loss_out, float* loss_per_token, void* dstudent, void* cuda_stream) {
  if (!grad_loss_device) return KDKL_ERR_NULL;
  return feature_loss_impl(student, teacher, loss_mask, T, H, kind, weight, 1.0f, grad_loss_device, denom_override,
                           accumulate, workspace, workspace_bytes, loss_out, loss_per_token, dstudent, cuda_stream);
}

// ------------------------------------------------------------------ bounded-wait self-test
int kdkl_wait_selftest(int32_t* status, int64_t limit_ns, void* cuda_stream) {
  if (!status) return KDKL_ERR_NULL;
  if (limit_ns < 1 || limit_ns > 1000000000ll) return KDKL_ERR_ARG;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  wait_expiry_kernel<<<1, 32, 0, st>>>(status, (unsigned long long)limit_ns, 99);
  KDKL_LAUNCHED("wait_expiry_kernel");
  return KDKL_OK;
}

// ------------------------------------------------------------------ bare GEMM
int kdkl_gemm_bf16(const void* A, const void* B, float* C, int64_t M, int64_t N, int64_t K, int32_t a_mn, int32_t b_mn,
                   int32_t* status, void* cuda_stream) {
  g_launches = 0;
  if (!A || !B || !C) return KDKL_ERR_NULL;
  if (M < 1 || N < 1 || K < 1 || (M % 8) || (N % 8) || (K % 8)) return KDKL_ERR_SHAPE;
  if (((uintptr_t)A & 15) || ((uintptr_t)B & 15) || ((uintptr_t)C & 15)) return KDKL_ERR_ALIGN;
  DeviceInfo di;
  int rc = device_info(&di);
  if (rc) return rc;
  if (di.cc_major != 10) return KDKL_ERR_ARCH;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(cuda_stream);
  CUtensorMap ta, tb;
  if (a_mn) rc = make_tmap_bf16(&ta, A, (uint64_t)M, (uint64_t)K, (uint64_t)M * 2, 64, BK);
  else      rc = make_tmap_bf16(&ta, A, (uint64_t)K, (uint64_t)M, (uint64_t)K * 2, BK, BM);
  if (rc) return rc;
  if (b_mn) rc = make_tmap_bf16(&tb, B, (uint64_t)N, (uint64_t)K, (uint64_t)N * 2, 64, BK);
  else      rc = make_tmap_bf16(&tb, B, (uint64_t)K, (uint64_t)N, (uint64_t)K * 2, BK, kBRows);
  if (rc) return rc;
  GemmParams p;
  memset(&p, 0, sizeof(p));
  p.M = (int)M; p.N = (int)N; p.K = (int)K;
  const bool wide = use_wide(N);                // the same choice of tile width as the loss's output GEMMs
  p.m_tiles = (int)((M + kTileM - 1) / kTileM); p.n_tiles = (int)n_tiles_for(N, wide); p.k_splits = 1;
  p.m_inner = p.m_tiles <= p.n_tiles ? 1 : 0;   // walk the shorter dimension first: the other operand streams once
  p.status = status; p.accumulate = 0;
  CUtensorMap tc;
  if ((rc = make_tmap_out_f32(&tc, C, (uint64_t)N, (uint64_t)M, (uint64_t)N))) return rc;
  if (wide) {
    if (a_mn && b_mn) return launch_gemm<EPI_STORE_F32, true, true, true>(ta, tb, tc, p, di, st);
    if (a_mn) return launch_gemm<EPI_STORE_F32, true, false, true>(ta, tb, tc, p, di, st);
    if (b_mn) return launch_gemm<EPI_STORE_F32, false, true, true>(ta, tb, tc, p, di, st);
    return launch_gemm<EPI_STORE_F32, false, false, true>(ta, tb, tc, p, di, st);
  }
  if (a_mn && b_mn) return launch_gemm<EPI_STORE_F32, true, true>(ta, tb, tc, p, di, st);
  if (a_mn) return launch_gemm<EPI_STORE_F32, true, false>(ta, tb, tc, p, di, st);
  if (b_mn) return launch_gemm<EPI_STORE_F32, false, true>(ta, tb, tc, p, di, st);
  return launch_gemm<EPI_STORE_F32, false, false>(ta, tb, tc, p, di, st);
}

}  // extern "C"
