// The small kernels around the GEMMs: teacher preparation, partial log-sum-exp combine,
// loss reduction and backward coefficients. All are bandwidth-trivial
// next to the tensor-core phases; they use warp-shuffle reductions and fixed-order sums
// (no floating-point atomics), so results are reproducible run to run.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "sm100_prims.cuh"

namespace kdkl {

constexpr int KDKL_MAGIC = 0x4b444b4c;  // "KDKL"
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kLog2e = 1.4426950408889634f;

// Head of the workspace (256 bytes). Written by forward, read by backward.
struct WsHeader {
  int status;        // 0 or the first device-detected error code
  int where;         // detail for the error (wait site, row, ...)
  int magic;         // KDKL_MAGIC once forward has completed its last kernel
  int go;            // backward gate: 1 when the state matches the call, else 0
  long long T, H, V;
  int K;
  int n_bad_idx;     // teacher indices >= V seen by prep (ignored entries)
  long long n_tokens;  // number of counted tokens (mask = 1)
  float denom;       // divisor of the mean actually used
  float tau;
  double loss_sum;   // sum of counted per-token losses
  long long chunk;   // tokens per chunk of the forward call that filled the workspace
  int g_state;       // what the [chunk, V] buffer holds after forward: G_NONE, G_EXPONENTIALS (option
                     // stored_exponentials: backward converts them once), G_CONSUMED (they have been converted)
  int neg_grad;      // 1 when the upstream gradient of the backward call in flight is negative (the recompute
                     // GEMM carries |a_t| in the exponent and needs the sign separately)
};
enum { G_NONE = 0, G_EXPONENTIALS = 1, G_CONSUMED = 2 };

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

__global__ void header_reset_kernel(WsHeader* hdr) {
  if (threadIdx.x == 0 && blockIdx.x == 0) {
    hdr->status = 0; hdr->where = 0; hdr->magic = 0; hdr->go = 0;
    hdr->n_bad_idx = 0; hdr->n_tokens = 0; hdr->denom = 0.f; hdr->loss_sum = 0.0;
    hdr->chunk = 0; hdr->g_state = G_NONE; hdr->neg_grad = 0;
  }
}

// ------------------------------------------------------------------------------------ prep
// One warp per token. From the cached teacher values l[t,k] and tau:
//   p_k = exp(l_k/tau - Lambda_t), Lambda_t = teacher_lse[t] | logsumexp_k(l_k/tau) | 0 (log-prob mode)
//   M_t = sum_k p_k (retained mass, never renormalised), Hent_t = sum_v p_v log p_v
// and an index-sorted copy of the row (idx ascending, p merged over duplicate indices, the
// original slot of every entry) that the GEMM epilogues walk with a cursor.
// Ignored tokens (mask = 0) get an empty row: their teacher entries are never read.
// Vocabulary shards: this rank owns rows [v0, v0 + V) of a vocabulary of V_total entries. Every
// usable teacher entry (index < V_total) counts towards p, M and Hent on every rank; only the
// entries inside the local window are gathered here, under their local index.
constexpr int PREP_WARPS = 4;
constexpr int kKeyUnusable = 0x7ffffffe, kKeyPad = 0x7fffffff;
__global__ void __launch_bounds__(PREP_WARPS * 32)
prep_kernel(const int* __restrict__ topk_idx, const float* __restrict__ topk_val,
            const float* __restrict__ teacher_lse, const uint8_t* __restrict__ mask, long long T, int V, int v0,
            int V_total, int K, int Kpad, float inv_tau, int teacher_mode, int* __restrict__ idx_sorted, float* __restrict__ p_sorted,
            uint16_t* __restrict__ perm, int* __restrict__ nvalid, float* __restrict__ Mout,
            float* __restrict__ Hent, WsHeader* hdr) {
  extern __shared__ uint8_t prep_smem[];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // One 64-bit word per entry is sorted: (key << 16) | slot. The probabilities stay where their slot put them and
  // are looked up through the slot afterwards, so a compare-exchange moves 8 bytes, not three arrays; equal indices
  // come out in slot order, which fixes the order their probabilities are added in.
  unsigned long long* ks = reinterpret_cast<unsigned long long*>(prep_smem) + warp * Kpad;
  float* pv = reinterpret_cast<float*>(prep_smem + sizeof(unsigned long long) * PREP_WARPS * Kpad) + warp * Kpad;
  auto key_of = [&](int j) { return (int)(ks[j] >> 16); };
  auto p_of = [&](int j) { return pv[(int)(ks[j] & 0xffffu)]; };

  const long long t = (long long)blockIdx.x * PREP_WARPS + warp;
  if (t >= T) return;
  const bool counted = mask == nullptr || mask[t] != 0;
  int* out_idx = idx_sorted + t * K;
  float* out_p = p_sorted + t * K;
  uint16_t* out_perm = perm + t * K;
  if (!counted) {
    for (int k = lane; k < K; k += 32) { out_idx[k] = 0x7fffffff; out_p[k] = 0.f; out_perm[k] = (uint16_t)k; }
    if (lane == 0) { nvalid[t] = 0; Mout[t] = 0.f; Hent[t] = 0.f; }
    return;
  }
  // load, validate, scaled values
  float mx = -INFINITY;
  int bad = 0;
  // keys: the global index < kKeyUnusable (real slot without a usable index) < kKeyPad (sort padding).
  // Every rank sorts the same keys, so M and Hent below are summed in the same order everywhere and
  // come out bitwise identical on all shards.
  for (int k = lane; k < Kpad; k += 32) {
    int key = k < K ? kKeyUnusable : kKeyPad;
    float u = -INFINITY;
    if (k < K) {
      const int id = topk_idx[t * K + k];
      if (id >= 0 && id < V_total) {
        key = id;
        u = topk_val[t * K + k] * inv_tau;
      } else if (id >= V_total) bad++;
    }
    ks[k] = ((unsigned long long)(unsigned)key << 16) | (unsigned)k;
    pv[k] = u;
    mx = fmaxf(mx, u);
  }
  bad = (int)warp_sum((float)bad);
  if (bad && lane == 0) { atomicAdd(&hdr->n_bad_idx, bad); atomicCAS(&hdr->status, 0, -10); }
  float lam;
  if (teacher_mode == 1) lam = 0.f;
  else if (teacher_lse != nullptr) lam = teacher_lse[t];
  else {
    mx = warp_max(mx);
    if (!(mx > -INFINITY)) mx = 0.f;
    __syncwarp();
    float s = 0.f;
    for (int k = lane; k < Kpad; k += 32) s += expf(pv[k] - mx);
    s = warp_sum(s);
    lam = mx + logf(s);
  }
  __syncwarp();
  for (int k = lane; k < Kpad; k += 32) pv[k] = key_of(k) < kKeyUnusable ? expf(pv[k] - lam) : 0.f;
  __syncwarp();
  // bitonic sort of the (key, slot) words
  for (int size = 2; size <= Kpad; size <<= 1) {
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
      for (int i = lane; i < (Kpad >> 1); i += 32) {
        const int lo = 2 * i - (i & (stride - 1));
        const int hi = lo + stride;
        const bool up = (lo & size) == 0;
        const unsigned long long a = ks[lo], b = ks[hi];
        if ((a > b) == up) { ks[lo] = b; ks[hi] = a; }
      }
      __syncwarp();
    }
  }
  // merge duplicate indices into the head of each run (scatter-add semantics). Shared memory is only
  // read from here on, so lanes may run ahead of each other.
  auto merged_p = [&](int j) -> float {
    const int key = key_of(j);
    if (key >= kKeyUnusable || (j > 0 && key_of(j - 1) == key)) return 0.f;
    float pj = p_of(j);
    for (int q = j + 1; q < Kpad && key_of(q) == key; ++q) pj += p_of(q);
    return pj;
  };
  // M, Hent, and the number of entries below / inside this rank's vocabulary window [v0, v0 + V)
  float msum = 0.f, hsum = 0.f;
  int lo = 0, hi = 0;
  for (int j = lane; j < Kpad; j += 32) {
    const int key = key_of(j);
    if (key < kKeyUnusable) {
      if (key < v0) lo++;
      if (key < v0 + V) hi++;
      const float pj = merged_p(j);
      msum += pj;
      if (pj > 0.f) hsum += pj * logf(pj);
    }
  }
  msum = warp_sum(msum); hsum = warp_sum(hsum);
  lo = (int)warp_sum((float)lo); hi = (int)warp_sum((float)hi);
  // write out with the local window rotated to the front: positions [0, hi - lo) hold this rank's
  // entries under their local index, ascending; the rest follows (never gathered here)
  const int nv = hi - lo;
  for (int j = lane; j < K; j += 32) {
    const int key = key_of(j);
    const bool local = j >= lo && j < hi;
    const int pos = local ? j - lo : (j < lo ? nv + j : j);
    out_idx[pos] = local ? key - v0 : key;
    out_p[pos] = merged_p(j);
    out_perm[pos] = (uint16_t)(ks[j] & 0xffffu);
  }
  if (lane == 0) { nvalid[t] = nv; Mout[t] = msum; Hent[t] = hsum; }
}

// ------------------------------------------------------------------------------------ single-pass step
// The single-pass forward + backward needs the divisor of the mean before the first chunk (the
// two-call path learns it at the end of forward): N = number of counted tokens, or the override (a host
// value, or a device value the caller reduced over its ranks: denom_dev).
__global__ void __launch_bounds__(1024)
count_tokens_kernel(const uint8_t* __restrict__ mask, long long T, float denom_override,
                    const double* __restrict__ denom_dev, WsHeader* hdr, double* __restrict__ count_out) {
  __shared__ long long part[32];
  long long c = 0;
  if (mask) { for (long long t = threadIdx.x; t < T; t += 1024) c += mask[t] != 0; }
  else if (threadIdx.x == 0) c = T;
  for (int o = 16; o; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
  if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = c;
  __syncthreads();
  if (threadIdx.x == 0) {
    long long n = 0;
    for (int i = 0; i < 32; ++i) n += part[i];
    if (count_out != nullptr) { *count_out = (double)n; return; }   // the stand-alone count (kdkl_count_tokens)
    hdr->n_tokens = n;
    hdr->denom = denom_dev != nullptr ? (float)*denom_dev : (denom_override > 0.f ? denom_override : (float)n);
  }
}

// a_t = g_t M_t / tau, b_t = g_t / tau with g_t = grad_loss * mask_t / N (Eq. "grad"), from the header's divisor.
// grad_dev: the upstream gradient on the device (nullptr: grad_loss).
__global__ void step_coef_kernel(const float* __restrict__ Mv, const uint8_t* __restrict__ mask, long long T,
                                 float grad_loss, const float* __restrict__ grad_dev, float inv_tau,
                                 float* __restrict__ coefA, float* __restrict__ coefB,
                                 const WsHeader* __restrict__ hdr) {
  const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= T) return;
  if (grad_dev != nullptr) grad_loss = *grad_dev;
  const float denom = hdr->denom;
  const bool counted = mask == nullptr || mask[t] != 0;
  const float g = (counted && denom > 0.f) ? grad_loss / denom : 0.f;
  coefA[t] = g * Mv[t] * inv_tau;
  coefB[t] = g * inv_tau;
}

// In place, per chunk: the forward sweep left e = 2^(s - bias) (bf16) in the G buffer; with log Z known,
//   G = a_t * 2^(s - lz2_t) - b_t p = (a_t * 2^(bias - lz2_t)) * e - b_t p at the support      (Eq. "grad")
// One block per (row, 8192-column segment): the dense scaling is a streaming pass (read + write of the
// chunk's G: the op is bound by HBM), then the row's support entries inside the segment are patched.
constexpr int E2G_VEC = 8;                     // 16-byte vectors per thread
constexpr int E2G_SEG = 256 * E2G_VEC * 8;     // columns per block: 256 threads x E2G_VEC vectors of 8
__global__ void __launch_bounds__(256)
e_to_g_kernel(__nv_bfloat16* __restrict__ G, long long ldg /* elements per row */, int n_cols /* V rounded up to 8 */,
              int V /* columns the forward sweep wrote; the rest of the last vector is stale memory */,
              const float* __restrict__ coefA, const float* __restrict__ coefB, const float* __restrict__ lz2,
              const int* __restrict__ idx_sorted, const float* __restrict__ p_sorted, const int* __restrict__ nvalid,
              int Ktop, float bias, int n_seg, WsHeader* hdr, const int* go) {
  if (go != nullptr && *go == 0) return;       // backward gate: the workspace does not hold this call's state
  // called from kdkl_backward (go given): the conversion is in place, so a second backward on this state must
  // not convert again - the header says so from here on (bwd_coef_kernel of that later call reads it)
  if (go != nullptr && blockIdx.x == 0 && threadIdx.x == 0) hdr->g_state = G_CONSUMED;
  const long long row = blockIdx.x / n_seg;
  const int c_begin = (int)(blockIdx.x - row * n_seg) * E2G_SEG;
  const int c_end = c_begin + E2G_SEG < n_cols ? c_begin + E2G_SEG : n_cols;
  const float a = coefA[row];
  uint4* g_row = reinterpret_cast<uint4*>(G + row * ldg);
  const int v_begin = c_begin / 8, v_end = c_end / 8;
  if (a == 0.f) {                              // ignored token (or zero upstream gradient): exact zeros, nothing read
    for (int v = v_begin + threadIdx.x; v < v_end; v += 256) g_row[v] = make_uint4(0u, 0u, 0u, 0u);
    return;
  }
  const float scale = a * exp2f(bias - lz2[row]);
  bool bad = false;                            // an exponential that overflowed bf16 (scaled logit beyond about 190)
  uint4 buf[E2G_VEC];
#pragma unroll
  for (int i = 0; i < E2G_VEC; ++i) {
    const int v = v_begin + threadIdx.x + i * 256;
    if (v < v_end) buf[i] = g_row[v];
  }
#pragma unroll
  for (int i = 0; i < E2G_VEC; ++i) {
    const int v = v_begin + threadIdx.x + i * 256;
    if (v < v_end) {
      __nv_bfloat162* h2 = reinterpret_cast<__nv_bfloat162*>(&buf[i]);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float2 x = __bfloat1622float2(h2[j]);
        const int col = v * 8 + 2 * j;
        const float y0 = col < V ? x.x * scale : 0.f, y1 = col + 1 < V ? x.y * scale : 0.f;
        bad |= !(fabsf(y0) <= 3.0e38f) || !(fabsf(y1) <= 3.0e38f);
        h2[j] = __floats2bfloat162_rn(y0, y1);
      }
      g_row[v] = buf[i];
    }
  }
  if (bad) { atomicCAS(&hdr->status, 0, -11); atomicCAS(&hdr->where, 0, (int)row); }
  // support entries of this row that fall into the segment (sorted ascending, duplicates merged by prep)
  const int nv = nvalid[row];
  if (nv == 0) return;
  __syncthreads();                             // the block's dense stores are visible to its own later loads
  const int* ids = idx_sorted + row * Ktop;
  int lo = 0, hi = nv;
  while (lo < hi) { const int mid = (lo + hi) >> 1; if (ids[mid] < c_begin) lo = mid + 1; else hi = mid; }
  const float b = coefB[row];
  __nv_bfloat16* g_el = G + row * ldg;
  for (int k = lo + threadIdx.x; k < nv; k += 256) {
    const int col = ids[k];
    if (col >= c_end) break;
    const float pk = p_sorted[row * Ktop + k];
    if (pk != 0.f) g_el[col] = __float2bfloat16_rn(__bfloat162float(g_el[col]) - b * pk);
  }
}

// Single-pass step without a dense conversion pass. With e = 2^(s - bias) stored by the forward sweep and log Z
// known, G = s_t e - b_t p with the row scale s_t = a_t 2^(bias - lz2_t) (Eq. "grad"). Instead of rewriting the
// whole [chunk, V] buffer, the scale is taken out of the two contractions:
//   dH[t,:] = s_t * (e' W)[t,:]           (applied in fp32 by the split-K fix-up)
//   dW      = e'^T (s (.) h)              (the chunk's hidden rows scaled once: chunk x H elements)
// with e' = e - (b_t / s_t) p at the <= K support entries of the row (patched in place). Rows without gradient
// (a_t = 0) were stored as zeros by the sweep and get scale 0.
__global__ void __launch_bounds__(256)
sp_scale_kernel(const uint4* __restrict__ h, int nvec /* H / 8 */, const float* __restrict__ coefA,
                const float* __restrict__ lz2, float bias, float* __restrict__ rs, uint4* __restrict__ hs) {
  const long long row = blockIdx.x;
  const float a = coefA[row];
  const float sc = a != 0.f ? a * exp2f(bias - lz2[row]) : 0.f;
  if (threadIdx.x == 0) rs[row] = sc;
  for (int v = threadIdx.x; v < nvec; v += 256) {
    uint4 x = h[row * nvec + v];
    __nv_bfloat162* h2 = reinterpret_cast<__nv_bfloat162*>(&x);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float2 f = __bfloat1622float2(h2[j]);
      h2[j] = __floats2bfloat162_rn(f.x * sc, f.y * sc);
    }
    hs[row * nvec + v] = x;
  }
}

// One warp per row: e'[t, v] = e[t, v] - (b_t / s_t) p_v at the row's support (sorted, duplicates merged by prep).
__global__ void __launch_bounds__(256)
sp_patch_kernel(__nv_bfloat16* __restrict__ G, long long ldg, long long rows, const float* __restrict__ rs,
                const float* __restrict__ coefB, const int* __restrict__ idx_sorted,
                const float* __restrict__ p_sorted, const int* __restrict__ nvalid, int Ktop) {
  const long long row = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
  if (row >= rows) return;
  const float sc = rs[row];
  if (sc == 0.f) return;
  const float c = coefB[row] / sc;
  const int nv = nvalid[row];
  __nv_bfloat16* g = G + row * ldg;
  for (int k = threadIdx.x & 31; k < nv; k += 32) {
    const float pk = p_sorted[row * Ktop + k];
    if (pk != 0.f) {
      const int col = idx_sorted[row * Ktop + k];
      g[col] = __float2bfloat16_rn(__bfloat162float(g[col]) - c * pk);
    }
  }
}

// ------------------------------------------------------------------------------------ live row tiles
// live[c * tiles_per_chunk + i] = 1 when at least one token of rows [c*chunk + i*tile_rows, ... + tile_rows)
// (clipped to the chunk and to T) is counted. The GEMM kernels skip row tiles whose flag is 0: a padding
// tail or a run of ignored tokens costs no tensor-core work. One warp per tile.
__global__ void __launch_bounds__(256)
tile_live_kernel(const uint8_t* __restrict__ mask, long long T, long long chunk, int tile_rows, int tiles_per_chunk,
                 long long n_flags, uint8_t* __restrict__ live) {
  const long long f = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
  if (f >= n_flags) return;
  const int lane = threadIdx.x & 31;
  const long long c = f / tiles_per_chunk, i = f - c * tiles_per_chunk;
  const long long r0 = c * chunk + i * tile_rows;
  long long r1 = r0 + tile_rows;
  if (r1 > (c + 1) * chunk) r1 = (c + 1) * chunk;
  if (r1 > T) r1 = T;
  int any = 0;
  for (long long r = r0 + lane; r < r1; r += 32) any |= mask[r] != 0;
  any = __any_sync(0xffffffffu, any);
  if (lane == 0) live[f] = any ? 1 : 0;
}

// ------------------------------------------------------------------------------------ combine
// Per chunk. Merges the per-vocab-tile (max, sum) partials of every row into the log-normaliser,
// adds the sparse terms and writes the per-token loss  L_t = Hent_t - C_t + M_t log Z_t
// (Eq. "decomp"), with C_t = sum_k p_k z_k / tau from the gathered logits. Also un-permutes the
// gathered logits / columns into the caller's slot order.
// Block = 32 rows x COMBINE_WARPS partial lanes; partial arrays are [n_tiles, part_stride] so reads
// coalesce. 32 lanes per row (1024 threads) keep 32 x 32 partial pairs in flight per block: the kernel
// reads chunk x n_tiles x 8 bytes (16 MiB at chunk 4096, V = 131072) and is bound by memory latency.
constexpr int COMBINE_WARPS = 32;
// With stored exponentials e = 2^(s - 64) in bf16, entries below s = -62 flush to zero. A row's entries that matter
// lie within about 20 of its log2-normaliser, so rows with lz2 >= -40 lose nothing; below that the call reports
// KDKL_ERR_RANGE (the two-call path has no such limit).
constexpr float kExpStoreMinLz2 = -40.f;
__global__ void __launch_bounds__(COMBINE_WARPS * 32)
combine_kernel(const float* __restrict__ part_m, const float* __restrict__ part_s, long long part_stride,
               int n_tiles, int rows, long long row0, int K, float inv_tau, const int* __restrict__ nvalid,
               const float* __restrict__ p_sorted, const uint16_t* __restrict__ perm, const float* __restrict__ zg,
               const int* __restrict__ colread, const float* __restrict__ Mv, const float* __restrict__ Hent,
               const uint8_t* __restrict__ mask, float* __restrict__ lz2, float* __restrict__ logZ_nat,
               float* __restrict__ loss_tok, float* __restrict__ loss_tok_user, float* __restrict__ g_logits,
               int* __restrict__ g_idx, int v0, float* __restrict__ shard_stats, long long T_total, WsHeader* hdr,
               int exp_stored) {
  __shared__ float sm_m[COMBINE_WARPS][32], sm_s[COMBINE_WARPS][32];
  __shared__ float sm_lz[32];
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const int r = blockIdx.x * 32 + tx;       // row within the chunk
  float m = -INFINITY, s = 0.f;
  // ignored tokens: their partials may not exist (a row tile with no counted token is skipped by the
  // GEMM), so nothing is read for them and their log Z is reported as 0
  const bool row_counted = r < rows && (mask == nullptr || mask[row0 + r] != 0);
  if (row_counted) {
    for (int nt = ty; nt < n_tiles; nt += COMBINE_WARPS) {
      const float pm = part_m[(long long)nt * part_stride + r];
      const float ps = part_s[(long long)nt * part_stride + r];
      const float mn = fmaxf(m, pm);
      s = s * exp2f(m - mn) + ps * exp2f(pm - mn);
      m = mn;
    }
  }
  sm_m[ty][tx] = m; sm_s[ty][tx] = s;
  __syncthreads();
  if (ty == 0 && r < rows) {
    float mm = sm_m[0][tx], ss = sm_s[0][tx];
    for (int i = 1; i < COMBINE_WARPS; ++i) {   // fixed order
      const float pm = sm_m[i][tx], ps = sm_s[i][tx];
      if (pm == -INFINITY) continue;
      const float mn = fmaxf(mm, pm);
      ss = ss * exp2f(mm - mn) + ps * exp2f(pm - mn);
      mm = mn;
    }
    const float l2 = row_counted ? mm + log2f(ss) : 0.f;
    // stored exponentials carry a fixed bias instead of the row maximum: a row whose scaled logits all sit
    // far below zero would flush to zero there (its softmax term would vanish from G unnoticed)
    if (exp_stored && row_counted && l2 < kExpStoreMinLz2) {
      atomicCAS(&hdr->status, 0, -13); atomicCAS(&hdr->where, 0, (int)(row0 + r));
    }
    sm_lz[tx] = l2;
    lz2[row0 + r] = l2;
    logZ_nat[row0 + r] = l2 * kLn2;
  }
  __syncthreads();
  // sparse terms: warp ty handles rows ty*RPW .. ty*RPW+RPW-1 of this block
  constexpr int RPW = 32 / COMBINE_WARPS;
  for (int i = 0; i < RPW; ++i) {
    const int rr = blockIdx.x * 32 + ty * RPW + i;
    if (rr >= rows) break;
    const long long t = row0 + rr;
    const int nv = nvalid[t];
    float c = 0.f;
    for (int j = tx; j < K; j += 32) {
      const int sl = perm[t * K + j];
      if (j < nv) {
        const float z = zg[t * K + j];
        c += p_sorted[t * K + j] * z;
        if (g_logits) g_logits[t * K + sl] = z;
        if (g_idx) g_idx[t * K + sl] = colread[t * K + j] + v0;
      } else {
        if (g_logits) g_logits[t * K + sl] = __int_as_float(0x7fc00000);
        if (g_idx) g_idx[t * K + sl] = -1;
      }
    }
    c = warp_sum(c) * inv_tau;
    if (shard_stats != nullptr) {
      // a vocabulary shard: hand the local log-normaliser and cross term to the cross-shard reduction
      if (tx == 0) { shard_stats[t] = sm_lz[ty * RPW + i]; shard_stats[T_total + t] = c; }
      continue;
    }
    if (tx == 0) {
      const bool counted = mask == nullptr || mask[t] != 0;
      const float lz = sm_lz[ty * RPW + i] * kLn2;
      float L = 0.f;
      if (counted) {
        L = Hent[t] - c + Mv[t] * lz;
        if (!isfinite(L)) { atomicCAS(&hdr->status, 0, -11); atomicCAS(&hdr->where, 0, (int)t); }
      }
      loss_tok[t] = L;
      if (loss_tok_user) loss_tok_user[t] = L;
    }
  }
}

// ------------------------------------------------------------------------------------ shard finish
// After the shards' statistics have been gathered ([R][2][T]: log2-domain local normaliser, local cross
// term): log Z = logsumexp over shards, C = sum over shards (fixed order), L = Hent - C + M log Z.
// Writes the global normaliser over the local one so that backward rebuilds the global softmax.
__global__ void shard_finish_kernel(const float* __restrict__ all_stats, int R, long long T,
                                    const float* __restrict__ Mv, const float* __restrict__ Hent,
                                    const uint8_t* __restrict__ mask, float* __restrict__ lz2,
                                    float* __restrict__ logZ_nat, float* __restrict__ loss_tok,
                                    float* __restrict__ loss_tok_user, WsHeader* hdr) {
  const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= T) return;
  float m = -INFINITY;
  for (int r = 0; r < R; ++r) m = fmaxf(m, all_stats[(long long)r * 2 * T + t]);
  float s = 0.f, c = 0.f;
  for (int r = 0; r < R; ++r) {
    s += exp2f(all_stats[(long long)r * 2 * T + t] - m);
    c += all_stats[(long long)r * 2 * T + T + t];
  }
  const float l2 = m + log2f(s);
  lz2[t] = l2;
  logZ_nat[t] = l2 * kLn2;
  const bool counted = mask == nullptr || mask[t] != 0;
  float L = 0.f;
  if (counted) {
    L = Hent[t] - c + Mv[t] * l2 * kLn2;
    if (!isfinite(L)) { atomicCAS(&hdr->status, 0, -11); atomicCAS(&hdr->where, 0, (int)t); }
  }
  loss_tok[t] = L;
  if (loss_tok_user) loss_tok_user[t] = L;
}

// ------------------------------------------------------------------------------------ loss reduce
// One block: loss = sum_t mask_t L_t / denom, summed in double in a fixed order. Marks the
// workspace as complete for backward.
__global__ void __launch_bounds__(1024)
loss_reduce_kernel(const float* __restrict__ loss_tok, const uint8_t* __restrict__ mask, long long T,
                   float denom_override, const double* __restrict__ denom_dev, float tau, long long H, long long V,
                   int K, long long chunk, int g_state, float* loss_out, WsHeader* hdr) {
  __shared__ double sm_sum[1024];
  __shared__ long long sm_cnt[1024];
  double acc = 0.0;
  long long cnt = 0;
  for (long long t = threadIdx.x; t < T; t += 1024) {
    const bool counted = mask == nullptr || mask[t] != 0;
    if (counted) { acc += (double)loss_tok[t]; cnt++; }
  }
  sm_sum[threadIdx.x] = acc; sm_cnt[threadIdx.x] = cnt;
  __syncthreads();
  for (int o = 512; o > 0; o >>= 1) {
    if (threadIdx.x < o) { sm_sum[threadIdx.x] += sm_sum[threadIdx.x + o]; sm_cnt[threadIdx.x] += sm_cnt[threadIdx.x + o]; }
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    const long long n = sm_cnt[0];
    const float denom = denom_dev != nullptr ? (float)*denom_dev : (denom_override > 0.f ? denom_override : (float)n);
    hdr->n_tokens = n; hdr->denom = denom; hdr->loss_sum = sm_sum[0]; hdr->tau = tau;
    hdr->T = T; hdr->H = H; hdr->V = V; hdr->K = K; hdr->chunk = chunk; hdr->g_state = g_state;
    *loss_out = denom > 0.f ? (float)(sm_sum[0] / (double)denom) : 0.f;
    __threadfence();
    hdr->magic = KDKL_MAGIC;
  }
}

// ------------------------------------------------------------------------------------ backward prep
// coefA_t = g_t M_t / tau, coefB_t = g_t / tau with g_t = grad_loss * mask_t / denom
// (Algorithm 1 backward: G = (M g) q, G -= p g; the 1/tau is the chain rule through z/tau).
// Also checks that the workspace was filled by a forward call of the same shape, chunk size and temperature,
// and - when backward is to convert stored exponentials instead of projecting again - that forward left
// them and no earlier backward has converted them already (the conversion is in place: it can run once;
// e_to_g_kernel marks them consumed). Block 0 records the decision in `go` for the kernels that follow;
// nothing the decision depends on is written by this grid.
__global__ void bwd_coef_kernel(const float* __restrict__ Mv, const uint8_t* __restrict__ mask, long long T,
                                long long H, long long V, int K, long long chunk, float tau, int want_exponentials,
                                float grad_loss, const float* __restrict__ grad_dev, float inv_tau,
                                float* __restrict__ coefA, float* __restrict__ coefB, WsHeader* hdr) {
  __shared__ int sm_ok;
  if (grad_dev != nullptr) grad_loss = *grad_dev;      // the upstream gradient lives on the device
  if (threadIdx.x == 0) {
    bool ok = hdr->magic == KDKL_MAGIC && hdr->T == T && hdr->H == H && hdr->V == V && hdr->K == K &&
              hdr->chunk == chunk && hdr->tau == tau;
    if (want_exponentials) ok = ok && hdr->g_state == G_EXPONENTIALS;
    sm_ok = ok ? 1 : 0;
  }
  __syncthreads();
  const bool state_ok = sm_ok != 0;
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    hdr->go = state_ok ? 1 : 0;
    hdr->neg_grad = grad_loss < 0.f ? 1 : 0;
    if (!state_ok) atomicCAS(&hdr->status, 0, -9);
  }
  if (!state_ok) return;
  const float denom = hdr->denom;
  const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= T) return;
  const bool counted = mask == nullptr || mask[t] != 0;
  const float g = (counted && denom > 0.f) ? grad_loss / denom : 0.f;
  coefA[t] = g * Mv[t] * inv_tau;
  coefB[t] = g * inv_tau;
}

// ------------------------------------------------------------------------------------ split-K fix-up
// out = part[0] + part[1] + ... in that fixed order (fp32), times the row's scale if given, then one rounding to
// bf16 if asked.
// part holds `splits` slabs `slab` elements apart; n4 = number of float4 groups to produce.
__global__ void __launch_bounds__(256)
splitk_fixup_kernel(const float* __restrict__ part, long long slab, int splits, long long n4,
                    __nv_bfloat16* __restrict__ out_bf16, float* __restrict__ out_f32, const int* go,
                    const float* __restrict__ row_scale, int row_n4 /* float4 groups per row */) {
  if (go != nullptr && *go == 0) return;
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n4) return;
  float4 a = reinterpret_cast<const float4*>(part)[i];
  for (int sidx = 1; sidx < splits; ++sidx) {
    const float4 b = reinterpret_cast<const float4*>(part + (long long)sidx * slab)[i];
    a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w;
  }
  if (row_scale != nullptr) {                  // single-pass step: the row's scale, taken out of the contraction
    const float sc = row_scale[i / row_n4];
    if (sc == 0.f) a = make_float4(0.f, 0.f, 0.f, 0.f);
    else { a.x *= sc; a.y *= sc; a.z *= sc; a.w *= sc; }
  }
  if (out_f32) reinterpret_cast<float4*>(out_f32)[i] = a;
  if (out_bf16) {
    __nv_bfloat162 lo = __floats2bfloat162_rn(a.x, a.y), hi = __floats2bfloat162_rn(a.z, a.w);
    uint2 v;
    v.x = *reinterpret_cast<uint32_t*>(&lo);
    v.y = *reinterpret_cast<uint32_t*>(&hi);
    reinterpret_cast<uint2*>(out_bf16)[i] = v;
  }
}

// ------------------------------------------------------------------------------------ teacher top-K
// Descending bitonic sort of n (power of two) keys in shared memory by one warp; `idx` (optional) is
// carried along and breaks ties by the smaller index.
__device__ __forceinline__ void warp_bitonic_desc(float* key, int* idx, int n, int lane) {
  for (int size = 2; size <= n; size <<= 1) {
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
      for (int i = lane; i < (n >> 1); i += 32) {
        const int lo = 2 * i - (i & (stride - 1));
        const int hi = lo + stride;
        const bool down = (lo & size) == 0;          // this block sorts descending
        const float a = key[lo], b = key[hi];
        bool a_first = a > b;                        // a belongs before b in descending order
        if (a == b && idx != nullptr) a_first = idx[lo] < idx[hi];
        if (a_first != down) {
          key[lo] = b; key[hi] = a;
          if (idx != nullptr) { const int t = idx[lo]; idx[lo] = idx[hi]; idx[hi] = t; }
        }
      }
      __syncwarp();
    }
  }
}

// Sweep 1 -> threshold. One warp (block) per row. From the per-vocab-tile partials of the log-sum-exp
// sweep: the row's log-sum-exp, and the K-th largest tile maximum. At least K logits reach that value
// (the K tile maxima themselves), so every member of the exact top-K does: it is a safe threshold.
__global__ void __launch_bounds__(32)
topk_threshold_kernel(const float* __restrict__ part_m, const float* __restrict__ part_s, long long part_stride,
                      int n_tiles, int npad, int K, float* __restrict__ thr, int* __restrict__ cand_cnt,
                      float* __restrict__ lse_out) {
  extern __shared__ float tk_smem[];
  const int row = blockIdx.x, lane = threadIdx.x;
  float m = -INFINITY;
  for (int i = lane; i < npad; i += 32) {
    const float v = i < n_tiles ? part_m[(long long)i * part_stride + row] : -INFINITY;
    tk_smem[i] = v;
    m = fmaxf(m, v);
  }
  m = warp_max(m);
  float s = 0.f;
  for (int i = lane; i < n_tiles; i += 32) s += part_s[(long long)i * part_stride + row] * exp2f(tk_smem[i] - m);
  s = warp_sum(s);
  __syncwarp();
  warp_bitonic_desc(tk_smem, nullptr, npad, lane);
  if (lane == 0) {
    thr[row] = n_tiles >= K ? tk_smem[K - 1] : -INFINITY;
    cand_cnt[row] = 0;
    lse_out[row] = (m + log2f(s)) * kLn2;
  }
}

// Teacher cache with stored logits: the candidates of a row are collected from the fp32 logits the first
// sweep stored, by the same test the recompute epilogue applies (z * scale >= the row's threshold, the
// same fp32 product). One block per (row, 8192-column segment); a streaming read of the logits.
constexpr int COLLECT_SEG = 8192;
__global__ void __launch_bounds__(256)
topk_collect_kernel(const float* __restrict__ z, long long ldz, int V, float scale_log2, const float* __restrict__ thr,
                    int* __restrict__ cand_cnt, int* __restrict__ cand_idx, float* __restrict__ cand_val, int cap,
                    int n_seg, const int* go) {
  if (go != nullptr && *go == 0) return;
  const long long row = blockIdx.x / n_seg;
  if (thr[row] == INFINITY) return;                  // a row that already holds its candidates
  const int c_begin = (int)(blockIdx.x - row * n_seg) * COLLECT_SEG;
  const float t = thr[row];
  const float4* zr = reinterpret_cast<const float4*>(z + row * ldz);
  float4 buf[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int c = c_begin + (threadIdx.x + i * 256) * 4;
    if (c < V) buf[i] = zr[c >> 2];                     // ldz is a multiple of 4: the last vector may hold stale columns
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int c = c_begin + (threadIdx.x + i * 256) * 4;
    if (c >= V) continue;
    const float v[4] = {buf[i].x, buf[i].y, buf[i].z, buf[i].w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      if (c + j < V && v[j] * scale_log2 >= t) {
        const int arrival = atomicAdd(cand_cnt + row, 1);
        const int slot = reservoir_slot(arrival, cap, (uint32_t)row, (uint32_t)(c + j));
        if (slot >= 0) {
          cand_idx[row * cap + slot] = c + j;
          cand_val[row * cap + slot] = v[j];
        }
      }
    }
  }
}

// Between sweep 2 and the record: a row whose candidate list overflowed (more logits reached the tile-maxima
// threshold than the list holds - large logits clustered in a few vocabulary tiles, as in a frequency-ordered
// vocabulary) gets a tighter threshold and is scanned again. The K-th largest of the candidates that were kept is
// a valid one: they are real logits of the row, so at least K logits reach it and every member of the exact
// top-K does. The kept ones are a uniform sample of all that arrived (reservoir_slot), so the tightened scan admits
// about K / cap of the previous count, whatever the order of arrival; the host enqueues a fixed number of such
// rounds, each skipped on the device when no row asked for it (*flag stays 0). Rows that fit keep their list and
// take no further candidates.
__global__ void __launch_bounds__(32)
topk_retighten_kernel(int* __restrict__ cand_cnt, const float* __restrict__ cand_val, int cap, int cpad, int K,
                      float scale_log2, float* __restrict__ thr, int* flag, const int* go) {
  extern __shared__ float tk_smem[];
  if (go != nullptr && *go == 0) return;             // second round: only when the first one ran
  const int row = blockIdx.x, lane = threadIdx.x;
  const int n = cand_cnt[row];
  if (n <= cap) {
    if (lane == 0) thr[row] = INFINITY;
    return;
  }
  for (int i = lane; i < cpad; i += 32) tk_smem[i] = i < cap ? cand_val[(long long)row * cap + i] : -INFINITY;
  __syncwarp();
  warp_bitonic_desc(tk_smem, nullptr, cpad, lane);
  if (lane == 0) {
    thr[row] = tk_smem[K - 1] * scale_log2;          // the same fp32 product the scan compares with
    cand_cnt[row] = 0;
    *flag = 1;
  }
}

// Sweep 2 -> record. One warp (block) per row: sort the emitted candidates by (logit descending, index
// ascending) and keep the first K. More candidates than the list holds is reported, not hidden.
__global__ void __launch_bounds__(32)
topk_select_kernel(const int* __restrict__ cand_cnt, const int* __restrict__ cand_idx,
                   const float* __restrict__ cand_val, int cap, int cpad, int K, int* __restrict__ out_idx,
                   float* __restrict__ out_val, long long row0, int* status) {
  extern __shared__ float tk_smem[];
  int* sidx = reinterpret_cast<int*>(tk_smem + cpad);
  const int row = blockIdx.x, lane = threadIdx.x;
  int n = cand_cnt[row];
  if (n > cap) {
    if (lane == 0) { atomicCAS(status, 0, -12); atomicCAS(status + 1, 0, (int)(row0 + row)); }
    n = cap;
  }
  for (int i = lane; i < cpad; i += 32) {
    tk_smem[i] = i < n ? cand_val[(long long)row * cap + i] : -INFINITY;
    sidx[i] = i < n ? cand_idx[(long long)row * cap + i] : 0x7fffffff;
  }
  __syncwarp();
  warp_bitonic_desc(tk_smem, sidx, cpad, lane);
  for (int k = lane; k < K; k += 32) {
    out_idx[(row0 + row) * K + k] = k < n ? sidx[k] : -1;
    out_val[(row0 + row) * K + k] = k < n ? tk_smem[k] : -INFINITY;
  }
}

// ------------------------------------------------------------------------------------ wait self-test
// One thread waits on an mbarrier that nothing will ever complete, with a short limit. The wait must
// give up, record KDKL_ERR_TIMEOUT and the site in status[0..1], and the kernel must return normally.
__global__ void wait_expiry_kernel(int* status, unsigned long long limit_ns, int site) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(smem_u32(&bar), 1);
    mbar_fence_init();
    const bool ok = mbar_wait(smem_u32(&bar), 0u, &abort_flag, status, site, limit_ns);
    if (ok) atomicExch(status + 1, -1);   // would mean the barrier completed by itself
  }
}

}  // namespace kdkl
