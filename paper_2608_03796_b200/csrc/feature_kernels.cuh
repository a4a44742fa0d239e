// Hidden-state feature loss added to the logit KL (paper, section "Additional Ablations", paragraph
// "Loss design": a mean-squared-error variant and a cosine variant; the paper prints no formula, so
// these are the textbook definitions).
//
// Per token t, student row s and teacher row r of width H:
//   MSE     f_t = (1/H) sum_h (s_h - r_h)^2            d s = g_t (2/H) (s - r)
//   cosine  f_t = 1 - <s,r> / (|s||r|)                 d s = -g_t ( r/(|s||r|) - <s,r> s/(|s|^3|r|) )
// loss = weight * sum_t mask_t f_t / N, g_t = grad_loss * weight * mask_t / N.
//
// The op is bound by HBM: 2 reads and 1 write of [T,H] bf16 with a few flops per element. Loss and
// gradient therefore come out of ONE pass over the inputs: a row's vectors stay in registers
// between the row reduction and the gradient, so nothing is read twice. Rows wider than the
// register budget re-read their tail (it is still in L1/L2 from the first touch).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace kdkl {

struct FeatHeader {
  long long n_counted;   // number of mask = 1 tokens in this call
  float g;               // grad_loss * weight / N (0 when N = 0)
  float loss_scale;      // weight / N (0 when N = 0)
};

// N = sum of the mask (or T), then the two scales every row needs. One block.
__global__ void __launch_bounds__(1024)
feature_count_kernel(const uint8_t* __restrict__ mask, long long T, float weight, float grad_loss,
                     const float* __restrict__ grad_dev /* the upstream gradient on the device, or nullptr */,
                     float denom_override, FeatHeader* __restrict__ hdr) {
  __shared__ long long part[32];
  if (grad_dev != nullptr) grad_loss = *grad_dev;
  long long c = 0;
  if (mask) {
    for (long long t = threadIdx.x; t < T; t += 1024) c += mask[t] != 0;
  } else if (threadIdx.x == 0) {
    c = T;
  }
  for (int o = 16; o; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
  if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = c;
  __syncthreads();
  if (threadIdx.x == 0) {
    long long n = 0;
    for (int i = 0; i < 32; ++i) n += part[i];
    const float denom = denom_override > 0.f ? denom_override : (float)n;
    hdr->n_counted = n;
    hdr->g = denom > 0.f ? grad_loss * weight / denom : 0.f;
    hdr->loss_scale = denom > 0.f ? weight / denom : 0.f;
  }
}

__device__ __forceinline__ void unpack8(const uint4& v, float (&f)[8]) {
  const __nv_bfloat162* p = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 x = __bfloat1622float2(p[i]);
    f[2 * i] = x.x; f[2 * i + 1] = x.y;
  }
}
__device__ __forceinline__ uint4 pack8(const float (&f)[8]) {
  uint4 v;
  __nv_bfloat162* p = reinterpret_cast<__nv_bfloat162*>(&v);
#pragma unroll
  for (int i = 0; i < 4; ++i) p[i] = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
  return v;
}

// Sums of up to three values over the GROUP threads that share a row (GROUP = 32: one warp, shuffles
// only; GROUP = 128 or 256: 4 or 8 warps through shared memory). One barrier per call: `sm` is one of
// two buffers used alternately by successive rows, so a warp that runs ahead into the next row writes
// the other buffer, and it cannot get two rows ahead without passing the next row's barrier.
template <int GROUP, int NVAL>
__device__ __forceinline__ void group_sum(float (&x)[3], float* sm) {
#pragma unroll
  for (int k = 0; k < NVAL; ++k)
    for (int o = 16; o; o >>= 1) x[k] += __shfl_xor_sync(0xffffffffu, x[k], o);
  if (GROUP == 32) return;
  constexpr int WPR = GROUP / 32;                   // warps per row
  const int warp = threadIdx.x >> 5;
  if ((threadIdx.x & 31) == 0) {
#pragma unroll
    for (int k = 0; k < NVAL; ++k) sm[k * 8 + warp] = x[k];
  }
  __syncthreads();
  const int first = (warp / WPR) * WPR;
#pragma unroll
  for (int k = 0; k < NVAL; ++k) {
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < WPR; ++i) s += sm[k * 8 + first + i];   // same order in every thread of the row
    x[k] = s;
  }
}

// KIND 0 = MSE, 1 = cosine. GROUP threads per row, 256 / GROUP rows per block pass, up to NV 16-byte
// vectors per thread held in registers; vectors past GROUP * NV are re-read in the gradient pass.
template <int KIND, int GROUP, int NV>
__global__ void __launch_bounds__(256)
feature_rows_kernel(const uint4* __restrict__ S, const uint4* __restrict__ R, const uint8_t* __restrict__ mask,
                    long long T, int nvec /* H / 8 */, const FeatHeader* __restrict__ hdr, FeatHeader direct,
                    int accumulate, float* __restrict__ loss_tok, uint4* __restrict__ dS) {
  __shared__ float sm[2][3 * 8];
  constexpr int ROWS = 256 / GROUP;
  int parity = 0;
  const int lane = threadIdx.x % GROUP;
  const int sub = threadIdx.x / GROUP;
  const float g = hdr ? hdr->g : direct.g;        // without a mask N = T is known on the host
  const float inv_h = 1.f / (8.f * (float)nvec);
  for (long long row0 = (long long)blockIdx.x * ROWS; row0 < T; row0 += (long long)gridDim.x * ROWS) {
    const long long t = row0 + sub;
    const bool live = t < T;
    const bool counted = live && (mask == nullptr || mask[t] != 0);
    const uint4* s_row = S + (size_t)t * nvec;
    const uint4* r_row = R + (size_t)t * nvec;
    uint4 sv[NV], rv[NV];
    float a0 = 0.f, a1 = 0.f, a2 = 0.f;           // MSE: a0 = sum (s-r)^2.  cosine: <s,r>, |s|^2, |r|^2
    if (counted) {
#pragma unroll
      for (int i = 0; i < NV; ++i) {
        const int v = lane + i * GROUP;
        if (v < nvec) { sv[i] = __ldg(s_row + v); rv[i] = __ldg(r_row + v); }
      }
#pragma unroll
      for (int i = 0; i < NV; ++i) {
        const int v = lane + i * GROUP;
        if (v < nvec) {
          float x[8], y[8];
          unpack8(sv[i], x); unpack8(rv[i], y);
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            if (KIND == 0) { const float d = x[j] - y[j]; a0 = fmaf(d, d, a0); }
            else { a0 = fmaf(x[j], y[j], a0); a1 = fmaf(x[j], x[j], a1); a2 = fmaf(y[j], y[j], a2); }
          }
        }
      }
      for (int v = lane + NV * GROUP; v < nvec; v += GROUP) {
        float x[8], y[8];
        unpack8(s_row[v], x); unpack8(r_row[v], y);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          if (KIND == 0) { const float d = x[j] - y[j]; a0 = fmaf(d, d, a0); }
          else { a0 = fmaf(x[j], y[j], a0); a1 = fmaf(x[j], x[j], a1); a2 = fmaf(y[j], y[j], a2); }
        }
      }
    }
    {
      float acc[3] = {a0, a1, a2};
      group_sum<GROUP, KIND == 0 ? 1 : 3>(acc, sm[parity]);
      parity ^= 1;
      a0 = acc[0]; a1 = acc[1]; a2 = acc[2];
    }

    // row scalars: f_t and the two gradient coefficients, d s = cs * s + cr * r
    float f = 0.f, cs = 0.f, cr = 0.f;
    if (counted) {
      if (KIND == 0) {
        f = a0 * inv_h;
        cs = 2.f * g * inv_h; cr = -cs;
      } else {
        const float nn = sqrtf(a1) * sqrtf(a2);
        if (nn > 1e-12f) {
          const float c = a0 / nn;
          f = 1.f - c;
          cr = -g / nn;
          cs = g * c / a1;
        } else {
          f = 1.f;
        }
      }
    }
    if (live && lane == 0 && loss_tok) loss_tok[t] = f;
    if (dS == nullptr || !live) continue;
    uint4* d_row = dS + (size_t)t * nvec;
    if (!counted) {
      if (!accumulate)
        for (int v = lane; v < nvec; v += GROUP) d_row[v] = make_uint4(0u, 0u, 0u, 0u);
      continue;
    }
#pragma unroll
    for (int i = 0; i < NV; ++i) {
      const int v = lane + i * GROUP;
      if (v < nvec) {
        float x[8], y[8], o[8];
        unpack8(sv[i], x); unpack8(rv[i], y);
        if (accumulate) unpack8(d_row[v], o);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const float d = KIND == 0 ? cs * (x[j] - y[j]) : fmaf(cs, x[j], cr * y[j]);
          o[j] = accumulate ? o[j] + d : d;
        }
        d_row[v] = pack8(o);
      }
    }
    for (int v = lane + NV * GROUP; v < nvec; v += GROUP) {
      float x[8], y[8], o[8];
      unpack8(s_row[v], x); unpack8(r_row[v], y);
      if (accumulate) unpack8(d_row[v], o);
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const float d = KIND == 0 ? cs * (x[j] - y[j]) : fmaf(cs, x[j], cr * y[j]);
        o[j] = accumulate ? o[j] + d : d;
      }
      d_row[v] = pack8(o);
    }
  }
}

// loss = loss_scale * sum_t f_t in a fixed order (double accumulators, one block): bitwise reproducible.
__global__ void __launch_bounds__(1024)
feature_reduce_kernel(const float* __restrict__ loss_tok, long long T, const FeatHeader* __restrict__ hdr,
                      FeatHeader direct, float* __restrict__ loss_out) {
  __shared__ double part[32];
  double acc = 0.0;
  for (long long t = threadIdx.x; t < T; t += 1024) acc += (double)loss_tok[t];
  for (int o = 16; o; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    double s = 0.0;
    for (int i = 0; i < 32; ++i) s += part[i];
    *loss_out = (float)(s * (double)(hdr ? hdr->loss_scale : direct.loss_scale));
  }
}

// Host side: pick the instantiation that holds ceil(nvec / GROUP) vectors per thread in registers.
template <int KIND, int GROUP>
static inline void launch_feature_rows(int nv, int grid, cudaStream_t st, const uint4* S, const uint4* R,
                                       const uint8_t* mask, long long T, int nvec, const FeatHeader* hdr,
                                       FeatHeader direct, int acc, float* tok, uint4* dS) {
#define KDKL_FEAT_LAUNCH(NV_) \
  feature_rows_kernel<KIND, GROUP, NV_><<<grid, 256, 0, st>>>(S, R, mask, T, nvec, hdr, direct, acc, tok, dS)
  if (nv <= 1)      KDKL_FEAT_LAUNCH(1);
  else if (nv <= 2) KDKL_FEAT_LAUNCH(2);
  else if (nv <= 4) KDKL_FEAT_LAUNCH(4);
  else              KDKL_FEAT_LAUNCH(8);
#undef KDKL_FEAT_LAUNCH
}

}  // namespace kdkl
