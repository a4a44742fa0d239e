// Persistent, warp-specialised bf16 GEMM for sm_100a: D[M,N] = A[M,K] * B[N,K]^T with fp32
// accumulation in tensor memory, operands staged by TMA into 128-byte-swizzled shared memory.
//
//   warp 0      TMA producer (one lane): fills a ring of STAGES shared-memory stages
//   warp 1      allocates TMEM; one lane issues tcgen05.mma and commits to mbarriers
//   warps 2..5  epilogue: tcgen05.ld gives each thread one accumulator row (32 columns at
//               a time); two TMEM accumulator stages let tile i's epilogue overlap tile
//               i+1's MMAs
//
// One CTA per SM; tiles of 128 x 256 per CTA (256 x 256 per CTA pair, see GemmCfg), k-blocks of 64. WIDE tiles
// (256 x 512 per pair) use both TMEM halves as one accumulator: a quarter less operand traffic per flop, no
// overlap of a tile's epilogue with the next tile's MMAs (for the two output GEMMs, whose epilogues are short).
// Either operand may be K-major (its rows are contiguous along K) or MN-major (stored
// [K, M] / [K, N], contiguous along M / N); the difference is confined to the TMA boxes
// and the shared-memory descriptors.
//
// Epilogues (the fused parts of the loss):
// Output tiles leave through swizzled shared-memory boxes and TMA store / reduce-add.
//   EPI_STORE_F32   plain fp32 store or += (dWeight accumulation, Algorithm 1 "dW += G^T h")
//   EPI_STORE_BF16  bf16 store (dHidden, Algorithm 1 "dh = G W")
//   EPI_LSE         forward: per (row, vocab tile) online max / sum-exp of z/tau and gather of
//                   z at the teacher's indices; logits never leave the SM (Algorithm 1,
//                   forward passes 1 and 2 in one sweep; Eq. "decomp")
//   EPI_DLOGITS     backward: G = a_t * exp(z/tau - logZ) - b_t * p at the support, cast to
//                   bf16 (Eq. "grad", Algorithm 1 backward)
//   EPI_TOPK        teacher cache: emits the (column, logit) pairs above a per-row threshold
//   EPI_LSE_Z       EPI_LSE that also stores the fp32 logits (teacher cache with one projection: the selection then
//                   reads them back instead of projecting again)
//   EPI_LSE_E       EPI_LSE that also stores the unnormalised exponentials 2^(z log2e / tau - 64) in bf16, for the
//                   single-pass forward + backward (no second projection: G is made from them once log Z is known)
#pragma once
#include <cuda_bf16.h>

#include "sm100_prims.cuh"

namespace kdkl {

constexpr int BM = 128, BN = 256, BK = 64;   // per-CTA accumulator: 128 TMEM lanes x 256 fp32 columns
constexpr int UMMA_K = 16;
constexpr int GEMM_THREADS = 192;
constexpr int MAX_LIVE_KB = 128;               // k-block skipping: 32 row-tile flags = at most 8192 tokens = 128 k-blocks
constexpr int MAX_LIVE_M = 256;                // row-tile skipping for launches of up to 256 row tiles
constexpr int TMEM_COLS = 512;
constexpr int STAGING_WARP_BYTES = 2 * 4096;   // per epilogue warp: two 32-row x 128-byte output boxes
constexpr int STAGING_BYTES = 4 * STAGING_WARP_BYTES;

// NCTA = 1: one CTA per 128 x 256 tile. NCTA = 2: a pair of CTAs (cluster of two, cta_group::2)
// shares one 256 x 256 tile: each CTA stages its 128 rows of A and its 128 rows of B, the leader
// issues one MMA for both, and each CTA keeps the 128 x 256 half of D in its own TMEM. A pair
// moves a third less operand data per flop through shared memory and L2.
// WIDE: the tile is 512 columns wide - two 256-column halves, each fed by its own MMA per K = 16 slice from the same
// A operand, together filling all 512 TMEM columns. Per flop a quarter less operand data comes through L2 and
// shared memory than with two 256 x 256 tiles, which is what the two output GEMMs need: dH = G W streams both
// operands from HBM once per wave of tiles (half the waves now), and in dW += G^T h every stored byte takes
// load bandwidth from the SM's memory port. The price: one accumulator stage, so the epilogue does not overlap
// the next tile's MMAs - acceptable where a tile's contraction is long next to its epilogue.
template <int NCTA, bool WIDE = false>
struct GemmCfg {
  static constexpr int TILE_M = BM * NCTA;
  static constexpr int N_HALVES = WIDE ? 2 : 1;
  static constexpr int TILE_N = BN * N_HALVES;
  static constexpr int B_ROWS = TILE_N / NCTA;           // rows of B each CTA stages (HALF_ROWS per accumulator half)
  static constexpr int A_STAGE_BYTES = BM * BK * 2;      // 16 KiB
  static constexpr int B_STAGE_BYTES = B_ROWS * BK * 2;  // 32 / 16 KiB
  static constexpr int STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;
  static constexpr int STAGES = 4;   // measured: 3 starves the tensor pipe, 5 and 6 are no faster than 4
  static constexpr int SMEM_BYTES = STAGES * STAGE_BYTES + STAGING_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/ +
                                    2 * MAX_LIVE_KB /*live k-block list*/ + 2 * MAX_LIVE_M /*live row-tile list*/;
};

enum { EPI_STORE_F32 = 0, EPI_STORE_BF16 = 1, EPI_LSE = 2, EPI_DLOGITS = 3, EPI_TOPK = 4, EPI_LSE_E = 5, EPI_LSE_Z = 6 };

// EPI_LSE_E stores e = 2^(z log2e / tau - kExpBias) in bf16: representable for scaled logits in about
// [-62, 190] (bf16 has fp32's exponent range), i.e. far below any weight that matters and far above any sane logit.
constexpr float kExpBias = 64.f;

struct GemmParams {
  int M, N, K;               // valid extents of this launch
  int m_tiles, n_tiles;      // tiles of TILE_M rows and of TILE_N columns (256, or 512 for the WIDE instantiation)
  int m_inner;               // 1: consecutive tile ids walk M first (B panel shared), 0: N first
  int m_group;               // m_inner only, 0 = all: row tiles per group. Tiles walk group by group (all column
                             // tiles of one group of row tiles before the next group), so that the A rows in use
                             // at any time are one group's (sized by the host to stay resident in L2) while B is
                             // streamed once per group
  int k_splits;              // >= 1: each tile's contraction is cut into this many work units, each
                             // writing its own partial output (split s goes to output rows + s * split_rows)
  int split_rows;
  int* status;               // device status word pair {code, where}
  const int* go;             // optional: kernel returns at once when *go == 0
  // Skipping work for ignored tokens (both optional, one flag per TILE_M rows, 0 = every token of
  // that row tile is ignored). m_live [m_tiles] (m_tiles <= MAX_LIVE_M): a dead row tile of D is not
  // computed - LSE / TOPK write nothing for it, the store epilogues write zeros (nothing when
  // accumulating); the work units are numbered over the live tiles only, so the workers stay balanced. k_live
  // [ceil(K / TILE_M)] (at most 32 flags, k_splits must be 1): dead k-blocks of the contraction are not
  // loaded or multiplied (their A columns are zeros by construction); if all are dead the first one is
  // processed, so that the accumulator is defined.
  const uint8_t* m_live;
  const uint8_t* k_live;
  // EPI_STORE_F32: 1 -> output += D (TMA reduce-add), 0 -> output = D. Outputs go through tmC.
  int accumulate;
  // EPI_LSE / EPI_DLOGITS: all row-indexed pointers are already offset to this chunk's row 0
  float scale_log2;          // log2(e) / tau
  int Ktop;                  // teacher slots per row
  const int* idx_sorted;     // [rows, Ktop] ascending, first nvalid[row] entries valid
  const int* nvalid;         // [rows]
  float* part_m;             // [n_tiles, part_stride] running max (log2 domain)
  float* part_s;             // [n_tiles, part_stride] sum of 2^(s - max)
  long long part_stride;
  float* zg;                 // [rows, Ktop] gathered logits, sorted order
  int* colread;              // [rows, Ktop] column actually read, sorted order
  const float* lz2;          // [rows] log2-domain log-normaliser
  const int* neg_a;          // device flag: 1 when the upstream gradient is negative (coefA <= 0 for every row)
  long long row_base;        // token index of row 0 of this launch (for error reports)
  const float* coefA;        // [rows] g_t * M_t / tau (EPI_DLOGITS; EPI_LSE_E, optional: rows with 0 store zeros)
  const float* coefB;        // [rows] g_t / tau
  const float* p_sorted;     // [rows, Ktop]
  // EPI_TOPK: every logit with z * scale_log2 >= thr[row] is appended to the row's candidate list
  const float* thr;          // [rows] threshold in the scaled (log2) domain
  int* cand_cnt;             // [rows] running count (may exceed cand_cap: overflow is detected later)
  int* cand_idx;             // [rows, cand_cap]
  float* cand_val;           // [rows, cand_cap] raw logits
  int cand_cap;
};

__device__ __forceinline__ int lower_bound_i32(const int* a, int n, int key) {
  int lo = 0, hi = n;
  while (lo < hi) {
    const int mid = (lo + hi) >> 1;
    if (a[mid] < key) lo = mid + 1; else hi = mid;
  }
  return lo;
}

__device__ __forceinline__ float sel32(const uint32_t (&r)[32], int off) {
  float v = 0.f;
#pragma unroll
  for (int j = 0; j < 32; ++j) v = (off == j) ? __uint_as_float(r[j]) : v;
  return v;
}

// 2^x by the special-function unit (relative error about 2^-22; 2^-inf = 0)
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

__device__ __forceinline__ int kblocks_all(int K) { return (K + BK - 1) / BK; }

template <int EPI, bool A_MN, bool B_MN, int NCTA, bool WIDE = false>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_tcgen05_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                    const __grid_constant__ CUtensorMap tmC, const GemmParams p) {
  using Cfg = GemmCfg<NCTA, WIDE>;
  constexpr int STAGES = Cfg::STAGES, STAGE_BYTES = Cfg::STAGE_BYTES, A_STAGE_BYTES = Cfg::A_STAGE_BYTES;
  constexpr int TILE_M = Cfg::TILE_M, B_ROWS = Cfg::B_ROWS, TILE_N = Cfg::TILE_N, N_HALVES = Cfg::N_HALVES;
  constexpr int HALF_ROWS = B_ROWS / N_HALVES;            // rows of B this CTA stages per accumulator half
  constexpr uint32_t HALF_BYTES = HALF_ROWS * BK * 2;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_al = smem_raw + (smem_base - smem_u32(smem_raw));
  // after the stage ring: the epilogue's output staging boxes, then barriers and bookkeeping
  const uint32_t staging0 = smem_base + STAGES * STAGE_BYTES;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem_al + STAGES * STAGE_BYTES + STAGING_BYTES);
  const uint32_t bar0 = staging0 + STAGING_BYTES;
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES + s); };
  auto tfull_bar = [&](int a) { return bar0 + 8u * (2 * STAGES + a); };
  auto tempty_bar = [&](int a) { return bar0 + 8u * (2 * STAGES + 2 + a); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (p.go != nullptr && *p.go == 0) return;   // uniform across the grid

  // pair bookkeeping: the leader (cluster rank 0) owns the barriers that gate the MMAs
  const uint32_t cta_rank = NCTA == 2 ? cluster_ctarank() : 0u;
  const bool leader = cta_rank == 0u;
  const int worker = blockIdx.x / NCTA, num_workers = gridDim.x / NCTA;
  auto leader_bar = [&](uint32_t bar) { return NCTA == 2 ? map_to_cta(bar, 0u) : bar; };

  if (threadIdx.x == 0) {
    // full (used in the leader): one arrival, the leader's producer announcing the bytes of both CTAs'
    // loads; tempty (leader): one arrival per epilogue warp of the pair
    for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 4 * NCTA); }
    *abort_flag = 0;
    mbar_fence_init();
    tma_prefetch_desc(&tmA);
    tma_prefetch_desc(&tmB);
    if (EPI != EPI_LSE && EPI != EPI_TOPK) tma_prefetch_desc(&tmC);
  }
  if (warp == 1) {
    if (NCTA == 2) { tmem_alloc_pair(smem_u32(tmem_slot), TMEM_COLS); tmem_relinquish_pair(); }
    else           { tmem_alloc(smem_u32(tmem_slot), TMEM_COLS); tmem_relinquish(); }
  }
  // Dead k-blocks: one warp turns the row-tile flags into the ascending list of live k-blocks in shared
  // memory, once per kernel. The two single-thread loops below then run over that list with exactly
  // the loop shape of the unskipped case (a test per k-block inside those loops costs whole percents
  // of the kernel even when it is never taken).
  const bool kskip = p.k_live != nullptr;
  uint16_t* live_kb = reinterpret_cast<uint16_t*>(smem_al + STAGES * STAGE_BYTES + STAGING_BYTES + 256);
  volatile int* n_live_kb = reinterpret_cast<volatile int*>(tmem_slot + 2);
  if (kskip && warp == 2) {
    const int nkt = (p.K + TILE_M - 1) / TILE_M;
    const uint32_t live_tiles = __ballot_sync(0xffffffffu, lane < nkt && p.k_live[lane] != 0);
    if (lane == 0) {
      int n = 0;
      for (int kb = 0; kb < kblocks_all(p.K); ++kb)
        if ((live_tiles >> ((kb * BK) / TILE_M)) & 1u) live_kb[n++] = (uint16_t)kb;
      if (n == 0) live_kb[n++] = 0;
      *n_live_kb = n;
    }
  }
  // Dead row tiles: another warp writes the live row tiles (ascending) to the front of a list and the
  // dead ones to its back. Units are then numbered over the live tiles only - with the static
  // round-robin assignment, skipping dead units in place would leave some workers with twice the work.
  const bool mskip = p.m_live != nullptr;
  uint16_t* live_m = live_kb + MAX_LIVE_KB;
  volatile int* n_live_m = reinterpret_cast<volatile int*>(tmem_slot + 3);
  if (mskip && warp == 3) {
    int n = 0, nd = 0;
    for (int base = 0; base < p.m_tiles; base += 32) {
      const int t = base + lane;
      const uint32_t bits = __ballot_sync(0xffffffffu, t < p.m_tiles && p.m_live[t] != 0);
      if (lane == 0) {
        for (int j = 0; j < 32 && base + j < p.m_tiles; ++j) {
          if ((bits >> j) & 1u) live_m[n++] = (uint16_t)(base + j);
          else live_m[p.m_tiles - 1 - nd++] = (uint16_t)(base + j);
        }
      }
    }
    if (lane == 0) *n_live_m = n;
  }
  tc_fence_before();
  __syncthreads();
  if (NCTA == 2) cluster_sync_all();   // the peer's barriers exist before anything arrives on them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  const int m_count = mskip ? *n_live_m : p.m_tiles;      // row tiles that are computed
  const int num_tiles = m_count * p.n_tiles;
  const int kblocks = (p.K + BK - 1) / BK;
  // work units: unit u = split * num_tiles + tile; a unit contracts k-blocks [kb0, kb1)
  const int num_units = num_tiles * p.k_splits;
  const int kb_per_split = (kblocks + p.k_splits - 1) / p.k_splits;
  auto unit_decode = [&](int unit, int& tile, int& split, int& kb0, int& kb1) {
    split = unit / num_tiles;
    tile = unit - split * num_tiles;
    kb0 = split * kb_per_split;
    kb1 = kb0 + kb_per_split < kblocks ? kb0 + kb_per_split : kblocks;
  };

  auto tile_coords = [&](int tile, int& mt, int& nt) {
    if (p.m_inner) {
      const int gm = (p.m_group > 0 && p.m_group < m_count) ? p.m_group : m_count;
      const int g = tile / (gm * p.n_tiles);           // only the last group can be short
      const int r = tile - g * gm * p.n_tiles;
      const int m_here = m_count - g * gm < gm ? m_count - g * gm : gm;
      mt = g * gm + r % m_here; nt = r / m_here;
    } else { nt = tile % p.n_tiles; mt = tile / p.n_tiles; }
    if (mskip) mt = live_m[mt];
  };

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t it = 0, issued = 0, last_par = 0;
      bool ok = true;
      // a load lands in this CTA's stage and signals the full barrier of the pair's leader
      auto load = [&](uint32_t dst, const CUtensorMap* tm, int x, int y, uint32_t bar) {
        if (NCTA == 2) tma_load_2d_pair(dst, tm, x, y, bar); else tma_load_2d(dst, tm, x, y, bar);
      };
      for (int unit = worker; unit < num_units && ok; unit += num_workers) {
        int tile, split, kb0, kb1, mt, nt;
        unit_decode(unit, tile, split, kb0, kb1);
        tile_coords(tile, mt, nt);
        const int m0 = mt * TILE_M + (int)cta_rank * BM;      // this CTA's rows of A
        const int n0 = nt * TILE_N + (int)cta_rank * HALF_ROWS;   // this CTA's rows of B (of the first half)
        const int nkb = kskip ? *n_live_kb : kb1 - kb0;
        for (int i = 0; i < nkb; ++i, ++it) {
          const int kb = kskip ? (int)live_kb[i] : kb0 + i;
          const int s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1u;
          if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag, p.status, 1)) { ok = false; break; }
          const uint32_t sa = smem_base + s * STAGE_BYTES;
          const uint32_t sb = sa + A_STAGE_BYTES;
          const uint32_t fb = leader_bar(full_bar(s));
          // The peer's bytes may land before this announcement: the phase still cannot complete
          // before the leader's single arrival, and the peer reuses a stage only after the MMAs
          // that consumed it have been committed.
          if (leader) mbar_arrive_expect_tx(full_bar(s), NCTA * STAGE_BYTES);
          const int k0 = kb * BK;
          if (!A_MN) {
            load(sa, &tmA, k0, m0, fb);
          } else {
#pragma unroll
            for (int i = 0; i < BM / 64; ++i) load(sa + i * (BK * 128), &tmA, m0 + 64 * i, k0, fb);
          }
#pragma unroll
          for (int hf = 0; hf < N_HALVES; ++hf) {         // half hf of the tile: columns [nt * TILE_N + hf * BN, + BN)
            const uint32_t sbh = sb + hf * HALF_BYTES;
            const int nh = n0 + hf * BN;
            if (!B_MN) {
              load(sbh, &tmB, k0, nh, fb);
            } else {
#pragma unroll
              for (int i = 0; i < HALF_ROWS / 64; ++i) load(sbh + i * (BK * 128), &tmB, nh + 64 * i, k0, fb);
            }
          }
          issued |= 1u << s;
          last_par = (last_par & ~(1u << s)) | (ph << s);
        }
      }
      if (!ok) {
        // aborted: give the copies still in flight a bounded time to land before the CTA exits
        if (NCTA == 1) {
          for (int s = 0; s < STAGES; ++s) {
            if (!((issued >> s) & 1u)) continue;
            const uint64_t t0 = globaltimer_ns();
            while (!mbar_try_wait(full_bar(s), (last_par >> s) & 1u) && globaltimer_ns() - t0 < 2000000ull) {}
          }
        } else {
          const uint64_t t0 = globaltimer_ns();   // the barrier may be the peer's: a bounded pause instead
          while (globaltimer_ns() - t0 < 2000000ull) {}
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (the leader's, for the pair)
    if (lane == 0 && leader) {
      const uint32_t idesc = make_idesc_bf16(TILE_M, BN, A_MN ? 1u : 0u, B_MN ? 1u : 0u);
      auto mma = [&](uint32_t d, uint64_t ad, uint64_t bd, uint32_t accf) {
        if (NCTA == 2) umma_bf16_pair(d, ad, bd, idesc, accf); else umma_bf16(d, ad, bd, idesc, accf);
      };
      auto commit = [&](uint32_t bar) { if (NCTA == 2) umma_commit_pair(bar); else umma_commit(bar); };
      // This single thread feeds the tensor pipe: every instruction here is on the critical path, so the
      // shared-memory descriptors are not rebuilt per instruction. Their upper words and the layout bits
      // of the lower words are constants; the 14-bit address field advances by STAGE_BYTES / 16 per
      // stage and by a fixed step per K = 16 slice (all addresses stay below 256 KiB: no carry).
      constexpr uint32_t A_LBO = A_MN ? BK * 128 : 0, B_LBO = B_MN ? BK * 128 : 0;
      constexpr uint32_t A_STEP = (A_MN ? UMMA_K * 128 : UMMA_K * 2) >> 4;
      constexpr uint32_t B_STEP = (B_MN ? UMMA_K * 128 : UMMA_K * 2) >> 4;
      constexpr uint32_t STAGE_STEP = STAGE_BYTES >> 4;
      const uint64_t a_proto = make_smem_desc(smem_base, A_LBO, 1024);
      const uint64_t b_proto = make_smem_desc(smem_base + A_STAGE_BYTES, B_LBO, 1024);
      const uint32_t a_hi = (uint32_t)(a_proto >> 32), a_lo0 = (uint32_t)a_proto;
      const uint32_t b_hi = (uint32_t)(b_proto >> 32), b_lo0 = (uint32_t)b_proto;
      auto desc = [](uint32_t lo, uint32_t hi) { return (static_cast<uint64_t>(hi) << 32) | lo; };
      uint32_t it = 0, lt = 0;
      bool ok = true;
      for (int unit = worker; unit < num_units && ok; unit += num_workers) {
        int tile, split, kb0, kb1, mt, nt;
        unit_decode(unit, tile, split, kb0, kb1);
        tile_coords(tile, mt, nt);
        const uint32_t acc = WIDE ? 0u : (lt & 1u);       // WIDE: one accumulator stage (all 512 columns)
        const uint32_t aph = WIDE ? (lt & 1u) : ((lt >> 1) & 1u);
        if (!mbar_wait(tempty_bar(acc), aph ^ 1u, abort_flag, p.status, 2)) { ok = false; break; }
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + acc * BN;
        uint32_t accf = 0u;                    // the unit's first MMA overwrites the accumulator
        const int nkb = kskip ? *n_live_kb : kb1 - kb0;
        for (int i = 0; i < nkb; ++i, ++it) {
          const uint32_t s = it % STAGES;
          const uint32_t ph = (it / STAGES) & 1u;
          if (!mbar_wait(full_bar(s), ph, abort_flag, p.status, 3)) { ok = false; break; }
          tc_fence_after();
          const uint32_t alo = a_lo0 + s * STAGE_STEP, blo = b_lo0 + s * STAGE_STEP;
#pragma unroll
          for (int j = 0; j < BK / UMMA_K; ++j) {
#pragma unroll
            for (int hf = 0; hf < N_HALVES; ++hf)
              mma(tmem_d + hf * BN, desc(alo + j * A_STEP, a_hi), desc(blo + hf * (HALF_BYTES >> 4) + j * B_STEP, b_hi),
                  accf);
            accf = 1u;
          }
          commit(empty_bar(s));                // frees the stage (in both CTAs) when these MMAs have read it
        }
        if (ok) commit(tfull_bar(acc));        // accumulator complete (signalled in both CTAs)
        ++lt;
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 2..5)
    const int lg = warp & 3;                   // TMEM lane group this warp may read
    const int row_in_tile = lg * 32 + lane;
    constexpr bool kBf16Out = (EPI == EPI_STORE_BF16 || EPI == EPI_DLOGITS || EPI == EPI_LSE_E);
    constexpr bool kLse = (EPI == EPI_LSE || EPI == EPI_LSE_E || EPI == EPI_LSE_Z);
    constexpr bool kStore = (EPI == EPI_STORE_F32 || EPI == EPI_LSE_Z || kBf16Out);
    uint32_t lt = 0, nbox = 0;
    bool ok = true;
    // Dead row tiles (every token ignored) belong to no work unit. LSE / TOPK have nothing to write for
    // them; a store epilogue writes their part of the output as zeros (nothing when it would add them),
    // for every split's slab, before it turns to the computed tiles.
    if (mskip && kStore && !(EPI == EPI_STORE_F32 && p.accumulate)) {
      const int n_dead = p.m_tiles - m_count;
      const int zero_units = n_dead * p.n_tiles * p.k_splits;
      constexpr int BOX_COLS = kBf16Out ? 64 : 32;
      for (int zu = worker; zu < zero_units; zu += num_workers) {
        const int split = zu / (n_dead * p.n_tiles);
        const int rem = zu - split * (n_dead * p.n_tiles);
        const int mt = live_m[m_count + rem / p.n_tiles], nt = rem % p.n_tiles;
        const int r0 = mt * TILE_M + (int)cta_rank * BM + lg * 32, n0 = nt * TILE_N;
        if (r0 >= p.M) continue;
        // zero boxes through the same staging / bulk-group protocol as the regular output path
        for (int c0 = n0; c0 < n0 + TILE_N && c0 < p.N; c0 += BOX_COLS) {
          const uint32_t sbox = staging0 + (warp - 2) * STAGING_WARP_BYTES + (nbox & 1u) * 4096u;
          if (lane == 0) bulk_wait_read<1>();
          __syncwarp();
#pragma unroll
          for (int c = 0; c < 8; ++c) st_shared_v4(sbox + lane * 128 + (c << 4), 0u, 0u, 0u, 0u);
          fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) {
            tma_store_2d(&tmC, sbox, c0, r0 + split * p.split_rows);
            bulk_commit();
          }
          ++nbox;
        }
      }
    }
    for (int unit = worker; unit < num_units && ok; unit += num_workers) {
      int tile, split, kb0, kb1, mt, nt;
      unit_decode(unit, tile, split, kb0, kb1);
      tile_coords(tile, mt, nt);
      const int m0 = mt * TILE_M + (int)cta_rank * BM, n0 = nt * TILE_N;   // this CTA's 128 x TILE_N part of D
      const int row = m0 + row_in_tile;
      const bool row_ok = row < p.M;
      const uint32_t acc = WIDE ? 0u : (lt & 1u);
      const uint32_t aph = WIDE ? (lt & 1u) : ((lt >> 1) & 1u);

      // per-row state that does not need the accumulator: fetched before the wait
      int cur = 0, nv = 0, next_idx = 0x7fffffff;
      const int* idxrow = nullptr;
      float row_b = 0.f, row_off = -INFINITY, row_thr = INFINITY;
      bool row_zero = false;                   // EPI_LSE_E: a row without gradient stores zeros, not exponentials
      if (EPI == EPI_LSE_E) { if (row_ok && p.coefA != nullptr) row_zero = p.coefA[row] == 0.f; }
      if (EPI == EPI_TOPK) { if (row_ok) row_thr = p.thr[row]; }
      const bool neg_a = EPI == EPI_DLOGITS && p.neg_a != nullptr && *p.neg_a != 0;   // uniform over the call
      if (kLse || EPI == EPI_DLOGITS) {
        if (row_ok) {
          idxrow = p.idx_sorted + (long long)row * p.Ktop;
          nv = p.nvalid[row];
          cur = lower_bound_i32(idxrow, nv, n0);
          next_idx = cur < nv ? idxrow[cur] : 0x7fffffff;
          if (EPI == EPI_DLOGITS) {
            const float a = p.coefA[row];
            row_b = p.coefB[row];
            row_off = a != 0.f ? log2f(fabsf(a)) - p.lz2[row] : -INFINITY;   // sign: see neg_a
          }
        }
      }

      // the decision to go on is taken by the whole warp: tcgen05.ld below is warp-collective
      const bool arrived = mbar_wait(tfull_bar(acc), aph, abort_flag, p.status, 4);
      if (!__all_sync(0xffffffffu, arrived)) { ok = false; break; }
      tc_fence_after();
      const uint32_t taddr = tmem_base + (uint32_t(lg * 32) << 16) + acc * BN;

      float m_run = -INFINITY, s_run = 0.f;
      const int box_row0 = m0 + lg * 32;       // first output row of this warp's boxes
      const bool box_ok = box_row0 < p.M;      // warp-uniform
#pragma unroll 1
      for (int w = 0; w < TILE_N / 32; ++w) {
        const int col0 = n0 + w * 32;
        // uniform: whole window past the edge. bf16 outputs are staged as pairs of windows
        // (64 columns = one 128-byte row), so a pair is always completed.
        if (col0 >= p.N && (!kBf16Out || (w & 1) == 0)) break;
        uint32_t r[32];
        __syncwarp();
        tmem_ld32(taddr + w * 32, r);
        tmem_ld_wait();
        const bool full_w = col0 + 32 <= p.N;
        float e_fac = 0.f;                     // EPI_LSE_E: 2^(running maximum - bias) of this row and window

        if (kLse) {
          if (row_ok) {
            // gather the student logit at every teacher index that falls in this window
            while (next_idx < col0 + 32) {
              const float zsel = sel32(r, next_idx - col0);
              p.zg[(long long)row * p.Ktop + cur] = zsel;
              p.colread[(long long)row * p.Ktop + cur] = next_idx;
              ++cur;
              next_idx = cur < nv ? idxrow[cur] : 0x7fffffff;
            }
            // online max / sum-exp in the log2 domain: max on the raw logits (the scale is positive),
            // then one FFMA + ex2 + add per element
            float wmax = -INFINITY;
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              if (!full_w && col0 + j >= p.N) r[j] = 0xff800000u;   // -inf: columns past the vocabulary
              wmax = fmaxf(wmax, __uint_as_float(r[j]));
            }
            const float m_new = fmaxf(m_run, wmax * p.scale_log2);
            float acc_s = 0.f;
            if (EPI == EPI_LSE_E) {
              // keep the window's exponentials (relative to the running maximum) in place of the logits:
              // e = 2^(s - bias) = 2^(s - m_new) * 2^(m_new - bias), one multiply instead of a second ex2
#pragma unroll
              for (int j = 0; j < 32; ++j) {
                const float tj = ex2_approx(fmaf(__uint_as_float(r[j]), p.scale_log2, -m_new));
                acc_s += tj;
                r[j] = __float_as_uint(tj);
              }
              e_fac = row_zero ? 0.f : ex2_approx(m_new - kExpBias);
              // bf16 tops out just below 2^128: a scaled logit beyond bias + 128 cannot be stored
              if (m_new - kExpBias >= 128.f && !row_zero && p.status != nullptr) {
                atomicCAS(p.status, 0, -11);               // KDKL_ERR_NONFINITE, with the token
                atomicCAS(p.status + 1, 0, (int)(p.row_base + row));
              }
            } else {
#pragma unroll
              for (int j = 0; j < 32; ++j) acc_s += ex2_approx(fmaf(__uint_as_float(r[j]), p.scale_log2, -m_new));
            }
            s_run = s_run * ex2_approx(m_run - m_new) + acc_s;
            m_run = m_new;
          }
        }
        if (EPI == EPI_TOPK) {
          if (row_ok) {
            // candidates of this window: a bit per column whose scaled logit reaches the row's threshold
            uint32_t hits = 0u;
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              const bool in = (full_w || col0 + j < p.N) && (__uint_as_float(r[j]) * p.scale_log2 >= row_thr);
              hits |= (in ? 1u : 0u) << j;
            }
            while (hits) {
              const int j = __ffs(hits) - 1;
              hits &= hits - 1u;
              const int arrival = atomicAdd(p.cand_cnt + row, 1);  // tiles of one row run on different SMs
              const int slot = reservoir_slot(arrival, p.cand_cap, (uint32_t)row, (uint32_t)(col0 + j));
              if (slot >= 0) {
                p.cand_idx[(long long)row * p.cand_cap + slot] = col0 + j;
                p.cand_val[(long long)row * p.cand_cap + slot] = sel32(r, j);
              }
            }
          }
        }
        if (kStore) {
          // Output path: the warp's 32 rows x 128 bytes go to a swizzled shared-memory box (16-byte
          // chunk c of row i sits at chunk c ^ (i & 7), the layout a 128-byte-swizzle tensor map
          // expects) and leave with one TMA store / reduce-add; two boxes alternate.
          const uint32_t sbox = staging0 + (warp - 2) * STAGING_WARP_BYTES + (nbox & 1u) * 4096u;
          const uint32_t srow = sbox + lane * 128;
          const bool first_half = !kBf16Out || (w & 1) == 0;
          if (first_half) {
            if (lane == 0) bulk_wait_read<1>();   // the store issued two boxes ago has read this box
            __syncwarp();
          }
          if (!kBf16Out) {                     // fp32 boxes: EPI_STORE_F32, EPI_LSE_Z
#pragma unroll
            for (int c = 0; c < 8; ++c)
              st_shared_v4(srow + ((c ^ (lane & 7)) << 4), r[4 * c], r[4 * c + 1], r[4 * c + 2], r[4 * c + 3]);
          } else {
            uint32_t v[16];
            if (EPI == EPI_STORE_BF16) {
#pragma unroll
              for (int j = 0; j < 16; ++j) v[j] = pack_bf16x2(__uint_as_float(r[2 * j]), __uint_as_float(r[2 * j + 1]));
            } else if (EPI == EPI_LSE_E) {
              // unnormalised exponentials with a fixed bias: G = A_t * e - b_t p is formed from them later
#pragma unroll
              for (int j = 0; j < 16; ++j)
                v[j] = pack_bf16x2(__uint_as_float(r[2 * j]) * e_fac, __uint_as_float(r[2 * j + 1]) * e_fac);
            } else {  // EPI_DLOGITS
              // a_t * 2^(s - lz2) = 2^(s + (log2 a_t - lz2)): the row coefficient rides in the exponent
              // (a_t = 0 for ignored tokens gives -inf, hence exact zeros)
              float g[32];
#pragma unroll
              for (int j = 0; j < 32; ++j) g[j] = ex2_approx(fmaf(__uint_as_float(r[j]), p.scale_log2, row_off));
              if (neg_a) {                     // the whole call has a negative upstream gradient
#pragma unroll
                for (int j = 0; j < 32; ++j) g[j] = -g[j];
              }
              while (next_idx < col0 + 32) {
                const int off = next_idx - col0;
                const float bp = row_b * p.p_sorted[(long long)row * p.Ktop + cur];
#pragma unroll
                for (int j = 0; j < 32; ++j) g[j] -= (off == j) ? bp : 0.f;
                ++cur;
                next_idx = cur < nv ? idxrow[cur] : 0x7fffffff;
              }
#pragma unroll
              for (int j = 0; j < 16; ++j) v[j] = pack_bf16x2(g[2 * j], g[2 * j + 1]);
            }
            const int cbase = (w & 1) * 4;
#pragma unroll
            for (int c = 0; c < 4; ++c)
              st_shared_v4(srow + (((cbase + c) ^ (lane & 7)) << 4), v[4 * c], v[4 * c + 1], v[4 * c + 2], v[4 * c + 3]);
          }
          if (!kBf16Out || (w & 1) == 1) {
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0 && box_ok) {
              const int cx = kBf16Out ? col0 - 32 : col0;
              const int cy = box_row0 + split * p.split_rows;
              if (EPI == EPI_STORE_F32 && p.accumulate) tma_reduce_add_2d(&tmC, sbox, cx, cy);
              else tma_store_2d(&tmC, sbox, cx, cy);
            }
            if (lane == 0) bulk_commit();
            ++nbox;
          }
        }
      }
      // accumulator stage is free again
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if (NCTA == 2) mbar_arrive_cluster(leader_bar(tempty_bar(acc))); else mbar_arrive(tempty_bar(acc));
      }
      ++lt;

      if (kLse) {
        if (row_ok) {
          p.part_m[(long long)nt * p.part_stride + row] = m_run;
          p.part_s[(long long)nt * p.part_stride + row] = s_run;
        }
      }
    }
    if (EPI != EPI_LSE && EPI != EPI_TOPK && lane == 0) bulk_wait_all();   // every output box has been written
  }

  // ---------------------------------------------------------------- teardown
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  if (NCTA == 2) cluster_sync_all();   // neither CTA leaves while the other may still reach its barriers
  tc_fence_after();
  if (warp == 1) {
    if (NCTA == 2) tmem_dealloc_pair(tmem_base, TMEM_COLS); else tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

}  // namespace kdkl
