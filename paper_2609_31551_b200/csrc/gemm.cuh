// Persistent bf16 GEMM for sm_100a:  D[M,N] = A[M,K] * W[N,K]^T  with a fused epilogue.
//
//   warp 0, 10  TMA producers, one thread per operand (A tiles in warp 0, W tiles in warp 10) into a shared-memory ring
//   warp 1      UMMA issuer: tcgen05.mma (128x256x16, or 256x256x16 for a CTA pair), fp32 accumulators in TMEM, two
//               accumulator buffers (2 x 256 columns) so that the epilogue of tile i overlaps the main loop of tile i+1
//   warps 2..9  epilogue: tcgen05.ld -> bias / activation / rotary -> swizzled shared-memory staging -> TMA store
//               (TMA reduce-add into the fp32 residual stream); scatter epilogues (row maps) store directly
//
// Three tile shapes (template arguments CTAS, NW, KD; the launcher picks by estimated time): one CTA per 128x256 tile,
// a CTA pair (cta_group::2) per 256x256 tile with "deep" stages, a pair per "wide" 256x512 tile.
//
// The grid is `sm_budget` CTAs (one per SM: the shared-memory request excludes a second resident
// CTA) and each CTA walks tiles  blockIdx.x, blockIdx.x + gridDim.x, ...  in a fixed order; every output element is
// accumulated over K in the same order whatever the tile shape, so the result never depends on the budget: no atomics on
// the accumulation (the fp32 residual update is one add per element).  The SPLIT instantiations (opt-in, small
// micro-batches) share a tile's K range among CTAs: the later splits store bare partial sums that the following
// normalisation kernel adds in a fixed order, so that mode is deterministic and budget-independent as well.
#pragma once
#include "ptx.cuh"

namespace eas {

constexpr int kBM = 128, kBN = 256, kBK = 64;
constexpr int kEpiWarps = 8;
constexpr int kGemmThreads = 64 + 32 * kEpiWarps + 32;   // + the second producer warp
constexpr int kProducerBWarp = 2 + kEpiWarps;
constexpr int kABytes = kBM * kBK * 2;            // 16 KB: 128 rows of A
// one CTA per tile: a stage holds A (16 KB) + the whole 256-row weight tile (32 KB), 4 stages;
// CTA pair per 256x256 tile: a stage holds A (16 KB) + this CTA's 128 weight rows (16 KB), 6 stages
// NW = 2 ("wide", CTA pairs only): the pair owns a 256x512 tile, i.e. two 256-column accumulators fed by the same
// A tile (three TMA operations for twice the columns) at the price of a single accumulator set: the epilogue no longer
// overlaps the next main loop, so it pays for large K only.
// KD = 2 ("deep"): a stage holds TWO 64-wide k-blocks of each operand, fetched by ONE TMA operation per operand
// (a 3-D box {64 columns, rows, 2 k-blocks}, which lands as two consecutive swizzle-atom blocks).  Measured on B200:
// what a CTA can pull from L2 is set by the number of TMA operations in flight, not by their bytes (two 16 KB
// boxes per 0.46 us, but also two 32 KB boxes per 0.47 us), so deep stages double the operand rate and move the main
// loop from the load path to the tensor pipe.  Half as many, twice as large stages: same shared memory.
template <int CTAS, int NW, int KD = 1> struct GemmCfg {
  static constexpr int kBBytes = (kBN / CTAS) * kBK * 2 * NW;      // per 64-wide k-block
  static constexpr int kStageBytes = (kABytes + kBBytes) * KD;
  static constexpr int kStages = (CTAS == 2 ? (NW == 2 ? 4 : 6) : 4) / KD;
  static constexpr int kAccBuffers = NW == 2 ? 1 : 2;
};
constexpr int kMaxStages = 6;
constexpr int kStagingOff = 4 * 49152;                         // == 6 * 32768; 8 epilogue warps x 4 KB output staging (TMA store source)
constexpr int kBiasOff = kStagingOff + kEpiWarps * 4096;       // 2 x 256 fp32 bias values of the current tiles
constexpr int kBarOff = kBiasOff + 2 * 256 * 4;
constexpr int kGemmSmemBytes = kBarOff + 192 /*barriers*/ + 832 /*alignment slack*/;
static_assert(kGemmSmemBytes <= 232448, "exceeds the 227 KB shared memory of an SM");
constexpr int kTmemCols = 512;
constexpr int kPanelM = 8;                        // m-blocks per rasterisation panel (L2 reuse of W tiles)

enum { ACT_NONE = 0, ACT_GELU = 1, ACT_SWIGLU = 2 };
// OUT_F32_FOLD: the fp32 residual update x = x + A W^T + b done in the epilogue's registers (instead of a reduce-add
// in L2), so that the same pass also writes the bf16 copy of the new rows and their statistics: what the next GEMM's
// folded normalisation reads (see GemmParams::fold_stats).
enum { OUT_BF16 = 0, OUT_F32 = 1, OUT_F32_FOLD = 2 };
constexpr int kFoldGroup = 128;                   // columns per statistics group

struct alignas(64) GemmParams {
  CUtensorMap tma_a;      // 3-D: {K-run, phase, rows}; box {64, 1, 128}.  Deep kernels: {64, rows, K/64}; box {64, 128, 2}
  CUtensorMap tma_b;      // 2-D: {K, N}; box {64, 256} (one CTA per tile) or {64, 128} (CTA pair).  Deep: {64, N, K/64}; box {64, rows, 2}
  CUtensorMap tma_out;    // 2-D over out: box {64 bf16 | 32 fp32, 32 rows}, 128-byte swizzle (valid if use_tma_out)
  int use_tma_out;        // 1: epilogue stages 32-row sub-tiles in shared memory and stores them with TMA
  int M, N;               // rows of A walked by tiles; rows of W
  int k_blocks;           // k-steps: K / 64, or ceil(K / 128) for the deep kernels (TMA fills past K with zeros)
  int kb_per_tap;         // k-blocks per convolution tap (== k_blocks for a plain GEMM)
  int conv_stride;        // 1 for a plain GEMM; row stride of a convolution otherwise
  int m_blocks, n_blocks; // m_blocks counts 128-row blocks (one CTA per tile) or 256-row blocks (CTA pair)
  int reverse;            // 1: walk the tiles last to first (start with the rows the producer of A wrote last: L2)
  const bf16* bias;       // [N] (for SWIGLU: interleaved gate/up like the W rows)
  void* out;              // bf16 or fp32 [*, ldo]
  long long ldo;          // leading dimension of out (elements)
  const float* resid;     // optional fp32 [*, ldo] added to the result (may alias out)
  const int* row_map;     // optional: output row of each A row, negative = drop the row
  const int* pos_idx;     // optional (with pos): row of the position table added to each A row
  const bf16* pos;        // optional position table [*, N]
  const float2* rope_cs;  // optional (cos, sin), stored [pair][A row] so that the 32 rows of a warp read consecutive
                          // entries: columns < rope_ncols are rotated as adjacent pairs
  long long rope_stride;  // entries per pair (= rows of the table)
  int rope_pairs;         // pairs per head (head_dim / 2)
  int rope_ncols;         // rotate output columns [0, rope_ncols)
  int head_dim;
  int w_const;            // W is never written by work earlier in the stream: its loads need not wait for that work
  // Split K (fp32 residual GEMMs with few tiles): a work item is (tile, split); split s accumulates k-blocks
  // [s * kb_per_split, (s + 1) * kb_per_split).  Split 0 runs the ordinary epilogue (bias, reduce-add into the residual
  // stream); split s > 0 stores its bare partial sums into rows [(s - 1) * part_rows, ...) of the fp32 scratch matrix
  // behind tma_part, and the normalisation kernel that follows adds them to the residual rows in a fixed order.
  int splits;             // >= 1
  int kb_per_split;
  int part_rows;          // rows of one split's region of the scratch matrix (a multiple of the tile height)
  CUtensorMap tma_part;   // [(splits - 1) * part_rows, N] fp32, 32-row boxes of 32 columns
  // Folded normalisation.  LayerNorm / RMSNorm followed by a linear layer is  rstd * ((gamma .* x) - mean gamma) W^T + const:
  // the GEMM can run on the rows scaled by gamma only (rounded to bf16: the same single rounding of the operand as
  // with a normalisation kernel) and apply the row's rstd and mean in its epilogue,
  //     out[i, n] = rstd_i * (acc[i, n] - mean_i * c1[n]) + c0[n],   c1[n] = sum_k gamma_k W[n, k],  c0[n] = b[n] + sum_k beta_k W[n, k],
  // so no normalisation kernel runs between the residual GEMM and this one.  The statistics arrive as one (mean, M2)
  // pair per row and group of kFoldGroup columns (M2 = sum of squared deviations from the group's mean), written by
  // the producer of the rows, and are merged in index order: budget- and tile-shape-independent.
  const float2* fold_stats;   // consumer: [fold_parts][fold_rows]; nullptr = no folding
  const float* fold_c0;       // consumer: [N] fp32, replaces bias
  const float* fold_c1;       // consumer: [N] fp32 (LayerNorm; nullptr for RMSNorm, which subtracts no mean)
  long long fold_rows;        // rows of one group's slab of the statistics (both sides)
  int fold_parts;             // groups per row: K / kFoldGroup
  int fold_rms;               // 1: rstd from the mean square; 0: from the variance
  float fold_eps;
  float2* fold_stats_out;     // producer (OUT_F32_FOLD): [N / kFoldGroup][fold_rows]
  bf16* fold_xb;              // producer: bf16(gamma .* updated rows), [*, ldo]
  const bf16* fold_gamma;     // producer: [N], the gamma of the normalisation the rows go through next
  uint32_t* status;       // device status word
};

#ifdef EAS_GEMM_PROFILE
// phase timestamps of epilogue warp 0 of CTA 0 (profiling builds only): [tile][k]
__device__ unsigned long long g_gemm_dbg[32 * 16];
#define GEMM_STAMP(k) do { if (blockIdx.x == 0 && ew == 0 && lane == 0 && tcount < 32) g_gemm_dbg[tcount * 16 + (k)] = clock64(); } while (0)
// one-off timeline of CTA 0 in nanoseconds (row 31 of the same array)
__device__ __forceinline__ unsigned long long gemm_globaltimer() { unsigned long long t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); return t; }
#define GEMM_TL(k) do { if (blockIdx.x == 0) g_gemm_dbg[31 * 16 + (k)] = gemm_globaltimer(); } while (0)
#else
#define GEMM_STAMP(k) do { } while (0)
#define GEMM_TL(k) do { } while (0)
#endif

__device__ __forceinline__ void tile_coords(int tile, int m_blocks, int n_blocks, int& mb, int& nb) {
  const int per_panel = kPanelM * n_blocks;
  const int panel = tile / per_panel;
  const int within = tile - panel * per_panel;
  const int rows_here = min(kPanelM, m_blocks - panel * kPanelM);
  nb = within / rows_here;
  mb = panel * kPanelM + (within - nb * rows_here);
}

// Folded normalisation: a row's factor and offset (rstd, -rstd * mean) from its group statistics, merged in index
// order (groups of equal size).  Kept out of line: the GEMM kernels sit at their register limit.
__device__ __noinline__ float2 fold_row_factors(const float2* stats, long long rows, int parts, int rms, float eps, long long r) {
  float mu = 0.f, m2 = 0.f;
  for (int g = 0; g < parts; ++g) {
    const float2 st = __ldg(stats + g * rows + r);
    const float delta = st.x - mu;
    const float inv = 1.0f / static_cast<float>(g + 1);
    mu += delta * inv;
    m2 += st.y + delta * delta * (static_cast<float>(kFoldGroup * g) * inv);
  }
  const float inv_k = 1.0f / static_cast<float>(kFoldGroup * parts);
  if (rms) return make_float2(1.0f / sqrtf((m2 * inv_k + mu * mu) + eps), 0.f);
  const float a = 1.0f / sqrtf(m2 * inv_k + eps);
  return make_float2(a, -a * mu);
}

// SPLIT: the launch splits K (GemmParams::splits > 1); the ordinary instantiations keep their code free of it.
template <int ACT, int OUT, int CTAS, int NW, int KD = 1, bool SPLIT = false>
__global__ void __launch_bounds__(kGemmThreads, 1) gemm_kernel(const __grid_constant__ GemmParams p) {
  static_assert(NW == 1 || (CTAS == 2 && ACT != ACT_SWIGLU), "wide tiles: CTA pairs, no gated epilogue");
  static_assert(KD == 1 || KD == 2, "one or two 64-wide k-blocks per stage");
  constexpr int kStages = GemmCfg<CTAS, NW, KD>::kStages;
  constexpr int kStageBytes = GemmCfg<CTAS, NW, KD>::kStageBytes;
  constexpr int kAccBuffers = GemmCfg<CTAS, NW, KD>::kAccBuffers;
  constexpr int kBRows = kBN / CTAS;               // weight rows per CTA and 256-column accumulator
  constexpr int kBAtom = kBRows * kBK * 2;         // bytes of one 64-wide k-block of those rows
  constexpr int kTileN = kBN * NW;                 // output columns of a tile
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  // 1024-byte alignment: the 128-byte swizzle pattern repeats every 8 rows of 128 bytes
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kBarOff);
  uint64_t* full_bar = bars;                       // [kStages]  TMA -> MMA (pair: the leader's copy collects both CTAs' bytes)
  uint64_t* empty_bar = bars + kMaxStages;         // [kStages]  MMA -> TMA (pair: signalled in both CTAs)
  uint64_t* acc_full = bars + 2 * kMaxStages;      // [2]        MMA -> epilogue (pair: signalled in both CTAs)
  uint64_t* acc_empty = bars + 2 * kMaxStages + 2; // [2]        epilogue -> MMA (pair: both CTAs' warps arrive at the leader)
  uint64_t* bias_bar = bars + 2 * kMaxStages + 4;  // [2]        epilogue warps: bias values staged
  uint64_t* bias_free = bars + 2 * kMaxStages + 7; // [1]        wide tiles: every epilogue warp has read the staged bias
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * kMaxStages + 6);
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  if (threadIdx.x == 0) GEMM_TL(0);
  const int num_tiles = p.m_blocks * p.n_blocks;
  const int n_splits = SPLIT ? p.splits : 1;
  const int kb_per_split = SPLIT ? p.kb_per_split : p.k_blocks;
  const int num_work = num_tiles * n_splits;       // work items: (tile, split), the splits of a tile on neighbouring CTAs
  const int cta_rank = CTAS == 2 ? static_cast<int>(cluster_ctarank()) : 0;
  const int first_tile = blockIdx.x / CTAS;        // both CTAs of a pair walk the same tiles
  const int tile_step = gridDim.x / CTAS;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&acc_full[a], 1); mbar_init(&acc_empty[a], kEpiWarps * CTAS); mbar_init(&bias_bar[a], kEpiWarps); }
    mbar_init(bias_free, kEpiWarps);
    *abort_flag = 0;
    mbar_fence_init();
    tma_prefetch_desc(&p.tma_a);
    tma_prefetch_desc(&p.tma_b);
    if (p.use_tma_out) tma_prefetch_desc(&p.tma_out);
  }
  if (warp == 1) {
    if (CTAS == 2) { tmem_alloc_pair(tmem_slot, kTmemCols); tmem_relinquish_pair(); }
    else { tmem_alloc(tmem_slot, kTmemCols); tmem_relinquish(); }
  }
  tc_fence_before_sync();
  __syncthreads();
  if (CTAS == 2) cluster_sync_all();               // the peer's barriers are initialised before anything signals them
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  if (threadIdx.x == 0) GEMM_TL(1);
  pdl_launch_dependents();   // the next kernel may set itself up while this one runs
  // everything before this kernel in the stream is complete and visible; the W producer of a GEMM on constant
  // weights goes ahead and fills the ring's W halves meanwhile (the stages complete once A has arrived too)
  if (!(p.w_const && warp == kProducerBWarp)) pdl_wait();
  if (threadIdx.x == 0) GEMM_TL(2);

  if (warp == 0 || warp == kProducerBWarp) {
    // ------------------------------------------------------------------ producers: warp 0 loads A, the last warp B
    // Issuing a TMA operation occupies the issuing thread for some 70 ns, and that is what bounds the operand rate
    // of a CTA (measured: a step of two 32 KB boxes takes 476 ns from one thread, 396 ns from two), so the two
    // operands have a thread each.  The A thread announces the bytes of the whole stage.
    const bool do_a = warp == 0, do_b = warp != 0;
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int work = first_tile; work < num_work && ok; work += tile_step) {
        const int tile = SPLIT ? work / n_splits : work, split = SPLIT ? work - tile * n_splits : 0;
        int mg, nb;
        tile_coords(p.reverse ? num_tiles - 1 - tile : tile, p.m_blocks, p.n_blocks, mg, nb);
        const int mb = mg * CTAS + cta_rank;       // this CTA's 128-row block
        const int kb0 = split * kb_per_split, kb1 = SPLIT ? min(p.k_blocks, kb0 + kb_per_split) : p.k_blocks;
        for (int kb = kb0; kb < kb1; ++kb, ++it) {
          const int s = it % kStages;
          const uint32_t ph = (it / kStages) & 1u;
          // The W producer of constant weights skipped the grid-dependency wait above and has filled every stage once;
          // its next wait needs the consumer, which needs A, which needs the earlier kernels: join the dependency first,
          // so that the bounded wait below never runs while a predecessor is still working.
          if (do_b && p.w_const && it == kStages) pdl_wait();
          if (!mbar_wait(&empty_bar[s], ph ^ 1u, abort_flag)) { ok = false; break; }
          uint8_t* sa = smem + s * kStageBytes;
          uint8_t* sb = sa + kABytes * KD;
          // both CTAs' loads of a pair complete on the leader's barrier; the leader announces the bytes of both
          if (do_a && cta_rank == 0) mbar_expect_tx(&full_bar[s], CTAS * kStageBytes);
          if (KD == 2) {
            // deep stage (plain GEMM only): [A k-block 0][A k-block 1][B ...] from one 3-D box per operand
            if (CTAS == 2) {
              if (do_a) tma_load_3d_pair(sa, &p.tma_a, &full_bar[s], 0, mb * kBM, kb * KD);
              if (do_b) {
#pragma unroll
                for (int h = 0; h < NW; ++h)
                  tma_load_3d_pair(sb + h * kBAtom * KD, &p.tma_b, &full_bar[s], 0, nb * kTileN + h * kBN + cta_rank * kBRows, kb * KD);
              }
            } else {
              if (do_a) tma_load_3d(sa, &p.tma_a, &full_bar[s], 0, mb * kBM, kb * KD);
              if (do_b) tma_load_3d(sb, &p.tma_b, &full_bar[s], 0, nb * kBN, kb * KD);
            }
            continue;
          }
          const int tap = kb / p.kb_per_tap;
          const int kx = (kb - tap * p.kb_per_tap) * kBK;
          if (CTAS == 2) {
            if (do_a) tma_load_3d_pair(sa, &p.tma_a, &full_bar[s], kx, tap % p.conv_stride, mb * kBM + tap / p.conv_stride);
            if (do_b) {
#pragma unroll
              for (int h = 0; h < NW; ++h)
                tma_load_2d_pair(sb + h * kBAtom, &p.tma_b, &full_bar[s], kb * kBK, nb * kTileN + h * kBN + cta_rank * kBRows);
            }
          } else {
            if (do_a) tma_load_3d(sa, &p.tma_a, &full_bar[s], kx, tap % p.conv_stride, mb * kBM + tap / p.conv_stride);
            if (do_b) tma_load_2d(sb, &p.tma_b, &full_bar[s], kb * kBK, nb * kBN);
          }
        }
      }
      if (!ok) {
        // give loads already in flight a bounded chance to land before the CTA retires
        for (int s = 0; s < kStages; ++s) {
          const long long t0 = clock64();
          while (clock64() - t0 < 2000000) {}
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ UMMA issuer
    if (lane == 0 && cta_rank == 0) {
      constexpr uint32_t idesc = make_idesc_bf16(kBM * CTAS, kBN, 0, 0);
      uint32_t it = 0, tcount = 0;
      bool ok = true;
      for (int work = first_tile; work < num_work && ok; work += tile_step, ++tcount) {
        const uint32_t acc = tcount % kAccBuffers;
        const uint32_t acc_ph = (tcount / kAccBuffers) & 1u;
        if (!mbar_wait(&acc_empty[acc], acc_ph ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after_sync();
        const uint32_t tmem_d = tmem_base + acc * kBN;
        const int split = SPLIT ? work % n_splits : 0;
        const int kb0 = split * kb_per_split, kb1 = SPLIT ? min(p.k_blocks, kb0 + kb_per_split) : p.k_blocks;
        for (int kb = kb0; kb < kb1; ++kb, ++it) {
          const int s = it % kStages;
          const uint32_t ph = (it / kStages) & 1u;
          if (!mbar_wait(&full_bar[s], ph, abort_flag)) { ok = false; break; }
          if (tcount == 0 && kb == kb0) GEMM_TL(3);
          tc_fence_after_sync();
          const uint32_t a_addr = smem_u32(smem + s * kStageBytes);
          const uint32_t b_addr = a_addr + kABytes * KD;
#pragma unroll
          for (int a = 0; a < KD; ++a) {         // the 64-wide k-blocks of the stage: one swizzle-atom block each
            const uint64_t adesc = make_smem_desc(a_addr + a * kABytes, 16, 1024, kSwizzle128B);
            const uint64_t bdesc = make_smem_desc(b_addr + a * kBAtom, 16, 1024, kSwizzle128B);
#pragma unroll
            for (int k = 0; k < kBK / 16; ++k) {
              // advancing 16 bf16 = 32 bytes along K inside the swizzle atom: +2 in the (>>4) address field
              if (CTAS == 2) {
#pragma unroll
                for (int h = 0; h < NW; ++h)   // second accumulator: the next 128 weight rows of each CTA
                  umma_bf16_ss_pair(tmem_d + h * kBN, adesc + 2 * k, bdesc + 2 * k + h * (kBAtom * KD / 16), idesc,
                                    ((kb - kb0) | a | k) != 0);
              } else {
                umma_bf16_ss(tmem_d, adesc + 2 * k, bdesc + 2 * k, idesc, ((kb - kb0) | a | k) != 0);
              }
            }
          }
          // frees the stage (in both CTAs of a pair) once these UMMAs have read it
          if (CTAS == 2) umma_commit_pair_multicast(&empty_bar[s], 3); else umma_commit(&empty_bar[s]);
        }
        if (ok) {                               // accumulator complete
          if (CTAS == 2) umma_commit_pair_multicast(&acc_full[acc], 3); else umma_commit(&acc_full[acc]);
        }
      }
    }
  } else if (warp < kProducerBWarp) {
    // ------------------------------------------------------------------ epilogue
    const int ew = warp - 2;                    // 0..7
    const int quarter = warp & 3;               // TMEM lane quarter this warp may read
    const int half = ew >> 2;                   // which 128 accumulator columns
    uint32_t tcount = 0;
    bool ok = true;
    auto release_accumulator = [&](uint32_t acc) {   // this warp has read its part of the accumulator
      tc_fence_before_sync();
      GEMM_STAMP(12);
      __syncwarp();
      GEMM_STAMP(13);
      if (lane == 0) {
        if (CTAS == 2) mbar_arrive_cluster_relaxed(&acc_empty[acc], 0); else mbar_arrive(&acc_empty[acc]);
      }
    };
    for (int work = first_tile; work < num_work && ok; work += tile_step, ++tcount) {
      const int tile = SPLIT ? work / n_splits : work, split = SPLIT ? work - tile * n_splits : 0;
      int mg, nb;
      tile_coords(p.reverse ? num_tiles - 1 - tile : tile, p.m_blocks, p.n_blocks, mg, nb);
      const int mb = mg * CTAS + cta_rank;
      const uint32_t acc = tcount % kAccBuffers;
      const uint32_t acc_ph = (tcount / kAccBuffers) & 1u;
      if (p.use_tma_out) {
        // ---- staged path: bias from shared memory, 32-row sub-tiles written to a swizzled staging buffer
        //      and stored (or reduce-added, for the fp32 residual stream) by TMA; rows >= M are clipped by TMA
        float* sbias = reinterpret_cast<float*>(smem + kBiasOff) + acc * 256;   // wide tiles use both halves as one
        // With two accumulator buffers the other buffer's bias_bar (eight arrivals) lies between two uses of a bias slot
        // and orders them.  A wide tile has ONE slot: nobody may overwrite it before all eight warps have finished
        // reading the previous tile's values (each arrives at bias_free after its last chunk).
        if (kAccBuffers == 1 && tcount > 0 && !mbar_wait(bias_free, (tcount - 1) & 1u, abort_flag)) { ok = false; break; }
        {
#pragma unroll
          for (int h = 0; h < NW; ++h) {
            const int col = nb * kTileN + h * 256 + ew * 32 + lane;
            sbias[h * 256 + ew * 32 + lane] = (col < p.N && split == 0) ? (p.fold_stats != nullptr ? p.fold_c0[col] : __bfloat162float(p.bias[col])) : 0.f;
          }
          __syncwarp();
          if (lane == 0) mbar_arrive(&bias_bar[acc]);
        }
        // folded normalisation: this thread's row factor and offset, from the row's group statistics (loaded while the
        // tile's main loop is still running)
        float fold_a = 1.f, fold_b = 0.f;
        if (p.fold_stats != nullptr) {
          const float2 f = fold_row_factors(p.fold_stats, p.fold_rows, p.fold_parts, p.fold_rms, p.fold_eps,
                                            min(mb * kBM + quarter * 32 + lane, p.M - 1));
          fold_a = f.x; fold_b = f.y;
        }
        if (OUT == OUT_F32_FOLD) {
          // the rows this tile updates, towards L2 while the main loop runs (the epilogue reads them with plain loads)
          const int r = mb * kBM + quarter * 32 + lane;
          if (r < p.M) {
            const char* base = reinterpret_cast<const char*>(p.resid + static_cast<long long>(r) * p.ldo + nb * kTileN + half * (128 * NW));
#pragma unroll
            for (int i = 0; i < 4 * NW; ++i)
              if (nb * kTileN + half * (128 * NW) + i * 32 < p.N) asm volatile("prefetch.global.L2 [%0];" ::"l"(base + i * 128));
          }
        }
        GEMM_STAMP(0);
        if (!mbar_wait(&acc_full[acc], acc_ph, abort_flag)) { ok = false; break; }
        GEMM_STAMP(1);
        if (tcount == 0 && ew == 0 && lane == 0) GEMM_TL(4);
        if (!mbar_wait(&bias_bar[acc], acc_ph, abort_flag)) { ok = false; break; }
        tc_fence_after_sync();
        GEMM_STAMP(2);
        uint8_t* stage = smem + kStagingOff + ew * 4096;
        uint8_t* srow = stage + lane * 128;
        const int sw = lane & 7;
        const int arow = mb * kBM + quarter * 32 + lane;
        const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + acc * kBN + half * (128 * NW);
        const int ycoord = mb * kBM + quarter * 32;

        auto finish_chunk = [&](float (&v)[32], int c) {   // bias, rotary, activation on 32 accumulator columns
          const int col0 = nb * kTileN + half * (128 * NW) + c * 32;
          const float4* b4 = reinterpret_cast<const float4*>(sbias + half * (128 * NW) + c * 32);
          if (p.fold_stats != nullptr) {
            // out = rstd * acc + (c0 - rstd * mean * c1): the staged "bias" is c0
            const bool centred = p.fold_c1 != nullptr && col0 < p.N;
            const float4* c4 = reinterpret_cast<const float4*>(p.fold_c1 + (centred ? col0 : 0));
#pragma unroll
            for (int q = 0; q < 8; ++q) {
              float4 b = b4[q];
              if (centred) {
                const float4 c1 = __ldg(c4 + q);
                b.x = fmaf(fold_b, c1.x, b.x); b.y = fmaf(fold_b, c1.y, b.y); b.z = fmaf(fold_b, c1.z, b.z); b.w = fmaf(fold_b, c1.w, b.w);
              }
              v[4 * q] = fmaf(fold_a, v[4 * q], b.x); v[4 * q + 1] = fmaf(fold_a, v[4 * q + 1], b.y);
              v[4 * q + 2] = fmaf(fold_a, v[4 * q + 2], b.z); v[4 * q + 3] = fmaf(fold_a, v[4 * q + 3], b.w);
            }
          } else {
#pragma unroll
            for (int q = 0; q < 8; ++q) {
              const float4 b = b4[q];
              v[4 * q] += b.x; v[4 * q + 1] += b.y; v[4 * q + 2] += b.z; v[4 * q + 3] += b.w;
            }
          }
          if (p.rope_cs != nullptr && col0 < p.rope_ncols && arow < p.M) {
            int pi = (col0 % p.head_dim) >> 1;
            const float2* cs = p.rope_cs + arow;
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const float2 t = __ldg(cs + pi * p.rope_stride);
              const float x0 = v[2 * j], x1 = v[2 * j + 1];
              v[2 * j] = x0 * t.x - x1 * t.y;
              v[2 * j + 1] = x1 * t.x + x0 * t.y;
              if (++pi == p.rope_pairs) pi = 0;
            }
          }
          if (ACT == ACT_GELU) {
#pragma unroll
            for (int i = 0; i < 32; i += 2) gelu_erf_pair(v[i], v[i + 1]);
          }
        };
        auto staging_free = [&]() {       // the previous bulk store has finished READING the staging buffer
          if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
          __syncwarp();
        };
        // where the sub-tiles go: the output (reduce-added into the fp32 residual stream), or, for the bare partial sums
        // of a later split, this split's region of the scratch matrix (plain stores)
        const bool later_split = SPLIT && OUT == OUT_F32 && split > 0;
        const uint64_t out_map = reinterpret_cast<uint64_t>(later_split ? &p.tma_part : &p.tma_out);
        const int out_y = later_split ? (split - 1) * p.part_rows + ycoord : ycoord;
        const bool out_reduce = OUT == OUT_F32 && p.resid != nullptr && !later_split;
        auto store_subtile = [&](int x) { // one TMA store / reduce-add of the 32-row staging buffer at column x
          fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) {
            if (out_reduce) {
              // the residual rows keep their place in L2 (evict-last): the normalisation that follows reads them there,
              // and their write-back does not compete with this launch's own traffic (measured: out-projection -5 %)
              asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.bulk_group.L2::cache_hint [%0, {%2, %3}], [%1], %4;"
                           ::"l"(out_map), "r"(smem_u32(stage)), "r"(x), "r"(out_y), "l"(l2_policy_evict_last()) : "memory");
            } else {
              asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                           ::"l"(out_map), "r"(smem_u32(stage)), "r"(x), "r"(out_y) : "memory");
            }
            asm volatile("cp.async.bulk.commit_group;" ::: "memory");
          }
        };

        if (OUT == OUT_F32_FOLD) {
          // x = x + A W^T + b in registers, one 32-column chunk per round: the old values by plain loads (one chunk
          // ahead, prefetched towards L2 before the main loop ended), the new ones through the staging buffer and a
          // TMA store; the bf16 copy (scaled by the next normalisation's gamma) straight from registers; the chunk's mean and squared deviations merged into its
          // 128-column group, written when the group is complete.
          static_assert(OUT != OUT_F32_FOLD || ACT == ACT_NONE, "the folding residual epilogue has no activation");
          constexpr int kChunks = 4 * NW;
          const bool row_ok = arow < p.M;
          const int tcol0 = nb * kTileN + half * (128 * NW);
          const long long roff = static_cast<long long>(row_ok ? arow : 0) * p.ldo + tcol0;
          const float4* xin = reinterpret_cast<const float4*>(p.resid + roff);
          uint4* xb = reinterpret_cast<uint4*>(p.fold_xb + roff);
          const float4* b4 = reinterpret_cast<const float4*>(sbias + half * (128 * NW));
          uint32_t r[32];
          float4 xo[8];
          __syncwarp();
          tmem_ld_32x32(taddr, r);
#pragma unroll
          for (int q = 0; q < 8; ++q) xo[q] = (row_ok && tcol0 < p.N) ? __ldcg(xin + q) : make_float4(0.f, 0.f, 0.f, 0.f);
          float gm = 0.f, gm2 = 0.f;
#pragma unroll 1
          for (int c = 0; c < kChunks; ++c) {
            tmem_ld_wait();
            float v[32];
#pragma unroll
            for (int q = 0; q < 8; ++q) {
              const float4 b = b4[c * 8 + q];
              v[4 * q] = (__uint_as_float(r[4 * q]) + b.x) + xo[q].x;
              v[4 * q + 1] = (__uint_as_float(r[4 * q + 1]) + b.y) + xo[q].y;
              v[4 * q + 2] = (__uint_as_float(r[4 * q + 2]) + b.z) + xo[q].z;
              v[4 * q + 3] = (__uint_as_float(r[4 * q + 3]) + b.w) + xo[q].w;
            }
            const int col0 = tcol0 + c * 32;
            if (c + 1 < kChunks) {
              __syncwarp();
              tmem_ld_32x32(taddr + (c + 1) * 32, r);
              const bool more = row_ok && col0 + 32 < p.N;
#pragma unroll
              for (int q = 0; q < 8; ++q) xo[q] = more ? __ldcg(xin + (c + 1) * 8 + q) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
            // the chunk's statistics (two passes over registers), merged into the group's (counts 32 k and 32)
            float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
            for (int i = 0; i < 32; i += 4) { s0 += v[i]; s1 += v[i + 1]; s2 += v[i + 2]; s3 += v[i + 3]; }
            const float cm = ((s0 + s1) + (s2 + s3)) * (1.0f / 32.0f);
            float q0 = 0.f, q1 = 0.f;
#pragma unroll
            for (int i = 0; i < 32; i += 2) {
              const float t0 = v[i] - cm, t1 = v[i + 1] - cm;
              q0 = fmaf(t0, t0, q0); q1 = fmaf(t1, t1, q1);
            }
            const int k = c & 3;
            if (k == 0) {
              gm = cm; gm2 = q0 + q1;
            } else {
              const float delta = cm - gm;
              const float inv = 1.0f / static_cast<float>(k + 1);
              gm += delta * inv;
              gm2 += (q0 + q1) + delta * delta * (static_cast<float>(32 * k) * inv);
            }
            if (k == 3 && row_ok && col0 < p.N)
              p.fold_stats_out[static_cast<long long>(col0 / kFoldGroup) * p.fold_rows + arow] = make_float2(gm, gm2);
            staging_free();
#pragma unroll
            for (int q = 0; q < 8; ++q)
              *reinterpret_cast<float4*>(srow + ((q ^ sw) << 4)) = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
            if (col0 < p.N) store_subtile(col0);
            if (row_ok && col0 < p.N) {
              const uint4* g4 = reinterpret_cast<const uint4*>(p.fold_gamma + col0);
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                const uint4 g = __ldg(g4 + q);
                xb[c * 4 + q] = make_uint4(pack_bf16x2(v[8 * q] * bf16_lo(g.x), v[8 * q + 1] * bf16_hi(g.x)),
                                           pack_bf16x2(v[8 * q + 2] * bf16_lo(g.y), v[8 * q + 3] * bf16_hi(g.y)),
                                           pack_bf16x2(v[8 * q + 4] * bf16_lo(g.z), v[8 * q + 5] * bf16_hi(g.z)),
                                           pack_bf16x2(v[8 * q + 6] * bf16_lo(g.w), v[8 * q + 7] * bf16_hi(g.w)));
              }
            }
          }
        } else if (OUT == OUT_F32) {
          // fp32 output: 32 columns = one 128-byte staging row, so every 32-column chunk is a sub-tile (and a TMA
          // operation) of its own.  One chunk per round, the next chunk's TMEM load in flight meanwhile, so that the
          // wait for the previous operation to release the staging buffer falls behind a load and the chunk's math.
          constexpr int kChunks = 4 * NW;
          uint32_t r[32];
          __syncwarp();
          tmem_ld_32x32(taddr, r);
#pragma unroll 1
          for (int c = 0; c < kChunks; ++c) {
            tmem_ld_wait();
            float v[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
            if (c + 1 < kChunks) {
              __syncwarp();
              tmem_ld_32x32(taddr + (c + 1) * 32, r);
            }
            finish_chunk(v, c);
            const int col0 = nb * kTileN + half * (128 * NW) + c * 32;
            staging_free();
#pragma unroll
            for (int q = 0; q < 8; ++q)
              *reinterpret_cast<float4*>(srow + ((q ^ sw) << 4)) = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
            if (col0 < p.N) store_subtile(col0);
          }
        } else {
#pragma unroll 1
        for (int pr = 0; pr < 2 * NW; ++pr) {       // two chunks (64 accumulator columns) per round
          uint32_t r0[32], r1[32];
          __syncwarp();
          tmem_ld_32x32(taddr + pr * 64, r0);
          tmem_ld_32x32(taddr + pr * 64 + 32, r1);
          tmem_ld_wait();
          GEMM_STAMP(3 + pr * 4);
          float v0[32], v1[32];
#pragma unroll
          for (int i = 0; i < 32; ++i) { v0[i] = __uint_as_float(r0[i]); v1[i] = __uint_as_float(r1[i]); }
          finish_chunk(v0, pr * 2);
          finish_chunk(v1, pr * 2 + 1);
          GEMM_STAMP(4 + pr * 4);
          const int col0 = nb * kTileN + half * (128 * NW) + pr * 64;
          if (OUT == OUT_F32) {
            // 32 fp32 columns = one 128-byte staging row; two sub-tiles per round
#pragma unroll
            for (int h2 = 0; h2 < 2; ++h2) {
              float (&v)[32] = h2 ? v1 : v0;
              staging_free();
#pragma unroll
              for (int q = 0; q < 8; ++q)
                *reinterpret_cast<float4*>(srow + ((q ^ sw) << 4)) = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
              if (col0 + h2 * 32 < p.N) store_subtile(col0 + h2 * 32);
            }
          } else if (ACT == ACT_SWIGLU) {
            // (gate, up) pairs -> 32 outputs per round; the 64 outputs of both rounds form one staging row
            if (pr == 0) staging_free();
#pragma unroll
            for (int h2 = 0; h2 < 2; ++h2) {
              float (&v)[32] = h2 ? v1 : v0;
              uint32_t w[8];
#pragma unroll
              for (int j = 0; j < 8; ++j)
                w[j] = pack_bf16x2(silu_f(v[4 * j]) * v[4 * j + 1], silu_f(v[4 * j + 2]) * v[4 * j + 3]);
              const int q0 = pr * 4 + h2 * 2;
              *reinterpret_cast<uint4*>(srow + (((q0) ^ sw) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
              *reinterpret_cast<uint4*>(srow + (((q0 + 1) ^ sw) << 4)) = make_uint4(w[4], w[5], w[6], w[7]);
            }
            if (pr == 1 && nb * kBN + half * 128 < p.N) store_subtile((nb * kBN + half * 128) >> 1);
          } else {
            // 64 bf16 columns = one 128-byte staging row
            staging_free();
            GEMM_STAMP(5 + pr * 4);
#pragma unroll
            for (int h2 = 0; h2 < 2; ++h2) {
              float (&v)[32] = h2 ? v1 : v0;
#pragma unroll
              for (int q = 0; q < 4; ++q)
                *reinterpret_cast<uint4*>(srow + (((h2 * 4 + q) ^ sw) << 4)) =
                    make_uint4(pack_bf16x2(v[8 * q], v[8 * q + 1]), pack_bf16x2(v[8 * q + 2], v[8 * q + 3]),
                               pack_bf16x2(v[8 * q + 4], v[8 * q + 5]), pack_bf16x2(v[8 * q + 6], v[8 * q + 7]));
            }
            if (col0 < p.N) store_subtile(col0);
            GEMM_STAMP(6 + pr * 4);
          }
        }
        }
        release_accumulator(acc);
        if (kAccBuffers == 1 && lane == 0) mbar_arrive(bias_free);   // this warp's reads of the staged bias are done (after the __syncwarp above)
        GEMM_STAMP(11);
        if (tcount == 0 && ew == 0 && lane == 0) GEMM_TL(5);
        continue;
      }

      if (!mbar_wait(&acc_full[acc], acc_ph, abort_flag)) { ok = false; break; }
      tc_fence_after_sync();

      const int arow = mb * kBM + quarter * 32 + lane;            // row of A (== accumulator row)
      long long orow = arow;
      bool row_ok = arow < p.M;
      if (row_ok && p.row_map != nullptr) {
        const int mapped = p.row_map[arow];
        row_ok = mapped >= 0;
        orow = mapped;
      }
      const int posrow = (row_ok && p.pos_idx != nullptr) ? p.pos_idx[arow] : 0;

#pragma unroll 1
      for (int c = 0; c < 4; ++c) {
        const int col_in_tile = half * 128 + c * 32;
        const int col0 = nb * kBN + col_in_tile;                  // first of 32 output-space accumulator columns
        uint32_t raw[32];
        __syncwarp();   // the TMEM load is warp-collective: reconverge after the per-row branches below
        tmem_ld_32x32(tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + acc * kBN + col_in_tile, raw);
        tmem_ld_wait();
        if (!row_ok || col0 >= p.N) continue;
        float v[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(raw[i]);
        {  // bias: 32 bf16 = 64 bytes, the same for every row
          const uint4* bp = reinterpret_cast<const uint4*>(p.bias + col0);
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const uint4 b = __ldg(bp + q);
            const uint32_t w[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              v[q * 8 + 2 * j] += bf16_lo(w[j]);
              v[q * 8 + 2 * j + 1] += bf16_hi(w[j]);
            }
          }
        }
        if (p.rope_cs != nullptr && col0 < p.rope_ncols) {
          // rotary: adjacent columns (2i, 2i+1) of a head form pair i (the weight rows were
          // re-ordered at create time so that the two halves of a pair sit side by side)
          const float2* cs = p.rope_cs + arow;
          int pi = (col0 % p.head_dim) >> 1;
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            const float2 t = __ldg(cs + pi * p.rope_stride);
            const float x0 = v[2 * j], x1 = v[2 * j + 1];
            v[2 * j] = x0 * t.x - x1 * t.y;
            v[2 * j + 1] = x1 * t.x + x0 * t.y;
            if (++pi == p.rope_pairs) pi = 0;
          }
        }
        if (ACT == ACT_GELU) {
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] = gelu_erf(v[i]);
        }
        if (ACT == ACT_SWIGLU) {
          // columns (2j, 2j+1) = (gate_j, up_j); 16 outputs per 32 accumulator columns
          bf16* o = reinterpret_cast<bf16*>(p.out) + orow * p.ldo + (col0 >> 1);
          uint32_t w[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const float a0 = silu_f(v[4 * j]) * v[4 * j + 1];
            const float a1 = silu_f(v[4 * j + 2]) * v[4 * j + 3];
            w[j] = pack_bf16x2(a0, a1);
          }
          uint4* o4 = reinterpret_cast<uint4*>(o);
          o4[0] = make_uint4(w[0], w[1], w[2], w[3]);
          o4[1] = make_uint4(w[4], w[5], w[6], w[7]);
          continue;
        }
        if (p.pos != nullptr) {
          const uint4* pp = reinterpret_cast<const uint4*>(p.pos + static_cast<long long>(posrow) * p.N + col0);
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const uint4 b = __ldg(pp + q);
            const uint32_t w[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              v[q * 8 + 2 * j] += bf16_lo(w[j]);
              v[q * 8 + 2 * j + 1] += bf16_hi(w[j]);
            }
          }
        }
        if (OUT != OUT_BF16) {
          float* o = reinterpret_cast<float*>(p.out) + orow * p.ldo + col0;
          if (p.resid != nullptr) {
            const float4* r4 = reinterpret_cast<const float4*>(p.resid + orow * p.ldo + col0);
#pragma unroll
            for (int q = 0; q < 8; ++q) {
              const float4 r = r4[q];
              v[4 * q] += r.x; v[4 * q + 1] += r.y; v[4 * q + 2] += r.z; v[4 * q + 3] += r.w;
            }
          }
          float4* o4 = reinterpret_cast<float4*>(o);
#pragma unroll
          for (int q = 0; q < 8; ++q) o4[q] = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
        } else {
          bf16* o = reinterpret_cast<bf16*>(p.out) + orow * p.ldo + col0;
          uint4* o4 = reinterpret_cast<uint4*>(o);
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            o4[q] = make_uint4(pack_bf16x2(v[8 * q], v[8 * q + 1]), pack_bf16x2(v[8 * q + 2], v[8 * q + 3]),
                               pack_bf16x2(v[8 * q + 4], v[8 * q + 5]), pack_bf16x2(v[8 * q + 6], v[8 * q + 7]));
          }
        }
      }
      // all TMEM reads of this warp are complete (wait::ld above): hand the accumulator back
      release_accumulator(acc);
    }
    // bulk stores still reading the staging buffer must finish before the CTA's shared memory is released
    if (p.use_tma_out && lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    if (ew == 0 && lane == 0) GEMM_TL(6);
  }

  tc_fence_before_sync();
  __syncthreads();
  if (CTAS == 2) cluster_sync_all();               // no CTA of the pair retires while the other may still signal it
  if (warp == 1) {
    tc_fence_after_sync();
    if (CTAS == 2) tmem_dealloc_pair(tmem_base, kTmemCols); else tmem_dealloc(tmem_base, kTmemCols);
  }
  if (threadIdx.x == 0) GEMM_TL(7);
  if (threadIdx.x == 0 && *abort_flag) atomicCAS(p.status, DEV_OK, DEV_ERR_WAIT_TIMEOUT);
}

}  // namespace eas
