// Patch embedding as an im2col-fused GEMM for sm_100a:
//
//     x[row(m), :] = patch(m) * W_emb^T + b (+ pos[posrow(m), :])        m = patch index over the micro-batch
//
// The A operand (one row per patch: its pixels in the order channel, frame-in-patch, row, column) is never
// materialised in global memory.  Gather warps read the pixel runs of 128 patches straight from the packed images /
// clips and write them into shared memory in the layout a 128-byte-swizzled TMA tile would have, so the tensor core
// reads them through the same UMMA descriptors as any other A tile.  (TMA itself cannot fetch them: a run of a
// 14-pixel patch row is 28 bytes long and starts on a 28-byte grid, neither a multiple of 16.)
//
// Gathering is the expensive part (small scattered loads), so it is done ONCE per patch: a CTA owns a block of 128
// patches, keeps up to kEgMaxResident 64-wide k-blocks of their rows resident in shared memory and runs ALL column
// blocks of the output against them while the weight tiles stream through a small TMA ring.  A patch vector longer
// than the resident part is processed in passes over K: the first pass stores bias + position + partial sum, every
// later pass adds its partial sum to the stored row (one fixed order, so the result is deterministic).
//
//   warp 0        TMA producer of the weight tiles (256 rows x 64 columns per stage), lane 0
//   warp 1        UMMA issuer (128 x 256 x 16, fp32 accumulators in TMEM, two accumulator buffers), lane 0
//   warps 2..9    gather: two threads per patch row, each loads 16 pixel pairs of a k-block (4-byte loads; a pair
//                 never straddles a run because patch edges are even) and stores four swizzled 16-byte chunks; the
//                 loads of the next k-block are issued before the current one is stored
//   warps 10..13  epilogue: tcgen05.ld -> + bias (+ position row) or + stored row -> fp32 rows of the residual stream,
//                 scattered by the row map (CLS rows and item boundaries make output rows differ from patch rows)
//
// The grid is at most `sm_budget` CTAs, one per SM, walking the patch blocks blockIdx.x, + gridDim.x, ...; every output
// element is accumulated over K in one fixed order, so results do not depend on the budget.
#pragma once
#include "elementwise.cuh"
#include "ptx.cuh"

namespace eas {

constexpr int kEgThreads = 14 * 32;
constexpr int kEgGatherWarps = 8;
constexpr int kEgMaxResident = 10;                      // k-blocks of the A rows kept in shared memory per pass, at most
constexpr int kEgWStages = 2;
constexpr int kEgABytes = 128 * 64 * 2;                 // 16 KB: 128 patch rows x 64 elements
constexpr int kEgBBytes = 256 * 64 * 2;                 // 32 KB: 256 weight rows x 64 elements
// shared memory: [resident A: R x 16 KB][weight ring: 2 x 32 KB][barriers]; R = 10 fills an SM's 227 KB
constexpr int kEgSmemBytes = kEgMaxResident * kEgABytes + kEgWStages * kEgBBytes + 512 + 1024;   // + barriers + alignment slack
static_assert(kEgSmemBytes <= 232448, "exceeds the shared memory of an SM");

struct EmbedGemmParams {
  CUtensorMap tma_w;       // W_emb [N, K_pad] (K zero-padded to a multiple of 64), box {64, 256}, 128-byte swizzle
  const bf16* data;        // packed items: image [C, H, W]; clip [F, C, H, W]
  const bf16* bias;        // [N]
  float* x;                // residual stream [*, N]
  const int* row_map;      // [n_patches] -> row of x
  const int* pos_idx;      // [n_patches] -> row of the position table (with pos)
  const bf16* pos;         // optional position table [*, N]
  int n_patches, N;
  int k, k_pad;            // patch elements C * pt * P * P, and the same padded to a multiple of 64
  int channels, patch, tpatch;
  int merge_order;         // 0: patches in raster order; 1: merge-group-major (the four patches of a 2x2 group adjacent)
  int pairs_ok;            // 1: patch edge, image widths and item offsets are even, so pixel pairs are 4-byte aligned
  const uint32_t* table;   // [k_pad / 2] where each pixel pair of the patch vector comes from (built once per encoder)
  uint32_t* status;
  ItemTable items;         // aux_start = patch-row prefix per item
};

// Table entry of a pixel pair (elements k, k + 1 of the patch vector): channel << 24 | frame-in-patch << 16 | py << 8 | px.
// 0xFFFFFFFF: padding behind the patch vector (zeros).
constexpr uint32_t kEgPad = 0xFFFFFFFFu;

// Fills the pair table of an architecture (create time).
__global__ void embed_table_kernel(uint32_t* table, int k, int k_pad, int patch, int tpatch) {
  const int PP = patch * patch;
  for (int j = blockIdx.x * blockDim.x + threadIdx.x; j < k_pad / 2; j += gridDim.x * blockDim.x) {
    const int kk = 2 * j;
    uint32_t e = kEgPad;
    if (kk < k) {
      const int plane = kk / PP, rem = kk - plane * PP;          // plane = channel * pt + frame-in-patch
      const int py = rem / patch, px = rem - py * patch;
      const int ch = plane / tpatch, f = plane - ch * tpatch;
      e = (static_cast<uint32_t>(ch) << 24) | (static_cast<uint32_t>(f) << 16) | (static_cast<uint32_t>(py) << 8) | static_cast<uint32_t>(px);
    }
    table[j] = e;
  }
}

__global__ void __launch_bounds__(kEgThreads, 1) embed_gemm_kernel(const __grid_constant__ EmbedGemmParams p) {
  extern __shared__ __align__(1024) uint8_t smem_raw_eg[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw_eg) + 1023) & ~uintptr_t(1023));
  const int k_blocks = p.k_pad / 64;
  const int resident = min(k_blocks, kEgMaxResident);
  uint8_t* wring = smem + resident * kEgABytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(wring + kEgWStages * kEgBBytes);
  uint64_t* a_full = bars;                             // [resident] the gather warps have written the slot
  uint64_t* a_free = bars + kEgMaxResident;            // [resident] the last UMMA that reads the slot has completed
  uint64_t* w_full = bars + 2 * kEgMaxResident;        // [kEgWStages]
  uint64_t* w_empty = w_full + kEgWStages;             // [kEgWStages]
  uint64_t* acc_full = w_empty + kEgWStages;           // [2]
  uint64_t* acc_empty = acc_full + 2;                  // [2] 4 epilogue warps
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m_blocks = (p.n_patches + 127) / 128;
  const int n_blocks = (p.N + 255) / 256;
  const int passes = (k_blocks + resident - 1) / resident;

  if (threadIdx.x == 0) {
    for (int s = 0; s < resident; ++s) { mbar_init(&a_full[s], kEgGatherWarps); mbar_init(&a_free[s], 1); }
    for (int s = 0; s < kEgWStages; ++s) { mbar_init(&w_full[s], 1); mbar_init(&w_empty[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&acc_full[a], 1); mbar_init(&acc_empty[a], 4); }
    *abort_flag = 0;
    mbar_fence_init();
    tma_prefetch_desc(&p.tma_w);
  }
  if (warp == 1) { tmem_alloc(tmem_slot, 512); tmem_relinquish(); }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  pdl_launch_dependents();
  if (warp != 0) pdl_wait();     // the weights are constant: their loads need not wait for the stream's earlier work

  // a whole warp waits on a barrier: lane 0 polls, the outcome is the same for all lanes (so the warp leaves a loop together)
  auto warp_wait = [&](uint64_t* bar, uint32_t parity) -> bool {
    uint32_t got = 1u;
    if (lane == 0) got = mbar_wait(bar, parity, abort_flag) ? 1u : 0u;
    return __shfl_sync(0xffffffffu, got, 0) != 0u;
  };
  // the k-blocks are dealt to the passes as evenly as possible: pass p covers [pass_first(p), pass_first(p) + pass_blocks(p))
  const int per_pass = k_blocks / passes, extra = k_blocks - per_pass * passes;
  auto pass_blocks = [&](int pass) { return per_pass + (pass < extra ? 1 : 0); };
  auto pass_first = [&](int pass) { return pass * per_pass + min(pass, extra); };

  if (warp == 0) {
    // ------------------------------------------------------------------ W producer
    if (lane == 0) {
      uint32_t it = 0;
      bool ok = true;
      for (int mb = blockIdx.x; mb < m_blocks && ok; mb += gridDim.x)
        for (int pass = 0; pass < passes && ok; ++pass)
          for (int nb = 0; nb < n_blocks && ok; ++nb)
            for (int j = 0; j < pass_blocks(pass); ++j, ++it) {
              const int s = it % kEgWStages;
              if (it == kEgWStages) pdl_wait();      // the next wait needs the consumer, hence the earlier kernels
              if (!mbar_wait(&w_empty[s], ((it / kEgWStages) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
              mbar_expect_tx(&w_full[s], kEgBBytes);
              tma_load_2d(wring + s * kEgBBytes, &p.tma_w, &w_full[s], (pass_first(pass) + j) * 64, nb * 256);
            }
      if (!ok) {
        const long long t0 = clock64();
        while (clock64() - t0 < 4000000) {}          // let loads in flight land before the CTA retires
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ UMMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc_bf16(128, 256, 0, 0);
      uint32_t it = 0, tcount = 0;                   // weight stages used, accumulators used
      uint32_t full_par = 0;                         // bit j: parity of slot j's next fill (slots are not all used in every pass)
      bool ok = true;
      for (int mb = blockIdx.x; mb < m_blocks && ok; mb += gridDim.x)
        for (int pass = 0; pass < passes && ok; ++pass) {
          const int nj = pass_blocks(pass);
          for (int nb = 0; nb < n_blocks && ok; ++nb, ++tcount) {
            const uint32_t acc = tcount & 1u;
            if (!mbar_wait(&acc_empty[acc], ((tcount >> 1) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
            tc_fence_after_sync();
            const uint32_t tmem_d = tmem_base + acc * 256;
            for (int j = 0; j < nj; ++j, ++it) {
              const int s = it % kEgWStages;
              // the first column block runs behind the gather; the others find every slot filled
              if (nb == 0) {
                if (!mbar_wait(&a_full[j], (full_par >> j) & 1u, abort_flag)) { ok = false; break; }
                full_par ^= 1u << j;
              }
              if (!mbar_wait(&w_full[s], (it / kEgWStages) & 1u, abort_flag)) { ok = false; break; }
              tc_fence_after_sync();
              const uint64_t adesc = make_smem_desc(smem_u32(smem + j * kEgABytes), 16, 1024, kSwizzle128B);
              const uint64_t bdesc = make_smem_desc(smem_u32(wring + s * kEgBBytes), 16, 1024, kSwizzle128B);
#pragma unroll
              for (int k = 0; k < 4; ++k) umma_bf16_ss(tmem_d, adesc + 2 * k, bdesc + 2 * k, idesc, (j | k) != 0);
              umma_commit(&w_empty[s]);
              if (nb == n_blocks - 1) umma_commit(&a_free[j]);   // the slot's last reader: the gather may refill it
            }
            if (ok) umma_commit(&acc_full[acc]);
          }
        }
    }
  } else if (warp < 2 + kEgGatherWarps) {
    // ------------------------------------------------------------------ gather: two threads per patch row
    const int t = threadIdx.x - 64;                 // 0..255
    const int row = t >> 1, half = t & 1;           // this thread writes 16-byte chunks 4 * half .. 4 * half + 3 of the row
    const int sw = row & 7;
    uint32_t used = 0, free_par = 0;                // bit j: slot j has been filled before; parity of its next hand-back
    bool ok = true;
    for (int mb = blockIdx.x; mb < m_blocks && ok; mb += gridDim.x) {
      const int m = mb * 128 + row;
      // this patch: first pixel of its top-left corner in frame-in-patch 0 of channel 0, and the strides
      const bf16* base = p.data;
      int plane_stride = 0, frame_stride = 0;       // elements between channels, and between frames of a clip (an item
      int W = 0;                                    // has fewer than 2^31 elements: checked by the host)
      const bool row_ok = m < p.n_patches;
      if (row_ok) {
        const int item = find_item(p.items.aux_start, p.items.n_items, m);
        const int local = m - p.items.aux_start[item];
        const int H = p.items.height[item];
        W = p.items.width[item];
        const int gh = H / p.patch, gw = W / p.patch;
        const int tt = local / (gh * gw);
        const int rem = local - tt * gh * gw;
        int r, c;
        if (p.merge_order) {
          const int grp = rem >> 2, within = rem & 3;
          const int hb = grp / (gw >> 1), wb = grp - hb * (gw >> 1);
          r = 2 * hb + (within >> 1);
          c = 2 * wb + (within & 1);
        } else {
          r = rem / gw;
          c = rem - r * gw;
        }
        plane_stride = H * W;
        const bool clip = p.tpatch > 1 || p.items.frames[item] > 1;
        frame_stride = clip ? plane_stride * p.channels : 0;
        base = p.data + p.items.offset[item] + static_cast<long long>(tt) * p.tpatch * frame_stride +
               static_cast<long long>(r) * p.patch * W + c * p.patch;
      }
      // the 16 pairs of this thread in k-block kb (registers only)
      auto load_block = [&](int kb, uint32_t (&v)[16]) {
        const uint4* tab4 = reinterpret_cast<const uint4*>(p.table + kb * 32 + half * 16);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const uint4 e4 = __ldg(tab4 + q);
          const uint32_t e[4] = {e4.x, e4.y, e4.z, e4.w};
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            uint32_t val = 0u;
            if (row_ok && e[j] != kEgPad) {
              const int ch = static_cast<int>(e[j] >> 24), f = static_cast<int>((e[j] >> 16) & 0xFFu);
              const int py = static_cast<int>((e[j] >> 8) & 0xFFu), px = static_cast<int>(e[j] & 0xFFu);
              const bf16* src = base + (f * frame_stride + ch * plane_stride + py * W + px);
              if (p.pairs_ok) {
                val = *reinterpret_cast<const uint32_t*>(src);
              } else {
                // odd geometry (odd patch edge, width or item offset): element loads; the second element of the pair
                // may belong to the next run
                const unsigned short lo = *reinterpret_cast<const unsigned short*>(src);
                int px1 = px + 1, py1 = py, f1 = f, ch1 = ch;
                if (px1 == p.patch) { px1 = 0; if (++py1 == p.patch) { py1 = 0; if (++f1 == p.tpatch) { f1 = 0; ++ch1; } } }
                unsigned short hi = 0;
                if (2 * (kb * 32 + half * 16 + q * 4 + j) + 1 < p.k)
                  hi = *reinterpret_cast<const unsigned short*>(base + (f1 * frame_stride + ch1 * plane_stride + py1 * W + px1));
                val = static_cast<uint32_t>(lo) | (static_cast<uint32_t>(hi) << 16);
              }
            }
            v[q * 4 + j] = val;
          }
        }
      };
      for (int pass = 0; pass < passes && ok; ++pass) {
        const int nj = pass_blocks(pass), kb0 = pass_first(pass);
        uint32_t cur[16], nxt[16];
        load_block(kb0, cur);
        for (int j = 0; j < nj; ++j) {
          if (j + 1 < nj) load_block(kb0 + j + 1, nxt);     // in flight while this one is stored
          // the slot's previous contents (an earlier pass or patch block) have been read by their last UMMA
          if ((used >> j) & 1u) {
            if (!warp_wait(&a_free[j], (free_par >> j) & 1u)) { ok = false; break; }
            free_par ^= 1u << j;
          }
          used |= 1u << j;
          uint8_t* srow = smem + j * kEgABytes + row * 128;
#pragma unroll
          for (int q = 0; q < 4; ++q)
            *reinterpret_cast<uint4*>(srow + (((half * 4 + q) ^ sw) << 4)) = make_uint4(cur[4 * q], cur[4 * q + 1], cur[4 * q + 2], cur[4 * q + 3]);
          fence_proxy_async_smem();               // generic-proxy stores -> visible to the tensor core's operand reads
          __syncwarp();
          if (lane == 0) mbar_arrive(&a_full[j]);
#pragma unroll
          for (int i = 0; i < 16; ++i) cur[i] = nxt[i];
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue
    const int quarter = warp & 3;                 // TMEM lane quarter this warp may read (warps 10..13 -> 2, 3, 0, 1)
    uint32_t tcount = 0;
    bool ok = true;
    for (int mb = blockIdx.x; mb < m_blocks && ok; mb += gridDim.x) {
      const int m = mb * 128 + quarter * 32 + lane;
      bool row_ok = m < p.n_patches;
      long long orow = 0;
      int posrow = 0;
      if (row_ok) {
        const int mapped = p.row_map[m];
        row_ok = mapped >= 0;
        orow = mapped;
        if (p.pos != nullptr) posrow = p.pos_idx[m];
      }
      for (int pass = 0; pass < passes && ok; ++pass)
        for (int nb = 0; nb < n_blocks && ok; ++nb, ++tcount) {
          const uint32_t acc = tcount & 1u;
          if (!warp_wait(&acc_full[acc], (tcount >> 1) & 1u)) { ok = false; break; }
          tc_fence_after_sync();
#pragma unroll 1
          for (int c = 0; c < 8; ++c) {
            const int col0 = nb * 256 + c * 32;
            uint32_t raw[32];
            __syncwarp();
            tmem_ld_32x32(tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + acc * 256 + c * 32, raw);
            tmem_ld_wait();
            if (!row_ok || col0 >= p.N) continue;
            float v[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(raw[i]);
            float4* o4 = reinterpret_cast<float4*>(p.x + orow * p.N + col0);
            if (pass == 0) {
              const uint4* bp = reinterpret_cast<const uint4*>(p.bias + col0);
              const uint4* pp = p.pos != nullptr ? reinterpret_cast<const uint4*>(p.pos + static_cast<long long>(posrow) * p.N + col0) : nullptr;
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                const uint4 b = __ldg(bp + q);
                const uint32_t wb[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) { v[q * 8 + 2 * j] += bf16_lo(wb[j]); v[q * 8 + 2 * j + 1] += bf16_hi(wb[j]); }
                if (pp != nullptr) {
                  const uint4 t4 = __ldg(pp + q);
                  const uint32_t wp[4] = {t4.x, t4.y, t4.z, t4.w};
#pragma unroll
                  for (int j = 0; j < 4; ++j) { v[q * 8 + 2 * j] += bf16_lo(wp[j]); v[q * 8 + 2 * j + 1] += bf16_hi(wp[j]); }
                }
              }
            } else {
              // a later pass over K: add to what the earlier passes stored (this thread wrote it: program order)
#pragma unroll
              for (int q = 0; q < 8; ++q) {
                const float4 r = o4[q];
                v[4 * q] += r.x; v[4 * q + 1] += r.y; v[4 * q + 2] += r.z; v[4 * q + 3] += r.w;
              }
            }
#pragma unroll
            for (int q = 0; q < 8; ++q) o4[q] = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
          }
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(&acc_empty[acc]);
        }
    }
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, 512);
  }
  if (threadIdx.x == 0 && *abort_flag) atomicCAS(p.status, DEV_OK, DEV_ERR_WAIT_TIMEOUT);
}

}  // namespace eas
