// Block-diagonal (variable-length) softmax attention, register-tile version on mma.sync.
// One work unit = (item, head, 128 query rows); keys and values are taken from the SAME item only,
// so nothing is ever read across an item boundary.  Online softmax in fp32, P rounded to bf16 for P*V.
// Persistent: gridDim.x = sm_budget CTAs walk units  blockIdx.x, +gridDim.x, ...  in a fixed order.
#pragma once
#include "ptx.cuh"

namespace eas {

constexpr int kMaxItems = 128;
constexpr int kAttnBQ = 128;        // query rows per unit
constexpr int kAttnBKV = 64;        // keys per inner step
constexpr int kAttnThreads = 256;   // 8 warps x 16 query rows

struct AttnParams {
  const bf16* qkv;        // [T, ld]: Q | K | V thirds, head h at columns h*hd within its third
  bf16* out;              // [T, ldo]
  long long ld, ldo;
  int d_model, n_heads;
  float scale_log2;       // log2(e) / sqrt(head_dim)
  int n_items;
  int total_units;
  int item_start[kMaxItems];     // first token row of the item (in schedule order)
  int item_len[kMaxItems];
  int unit_prefix[kMaxItems + 1];  // units before item i (schedule order: longest items first)
};

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc, bool valid) {
  const int sz = valid ? 16 : 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_u32(smem_dst)), "l"(gsrc), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

template <int HD>
constexpr int attn_mma_smem_bytes() { return (kAttnBQ + 4 * kAttnBKV) * (HD + 8) * 2; }

template <int HD>
__global__ void __launch_bounds__(kAttnThreads, 1) attn_mma_kernel(const __grid_constant__ AttnParams p) {
  constexpr int LDS = HD + 8;              // padded row (elements): conflict-free ldmatrix
  constexpr int CH = HD / 8;               // 16-byte chunks per row
  constexpr int KS = HD / 16;              // k-steps of Q*K^T
  constexpr int NT_O = HD / 8;             // 8-wide output column tiles
  extern __shared__ __align__(16) uint8_t smem_attn[];
  bf16* sQ = reinterpret_cast<bf16*>(smem_attn);
  bf16* sK = sQ + kAttnBQ * LDS;           // [2][64][LDS]
  bf16* sV = sK + 2 * kAttnBKV * LDS;      // [2][64][LDS]

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  pdl_launch_dependents();
  pdl_wait();

  for (int unit = blockIdx.x; unit < p.total_units; unit += gridDim.x) {
    // decode (item, head, q-tile); q-tile varies fastest so that neighbours share K and V in L2
    int lo = 0, hi = p.n_items - 1;
    while (lo < hi) {
      const int mid = (lo + hi + 1) >> 1;
      if (p.unit_prefix[mid] <= unit) lo = mid; else hi = mid - 1;
    }
    const int item = lo;
    const int S = p.item_len[item];
    const int nq = (S + kAttnBQ - 1) / kAttnBQ;
    const int r = unit - p.unit_prefix[item];
    const int head = r / nq;
    const int q0 = (r - head * nq) * kAttnBQ;
    const long long row0 = p.item_start[item];
    const bf16* gQ = p.qkv + row0 * p.ld + head * HD;
    const bf16* gK = gQ + p.d_model;
    const bf16* gV = gQ + 2 * p.d_model;
    const int n_kv = (S + kAttnBKV - 1) / kAttnBKV;

    __syncthreads();   // previous unit's shared memory is no longer read
    for (int c = tid; c < kAttnBQ * CH; c += kAttnThreads) {
      const int rr = c / CH, cc = c - rr * CH;
      const bool v = (q0 + rr) < S;
      cp_async16(sQ + rr * LDS + cc * 8, gQ + static_cast<long long>(v ? q0 + rr : 0) * p.ld + cc * 8, v);
    }
    auto load_kv = [&](int t, int buf) {
      const int k0 = t * kAttnBKV;
      for (int c = tid; c < kAttnBKV * CH; c += kAttnThreads) {
        const int rr = c / CH, cc = c - rr * CH;
        const bool v = (k0 + rr) < S;
        const long long off = static_cast<long long>(v ? k0 + rr : 0) * p.ld + cc * 8;
        cp_async16(sK + (buf * kAttnBKV + rr) * LDS + cc * 8, gK + off, v);
        cp_async16(sV + (buf * kAttnBKV + rr) * LDS + cc * 8, gV + off, v);
      }
    };
    load_kv(0, 0);
    cp_async_commit();

    uint32_t qf[KS][4];
    float o[NT_O][4];
#pragma unroll
    for (int j = 0; j < NT_O; ++j) { o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.f; }
    float m_run[2] = {-INFINITY, -INFINITY};
    float l_run[2] = {0.f, 0.f};

    for (int t = 0; t < n_kv; ++t) {
      const int buf = t & 1;
      if (t + 1 < n_kv) load_kv(t + 1, buf ^ 1);
      cp_async_commit();
      cp_async_wait<1>();
      __syncthreads();
      if (t == 0) {
#pragma unroll
        for (int k = 0; k < KS; ++k) {
          const uint32_t a = smem_u32(sQ + (warp * 16 + (lane & 15)) * LDS + k * 16 + (lane >> 4) * 8);
          ldsm_x4(a, qf[k][0], qf[k][1], qf[k][2], qf[k][3]);
        }
      }
      // S = Q K^T : 16 x 64 per warp
      float s[8][4];
#pragma unroll
      for (int j = 0; j < 8; ++j) { s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f; }
      const bf16* kb = sK + buf * kAttnBKV * LDS;
#pragma unroll
      for (int k = 0; k < KS; ++k) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {      // pairs of 8-key tiles
          uint32_t b0, b1, b2, b3;
          const uint32_t a = smem_u32(kb + (j * 16 + (lane & 7) + (lane >> 4) * 8) * LDS + k * 16 + ((lane >> 3) & 1) * 8);
          ldsm_x4(a, b0, b1, b2, b3);
          mma_bf16_16816(s[2 * j], qf[k], b0, b1);
          mma_bf16_16816(s[2 * j + 1], qf[k], b2, b3);
        }
      }
      // mask keys past the end of the item (only the last step can have any)
      const int k0 = t * kAttnBKV;
      if (k0 + kAttnBKV > S) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int key = k0 + j * 8 + (lane & 3) * 2;
          if (key >= S) { s[j][0] = -INFINITY; s[j][2] = -INFINITY; }
          if (key + 1 >= S) { s[j][1] = -INFINITY; s[j][3] = -INFINITY; }
        }
      }
      // online softmax for rows (lane/4) and (lane/4 + 8)
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        float mx = -INFINITY;
#pragma unroll
        for (int j = 0; j < 8; ++j) mx = fmaxf(mx, fmaxf(s[j][2 * h], s[j][2 * h + 1]));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        const float m_new = fmaxf(m_run[h], mx);
        const float corr = fast_ex2((m_run[h] - m_new) * p.scale_log2);   // first step: ex2(-inf) = 0
        const float mb = m_new * p.scale_log2;
        float sum = 0.f;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const float p0 = fast_ex2(fmaf(s[j][2 * h], p.scale_log2, -mb));
          const float p1 = fast_ex2(fmaf(s[j][2 * h + 1], p.scale_log2, -mb));
          s[j][2 * h] = p0; s[j][2 * h + 1] = p1;
          sum += p0 + p1;
        }
        l_run[h] = l_run[h] * corr + sum;
        m_run[h] = m_new;
#pragma unroll
        for (int j = 0; j < NT_O; ++j) { o[j][2 * h] *= corr; o[j][2 * h + 1] *= corr; }
      }
      // O += P V
      const bf16* vb = sV + buf * kAttnBKV * LDS;
#pragma unroll
      for (int kk = 0; kk < kAttnBKV / 16; ++kk) {
        uint32_t pa[4];
        pa[0] = pack_bf16x2(s[2 * kk][0], s[2 * kk][1]);
        pa[1] = pack_bf16x2(s[2 * kk][2], s[2 * kk][3]);
        pa[2] = pack_bf16x2(s[2 * kk + 1][0], s[2 * kk + 1][1]);
        pa[3] = pack_bf16x2(s[2 * kk + 1][2], s[2 * kk + 1][3]);
#pragma unroll
        for (int j = 0; j < NT_O / 2; ++j) {
          uint32_t b0, b1, b2, b3;
          const uint32_t a = smem_u32(vb + (kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8) * LDS + j * 16 + (lane >> 4) * 8);
          ldsm_x4_t(a, b0, b1, b2, b3);
          mma_bf16_16816(o[2 * j], pa, b0, b1);
          mma_bf16_16816(o[2 * j + 1], pa, b2, b3);
        }
      }
      __syncthreads();   // this buffer may be refilled two steps from now
    }
    cp_async_wait<0>();

    // finalise: divide by the row sums (summed over the 4 lanes of a quad) and store
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      float l = l_run[h];
      l += __shfl_xor_sync(0xffffffffu, l, 1);
      l += __shfl_xor_sync(0xffffffffu, l, 2);
      const float inv = 1.0f / l;
      const int qrow = q0 + warp * 16 + (lane >> 2) + h * 8;
      if (qrow < S) {
        bf16* orow = p.out + (row0 + qrow) * p.ldo + head * HD + (lane & 3) * 2;
#pragma unroll
        for (int j = 0; j < NT_O; ++j) {
          *reinterpret_cast<uint32_t*>(orow + j * 8) = pack_bf16x2(o[j][2 * h] * inv, o[j][2 * h + 1] * inv);
        }
      }
    }
  }
}

}  // namespace eas
