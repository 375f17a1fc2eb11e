// HBM-bound kernels of the encoder: row normalisation (LayerNorm / RMSNorm / plain cast) with an
// optional row gather, per-call tables (row maps, rotary table), audio staging, and the one-off weight
// re-layouts done at create time.  (Patch gathering is part of the embedding GEMM: embed_gemm.cuh.)
// All per-call kernels are persistent grid-stride loops launched with `sm_budget` CTAs.
#pragma once
#include "ptx.cuh"

namespace eas {

constexpr int kMaxItemsEw = 128;

// per-item geometry, passed by value in kernel parameters
struct ItemTable {
  int n_items;
  int tok_start[kMaxItemsEw + 1];   // encoder-token prefix (cu_seqlens)
  int aux_start[kMaxItemsEw + 1];   // family specific: patch-row prefix (ViT) or padded-frame prefix (audio)
  int frames[kMaxItemsEw];          // frames (video: raw frames; audio: mel frames)
  int height[kMaxItemsEw];
  int width[kMaxItemsEw];
  long long offset[kMaxItemsEw];    // element offset of the item in the packed input
};

__device__ __forceinline__ int find_item(const int* prefix, int n_items, int idx) {
  int lo = 0, hi = n_items - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (prefix[mid] <= idx) lo = mid; else hi = mid - 1;
  }
  return lo;
}

// ------------------------------------------------------------------------------- normalisation
enum { NORM_LN = 0, NORM_RMS = 1, NORM_CAST = 2 };

struct NormParams {
  const float* x;        // [*, d] fp32 residual stream
  void* y;               // [rows, d] bf16 or fp32
  const bf16* gamma;     // [d]
  const bf16* beta;      // [d] (LayerNorm only)
  const int* src_rows;   // optional gather: input row of each output row
  int rows, d;
  float eps;
  int reverse;           // 1: walk the rows last to first (see the row loop)
  // Split-K partial sums of the GEMM that produced x (see GemmParams::splits): n_part matrices [part_rows, d], added to
  // the row in index order before anything else; the completed row is written back to x_rw (== x).
  const float* part;
  long long part_stride; // elements between consecutive partial matrices
  int n_part;
  float* x_rw;
};

// One warp per row, the row held in registers (NV float4 per lane), two-pass statistics in fp32.
// PART: the launch adds split-K partial sums to the rows first (a kernel of its own: the ordinary one stays as lean as it was).
template <int NV, int KIND, bool OUT_FP32, bool PART = false>
__global__ void __launch_bounds__(512, 1) norm_kernel(const NormParams p) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int warps_per_cta = blockDim.x >> 5;
  float4 g[NV], b[NV];
  if (KIND != NORM_CAST) {
#pragma unroll
    for (int i = 0; i < NV; ++i) {
      const int c = i * 128 + lane * 4;
      const uint2 gv = __ldg(reinterpret_cast<const uint2*>(p.gamma + c));
      g[i] = make_float4(bf16_lo(gv.x), bf16_hi(gv.x), bf16_lo(gv.y), bf16_hi(gv.y));
      if (KIND == NORM_LN) {
        const uint2 bv = __ldg(reinterpret_cast<const uint2*>(p.beta + c));
        b[i] = make_float4(bf16_lo(bv.x), bf16_hi(bv.x), bf16_lo(bv.y), bf16_hi(bv.y));
      }
    }
  }
  const float inv_d = 1.0f / static_cast<float>(p.d);
  pdl_launch_dependents();
  pdl_wait();
  // The forward pass alternates the direction in which consecutive kernels walk the token rows: a kernel starts with
  // the rows its producer wrote last, which are the ones still in L2.  (Rows are independent: the order does not change
  // any value.)
  for (int rr = blockIdx.x * warps_per_cta + warp; rr < p.rows; rr += gridDim.x * warps_per_cta) {
    const int row = p.reverse ? p.rows - 1 - rr : rr;
    const long long src = p.src_rows ? p.src_rows[row] : row;
    const float4* xr = reinterpret_cast<const float4*>(p.x + src * p.d);
    float4 v[NV];
#pragma unroll
    for (int i = 0; i < NV; ++i) v[i] = __ldcs(xr + i * 32 + lane);    // streaming: the rows are not read again before they are rewritten
    if (PART) {
      for (int s = 0; s < p.n_part; ++s) {
        const float4* pr = reinterpret_cast<const float4*>(p.part + s * p.part_stride + src * p.d);
#pragma unroll
        for (int i = 0; i < NV; ++i) {
          const float4 t = pr[i * 32 + lane];
          v[i].x += t.x; v[i].y += t.y; v[i].z += t.z; v[i].w += t.w;
        }
      }
      float4* xw = reinterpret_cast<float4*>(p.x_rw + src * p.d);
#pragma unroll
      for (int i = 0; i < NV; ++i) xw[i * 32 + lane] = v[i];
    }
    float mean = 0.f, rstd = 1.f;
    if (KIND == NORM_LN) {
      float s = 0.f;
#pragma unroll
      for (int i = 0; i < NV; ++i) s += (v[i].x + v[i].y) + (v[i].z + v[i].w);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      mean = s * inv_d;
    }
    if (KIND != NORM_CAST) {
      float q = 0.f;
#pragma unroll
      for (int i = 0; i < NV; ++i) {
        const float a = v[i].x - mean, bq = v[i].y - mean, c = v[i].z - mean, e = v[i].w - mean;
        q += (a * a + bq * bq) + (c * c + e * e);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) q += __shfl_xor_sync(0xffffffffu, q, o);
      rstd = rsqrtf(q * inv_d + p.eps);
    }
#pragma unroll
    for (int i = 0; i < NV; ++i) {
      float4 r;
      if (KIND == NORM_CAST) {
        r = v[i];
      } else {
        r.x = (v[i].x - mean) * rstd * g[i].x; r.y = (v[i].y - mean) * rstd * g[i].y;
        r.z = (v[i].z - mean) * rstd * g[i].z; r.w = (v[i].w - mean) * rstd * g[i].w;
        if (KIND == NORM_LN) { r.x += b[i].x; r.y += b[i].y; r.z += b[i].z; r.w += b[i].w; }
      }
      if (OUT_FP32) {
        reinterpret_cast<float4*>(reinterpret_cast<float*>(p.y) + static_cast<long long>(row) * p.d)[i * 32 + lane] = r;
      } else {
        uint2 o2 = make_uint2(pack_bf16x2(r.x, r.y), pack_bf16x2(r.z, r.w));
        reinterpret_cast<uint2*>(reinterpret_cast<bf16*>(p.y) + static_cast<long long>(row) * p.d)[i * 32 + lane] = o2;
      }
    }
  }
}

// ------------------------------------------------------------------------------- folded normalisation: first producer
// What the residual GEMMs' folding epilogue writes for the rows it updates (GemmParams::fold_stats_out, fold_xb), for
// rows that come from somewhere else (the embedding): each row scaled by gamma and rounded to bf16 and, per group of 128
// columns, the mean and the sum of squared deviations from it (of the unscaled values).  One warp per row; lane l holds columns 128 i + 4 l ... + 3 of group i.
struct FoldStatsParams {
  const float* x;        // [rows, d]
  bf16* xb;              // [rows, d]
  float2* stats;         // [d / 128][rows]
  const bf16* gamma;     // [d]
  int rows, d;
};
template <int NV>
__global__ void __launch_bounds__(512, 1) fold_stats_kernel(const FoldStatsParams p) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int warps_per_cta = blockDim.x >> 5;
  float4 g[NV];
#pragma unroll
  for (int i = 0; i < NV; ++i) {
    const uint2 gv = __ldg(reinterpret_cast<const uint2*>(p.gamma + i * 128 + lane * 4));
    g[i] = make_float4(bf16_lo(gv.x), bf16_hi(gv.x), bf16_lo(gv.y), bf16_hi(gv.y));
  }
  pdl_launch_dependents();
  pdl_wait();
  for (int row = blockIdx.x * warps_per_cta + warp; row < p.rows; row += gridDim.x * warps_per_cta) {
    const float4* xr = reinterpret_cast<const float4*>(p.x + static_cast<long long>(row) * p.d);
    float4 v[NV];
#pragma unroll
    for (int i = 0; i < NV; ++i) v[i] = xr[i * 32 + lane];
#pragma unroll
    for (int i = 0; i < NV; ++i) {
      float s = (v[i].x + v[i].y) + (v[i].z + v[i].w);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      const float mean = s * (1.0f / 128.0f);
      const float a = v[i].x - mean, b = v[i].y - mean, c = v[i].z - mean, e = v[i].w - mean;
      float q = (a * a + b * b) + (c * c + e * e);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) q += __shfl_xor_sync(0xffffffffu, q, o);
      if (lane == 0) p.stats[static_cast<long long>(i) * p.rows + row] = make_float2(mean, q);
      reinterpret_cast<uint2*>(p.xb + static_cast<long long>(row) * p.d)[i * 32 + lane] =
          make_uint2(pack_bf16x2(v[i].x * g[i].x, v[i].y * g[i].y), pack_bf16x2(v[i].z * g[i].z, v[i].w * g[i].w));
    }
  }
}

// Create time: the two per-output constants of GemmParams::fold_stats for a linear layer that follows a normalisation.
// One warp per weight row.
struct FoldWeightsParams {
  const bf16* w;         // [n, k]
  const bf16* bias;      // [n]
  const bf16* gamma;     // [k]
  const bf16* beta;      // [k] or nullptr (RMSNorm)
  float* c0;             // [n]     bias[n] + sum_k beta_k * w[n, k]
  float* c1;             // [n]     sum_k gamma_k * w[n, k]
  int n, k;
};
__global__ void __launch_bounds__(256) fold_weights_kernel(const FoldWeightsParams p) {
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  const int n_warps = (gridDim.x * blockDim.x) >> 5;
  for (int row = warp; row < p.n; row += n_warps) {
    const bf16* wr = p.w + static_cast<long long>(row) * p.k;
    float s1 = 0.f, s0 = 0.f;
    for (int j = lane; j < p.k; j += 32) {
      const float w = __bfloat162float(wr[j]);
      s1 = fmaf(w, __bfloat162float(p.gamma[j]), s1);
      if (p.beta != nullptr) s0 = fmaf(w, __bfloat162float(p.beta[j]), s0);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) { s1 += __shfl_xor_sync(0xffffffffu, s1, o); s0 += __shfl_xor_sync(0xffffffffu, s0, o); }
    if (lane == 0) { p.c1[row] = s1; p.c0[row] = s0 + __bfloat162float(p.bias[row]); }
  }
}

// ------------------------------------------------------------------------------- per-call tables
struct PrepParams {
  ItemTable items;
  int family;             // 0 learned-position ViT, 1 RoPE ViT, 2 audio
  int has_cls;
  int patch;
  int d_model;
  int total_tokens;
  int n_embed_rows;       // rows of the embedding GEMM's A operand
  int rope_pairs;         // head_dim / 2 (RoPE only)
  float rope_theta;
  const int* cu_seqlens_dev;  // caller's device copy, checked against the host copy
  int* embed_row_map;     // [n_embed_rows] -> residual-stream row or -1
  int* embed_pos_idx;     // [n_embed_rows] -> position-table row
  int* head_src_rows;     // [out rows] (MLP projector: tokens without CLS)
  float2* rope_cs;        // [rope_pairs][total_tokens]: the GEMM epilogue's 32 rows of a warp read consecutive entries
  float* x;               // residual stream (CLS rows are written here)
  const bf16* cls;        // [d]
  const bf16* pos;        // [max_pos, d]
  int* conv1_row_map;     // audio: [padded frames] -> padded h1 row or -1
  int n_conv1_rows;
  uint32_t* status;
};

__global__ void __launch_bounds__(256) prep_kernel(const __grid_constant__ PrepParams p) {
  const int gtid = blockIdx.x * blockDim.x + threadIdx.x;
  const int gsz = gridDim.x * blockDim.x;
  const int n = p.items.n_items;
  pdl_launch_dependents();
  pdl_wait();
  if (p.cu_seqlens_dev != nullptr) {
    for (int i = gtid; i <= n; i += gsz)
      if (p.cu_seqlens_dev[i] != p.items.tok_start[i]) atomicCAS(p.status, DEV_OK, DEV_ERR_CU_SEQLENS_MISMATCH);
  }
  if (p.family == 0 || p.family == 1) {
    for (int m = gtid; m < p.n_embed_rows; m += gsz) {
      const int it = find_item(p.items.aux_start, n, m);
      const int local = m - p.items.aux_start[it];
      p.embed_row_map[m] = p.items.tok_start[it] + local + (p.has_cls ? 1 : 0);
      p.embed_pos_idx[m] = local + (p.has_cls ? 1 : 0);
    }
  }
  if (p.family == 0 && p.has_cls) {
    for (int i = gtid; i < n * p.d_model; i += gsz) {
      const int it = i / p.d_model, c = i - it * p.d_model;
      p.x[static_cast<long long>(p.items.tok_start[it]) * p.d_model + c] =
          __bfloat162float(p.cls[c]) + __bfloat162float(p.pos[c]);
    }
    if (p.head_src_rows != nullptr) {
      const int out_rows = p.total_tokens - n;
      for (int o = gtid; o < out_rows; o += gsz) {
        const int it = find_item(p.items.aux_start, n, o);   // aux_start is also the prefix of tokens without CLS
        p.head_src_rows[o] = o + it + 1;
      }
    }
  }
  if (p.family == 1) {
    // (cos, sin) of the rotary angles.  Pair i < pairs/2 turns with the token's grid row and frequency
    // theta^(-i/(pairs/2)); pair i >= pairs/2 with the grid column and frequency theta^(-(i-pairs/2)/(pairs/2)).
    const int P = p.patch;
    const int nf = p.rope_pairs >> 1;
    const long long total = static_cast<long long>(p.total_tokens) * p.rope_pairs;
    for (long long idx = gtid; idx < total; idx += gsz) {
      const int tok = static_cast<int>(idx / p.rope_pairs);
      const int i = static_cast<int>(idx - static_cast<long long>(tok) * p.rope_pairs);
      const int it = find_item(p.items.tok_start, n, tok);
      const int gh = p.items.height[it] / P, gw = p.items.width[it] / P;
      const int rem = (tok - p.items.tok_start[it]) % (gh * gw);
      const int grp = rem >> 2, within = rem & 3;
      const int hb = grp / (gw >> 1), wb = grp - hb * (gw >> 1);
      const int r = 2 * hb + (within >> 1), c = 2 * wb + (within & 1);
      const int fi = i < nf ? i : i - nf;
      const float freq = exp2f(-log2f(p.rope_theta) * static_cast<float>(fi) / static_cast<float>(nf));
      const float ang = static_cast<float>(i < nf ? r : c) * freq;
      float sn, cs;
      sincosf(ang, &sn, &cs);
      p.rope_cs[static_cast<long long>(i) * p.total_tokens + tok] = make_float2(cs, sn);   // [pair][token]
    }
  }
  if (p.family == 2) {
    // conv1 walks padded frame rows (one zero row before and after each item); row t of an item
    // lands in padded h1 row t + 1; the two window positions that straddle items are dropped.
    for (int m = gtid; m < p.n_conv1_rows; m += gsz) {
      const int it = find_item(p.items.aux_start, n, m);
      const int t = m - p.items.aux_start[it];
      p.conv1_row_map[m] = t < p.items.frames[it] ? m + 1 : -1;
    }
    // conv2 walks (ceil(frames/2) + 1) rows per item; the last one is dropped
    for (int m = gtid; m < p.n_embed_rows; m += gsz) {
      // aux_start[i] / 2 is the conv2 row prefix because every padded item has an even row count
      int lo = 0, hi = n - 1;
      while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if ((p.items.aux_start[mid] >> 1) <= m) lo = mid; else hi = mid - 1;
      }
      const int t = m - (p.items.aux_start[lo] >> 1);
      const bool ok = t < ((p.items.frames[lo] + 1) >> 1);
      p.embed_row_map[m] = ok ? p.items.tok_start[lo] + t : -1;
      p.embed_pos_idx[m] = ok ? t : 0;
    }
  }
}

// audio: copy mel frames into a staging buffer with one zero row before and one (odd frame counts: two) after each
// item, and zero the matching pad rows of the h1 staging buffer
struct AudioStageParams {
  const bf16* data;
  bf16* mel_pad;       // [padded rows, n_mel]
  bf16* h1_pad;        // [padded rows, d]
  int n_mel, d_model, padded_rows;
  ItemTable items;     // aux_start = padded-row prefix
};

__global__ void __launch_bounds__(512, 1) audio_stage_kernel(const __grid_constant__ AudioStageParams p) {
  const long long total = static_cast<long long>(p.padded_rows) * p.n_mel;
  const long long gsz = static_cast<long long>(gridDim.x) * blockDim.x;
  pdl_launch_dependents();
  pdl_wait();
  for (long long idx = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; idx < total; idx += gsz) {
    const int m = static_cast<int>(idx / p.n_mel);
    const int c = static_cast<int>(idx - static_cast<long long>(m) * p.n_mel);
    const int it = find_item(p.items.aux_start, p.items.n_items, m);
    const int t = m - p.items.aux_start[it] - 1;
    bf16 v = __float2bfloat16(0.f);
    if (t >= 0 && t < p.items.frames[it]) v = p.data[p.items.offset[it] + static_cast<long long>(t) * p.n_mel + c];
    p.mel_pad[idx] = v;
  }
  // pad rows of h1: the item's first staging row and every row behind its last frame (one, or two for an odd count)
  const long long pad_total = static_cast<long long>(p.items.n_items) * 3 * p.d_model;
  for (long long idx = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; idx < pad_total; idx += gsz) {
    const int c = static_cast<int>(idx % p.d_model);
    const int which = static_cast<int>(idx / p.d_model);
    const int it = which / 3, k = which - it * 3;
    const int row = k == 0 ? p.items.aux_start[it] : p.items.aux_start[it + 1] - k;
    if (k == 2 && (p.items.frames[it] & 1) == 0) continue;      // even count: that row holds the last frame
    p.h1_pad[static_cast<long long>(row) * p.d_model + c] = __float2bfloat16(0.f);
  }
}

// ------------------------------------------------------------------------------- create-time re-layouts
// dst[r, 0:k_pad] = src[perm(r), 0:k] zero padded, r < rows.  mode 0: identity; mode 1: rotary pairing
// (within each head of the first `rope_rows` rows: new 2i <- old i, new 2i+1 <- old i + hd/2);
// mode 2: gate/up interleave (new 2j <- gate j, new 2j+1 <- up j; src = gate, src2 = up).
struct RelayoutParams {
  const bf16* src; const bf16* src2; bf16* dst;
  long long rows; int k, k_pad; int mode; int head_dim; long long rope_rows;
};
__global__ void relayout_kernel(const RelayoutParams p) {
  const long long total = p.rows * p.k_pad;
  for (long long idx = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; idx < total;
       idx += static_cast<long long>(gridDim.x) * blockDim.x) {
    const long long r = idx / p.k_pad;
    const int c = static_cast<int>(idx - r * p.k_pad);
    bf16 v = __float2bfloat16(0.f);
    if (c < p.k) {
      if (p.mode == 0) {
        v = p.src[r * p.k + c];
      } else if (p.mode == 1) {
        long long sr = r;
        if (r < p.rope_rows) {
          const long long head = r / p.head_dim;
          const int w = static_cast<int>(r - head * p.head_dim);
          sr = head * p.head_dim + (w >> 1) + (w & 1) * (p.head_dim >> 1);
        }
        v = p.src[sr * p.k + c];
      } else {
        const bf16* s = (r & 1) ? p.src2 : p.src;
        v = s[(r >> 1) * p.k + c];
      }
    }
    p.dst[idx] = v;
  }
}

}  // namespace eas
