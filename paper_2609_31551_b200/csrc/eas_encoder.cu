// C ABI of the Encode-stage library: handle, weight re-layout, workspace plan, and the launch
// sequence of one micro-batch forward pass.  All arithmetic runs in the kernels included below.
#include "../../include/eas_encoder.h"

#include <cuda.h>
#include <cuda_runtime.h>
#include <cudaTypedefs.h>

#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <map>
#include <memory>
#include <mutex>
#include <string>
#include <vector>

#include "attention_mma.cuh"
#include "attention_tc.cuh"
#include "elementwise.cuh"
#include "embed_gemm.cuh"
#include "gemm.cuh"

using namespace eas;

// ------------------------------------------------------------------------------------ errors
static thread_local char g_err[512] = "";
static eas_status fail(eas_status s, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
  return s;
}
#define CUDA_TRY(expr)                                                                              \
  do {                                                                                              \
    cudaError_t e_ = (expr);                                                                        \
    if (e_ != cudaSuccess) return fail(EAS_ERR_CUDA, "%s failed: %s", #expr, cudaGetErrorString(e_)); \
  } while (0)

extern "C" const char* eas_last_error(void) { return g_err; }

// ------------------------------------------------------------------------------------ tensor maps
static PFN_cuTensorMapEncodeTiled_v12000 get_encode_fn() {
  static PFN_cuTensorMapEncodeTiled_v12000 fn = nullptr;
  if (fn == nullptr) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(p);
  }
  return fn;
}

// bf16 tensor map.  dims/strides innermost first; strides (bytes) for dims 1..rank-1.
static eas_status make_tmap(CUtensorMap* m, const void* base, int rank, const uint64_t* dims, const uint64_t* strides,
                            const uint32_t* box, CUtensorMapSwizzle swz) {
  PFN_cuTensorMapEncodeTiled_v12000 fn = get_encode_fn();
  if (fn == nullptr) return fail(EAS_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
  cuuint64_t gdim[5], gstr[5];
  cuuint32_t bx[5], es[5];
  for (int i = 0; i < rank; ++i) { gdim[i] = dims[i]; bx[i] = box[i]; es[i] = 1; }
  for (int i = 0; i + 1 < rank; ++i) gstr[i] = strides[i];
  CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, rank, const_cast<void*>(base), gdim, gstr, bx, es,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(EAS_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", static_cast<int>(r));
  return EAS_OK;
}

// W [N, K] row-major -> 2-D map, box 64 x `box_rows` (256: one CTA loads the whole weight tile; 128: half of it)
static eas_status make_w_tmap(CUtensorMap* m, const void* w, int64_t N, int64_t K, uint32_t box_rows) {
  const uint64_t dims[2] = {static_cast<uint64_t>(K), static_cast<uint64_t>(N)};
  const uint64_t strides[1] = {static_cast<uint64_t>(K) * 2};
  const uint32_t box[2] = {kBK, box_rows};
  return make_tmap(m, w, 2, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B);
}
// A as {run, phase, rows}: a plain [M, K] matrix is {K, 1, M}; a k=3 convolution over rows of width C with row
// stride s is {C, s, rows/s} and the kernel walks taps as extra k-blocks
static eas_status make_a_tmap(CUtensorMap* m, const void* a, int64_t run, int64_t row_elems, int conv_stride, int64_t rows) {
  const uint64_t dims[3] = {static_cast<uint64_t>(run), static_cast<uint64_t>(conv_stride),
                            static_cast<uint64_t>((rows + conv_stride - 1) / conv_stride)};
  const uint64_t strides[2] = {static_cast<uint64_t>(row_elems) * 2, static_cast<uint64_t>(row_elems) * 2 * conv_stride};
  const uint32_t box[3] = {kBK, 1, kBM};
  return make_tmap(m, a, 3, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B);
}

// "Deep" maps: the same matrices seen as {64 columns, rows, K/64 blocks}, so that ONE box {64, rows, 2} brings two
// 64-wide k-blocks, each landing as its own swizzle-atom block [rows x 128 bytes] (see GemmCfg).  A k-block index
// past K/64 is filled with zeros.
static eas_status make_w_tmap_deep(CUtensorMap* m, const void* w, int64_t N, int64_t K, uint32_t box_rows) {
  const uint64_t dims[3] = {kBK, static_cast<uint64_t>(N), static_cast<uint64_t>(K / kBK)};
  const uint64_t strides[2] = {static_cast<uint64_t>(K) * 2, kBK * 2};
  const uint32_t box[3] = {kBK, box_rows, 2};
  return make_tmap(m, w, 3, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B);
}
static eas_status make_a_tmap_deep(CUtensorMap* m, const void* a, int64_t run, int64_t row_elems, int64_t rows) {
  const uint64_t dims[3] = {kBK, static_cast<uint64_t>(rows), static_cast<uint64_t>(run / kBK)};
  const uint64_t strides[2] = {static_cast<uint64_t>(row_elems) * 2, kBK * 2};
  const uint32_t box[3] = {kBK, kBM, 2};
  return make_tmap(m, a, 3, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B);
}

// output [rows, ld] as a store / reduce target: 32-row boxes whose rows are 128 bytes (64 bf16 or 32 fp32)
static eas_status make_out_tmap(CUtensorMap* m, const void* out, bool fp32, int64_t cols, int64_t ld, int64_t rows) {
  PFN_cuTensorMapEncodeTiled_v12000 fn = get_encode_fn();
  if (fn == nullptr) return fail(EAS_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
  const cuuint64_t gdim[2] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows)};
  const cuuint64_t gstr[1] = {static_cast<cuuint64_t>(ld) * (fp32 ? 4 : 2)};
  const cuuint32_t box[2] = {fp32 ? 32u : 64u, 32u};
  const cuuint32_t es[2] = {1, 1};
  CUresult r = fn(m, fp32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(out),
                  gdim, gstr, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                  CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(EAS_ERR_CUDA, "cuTensorMapEncodeTiled (output) failed with code %d", static_cast<int>(r));
  return EAS_OK;
}

// ------------------------------------------------------------------------------------ handle
struct Linear {
  const bf16* w = nullptr;   // [N, K] (possibly re-laid)
  const bf16* b = nullptr;   // [N]
  int N = 0, K = 0;
  CUtensorMap tmap;        // box of 256 weight rows
  CUtensorMap tmap_half;   // box of 128 weight rows (CTA-pair kernel)
  CUtensorMap tmap_deep, tmap_half_deep;   // the same for the deep kernels (two k-blocks per box)
};
struct Layer {
  const bf16 *n1g = nullptr, *n1b = nullptr, *n2g = nullptr, *n2b = nullptr;
  Linear qkv, proj, fc1, fc2;
  // folded normalisation (GemmParams::fold_stats): the two per-output constants of the qkv and MLP-up layers
  const float *qkv_c0 = nullptr, *qkv_c1 = nullptr, *fc1_c0 = nullptr, *fc1_c1 = nullptr;
};

// One captured forward pass: every launch of a micro-batch with exactly these shapes, pointers and SM budget.
struct GraphEntry {
  std::vector<int64_t> key;
  cudaGraphExec_t exec = nullptr;
  int launches = 0;
  uint32_t* status = nullptr;
  uint64_t last_use = 0;
};
constexpr size_t kMaxGraphs = 16;

struct eas_encoder {
  eas_arch_config cfg;
  int device = 0;             // ordinal of the device that was current at create: weights, tensor maps and kernel attributes belong to it
  int sm_count = 0;
  int hd = 0;
  int embed_k = 0, embed_k_pad = 0;
  const uint32_t* embed_table = nullptr;   // where each pixel pair of a patch vector comes from (embed_gemm.cuh)
  Linear embed, conv1, conv2, head1, head2;
  const bf16 *cls = nullptr, *pos = nullptr, *eng = nullptr, *enb = nullptr, *fng = nullptr, *fnb = nullptr, *hng = nullptr;
  std::vector<Layer> layers;
  int attn_impl = 0;
  int split_k = 0;            // small micro-batches split the K loop of the residual GEMMs (eas_encoder_set_split_k)
  int fold = 0;               // 1: the blocks' normalisations are folded into the GEMMs around them (eas_encoder_set_norm_fold)
  int last_launches = 0;
  uint32_t* last_status = nullptr;
  // optional per-kernel timing: one event before every launch and one after the last
  bool timing = false;
  std::vector<cudaEvent_t> tev;
  std::vector<int> tcls;
  // optional replay of captured forward passes (small micro-batches are bound by launch overhead)
  int graph_mode = 0;
  std::vector<GraphEntry> graphs;
  uint64_t graph_clock = 0;
  int64_t graph_hits = 0, graph_captures = 0;
  ~eas_encoder() {
    for (cudaEvent_t ev : tev) cudaEventDestroy(ev);
    for (GraphEntry& g : graphs) if (g.exec) cudaGraphExecDestroy(g.exec);
  }
};

// records an event in front of the next launch when timing is on; cls < 0 closes the sequence
static eas_status mark(eas_encoder* e, int cls, cudaStream_t stream) {
  if (!e->timing) return EAS_OK;
  const size_t i = e->tcls.size();
  if (i >= e->tev.size()) {
    cudaEvent_t ev;
    CUDA_TRY(cudaEventCreate(&ev));
    e->tev.push_back(ev);
  }
  CUDA_TRY(cudaEventRecord(e->tev[i], stream));
  e->tcls.push_back(cls);
  return EAS_OK;
}

static size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

static eas_status check_cfg(const eas_arch_config* c) {
  if (c == nullptr) return fail(EAS_ERR_INVALID_ARG, "arch config is null");
  if (c->family < 0 || c->family > 2) return fail(EAS_ERR_INVALID_ARG, "unknown family %d", c->family);
  if (c->n_layers < 0 || c->d_model <= 0 || c->n_heads <= 0 || c->d_mlp <= 0)
    return fail(EAS_ERR_INVALID_ARG, "non-positive model dimension");
  if (c->d_model % c->n_heads != 0) return fail(EAS_ERR_INVALID_ARG, "d_model %% n_heads != 0");
  const int hd = c->d_model / c->n_heads;
  if (hd != 64 && hd != 80) return fail(EAS_ERR_UNSUPPORTED, "head_dim %d (supported: 64, 80)", hd);
  if (c->d_model % 128 != 0 || c->d_model > 2048) return fail(EAS_ERR_UNSUPPORTED, "d_model must be a multiple of 128, at most 2048");
  if (c->d_mlp % 64 != 0) return fail(EAS_ERR_UNSUPPORTED, "d_mlp must be a multiple of 64");
  if (c->norm != EAS_NORM_LAYERNORM && c->norm != EAS_NORM_RMSNORM) return fail(EAS_ERR_INVALID_ARG, "unknown norm");
  if (c->mlp != EAS_MLP_GELU && c->mlp != EAS_MLP_SWIGLU) return fail(EAS_ERR_INVALID_ARG, "unknown mlp");
  if (c->pos != EAS_POS_TABLE && c->pos != EAS_POS_ROPE_2D) return fail(EAS_ERR_INVALID_ARG, "unknown position scheme");
  if (c->head < 0 || c->head > 2) return fail(EAS_ERR_INVALID_ARG, "unknown head");
  if (c->in_channels <= 0 || c->patch <= 0 || c->temporal_patch <= 0) return fail(EAS_ERR_INVALID_ARG, "bad input geometry");
  if (c->family == EAS_FAMILY_VIT_LEARNED && (c->pos != EAS_POS_TABLE || c->max_pos <= 0))
    return fail(EAS_ERR_INVALID_ARG, "learned-position ViT needs a position table");
  if (c->family == EAS_FAMILY_VIT_ROPE_MERGER && (c->pos != EAS_POS_ROPE_2D || c->head != EAS_HEAD_MERGER_2X2 || c->has_cls))
    return fail(EAS_ERR_INVALID_ARG, "RoPE ViT needs 2-D rotary positions, the 2x2 merger and no CLS");
  if (c->family == EAS_FAMILY_AUDIO_CONV && (c->pos != EAS_POS_TABLE || c->has_cls || c->in_channels % 64 != 0 || c->head != EAS_HEAD_NONE))
    return fail(EAS_ERR_INVALID_ARG, "audio encoder needs a position table, mel bins %% 64 == 0, no CLS, no head");
  if (c->pos == EAS_POS_ROPE_2D && (hd % 4 != 0 || c->rope_theta <= 1.0f)) return fail(EAS_ERR_INVALID_ARG, "bad rotary setup");
  if (c->head != EAS_HEAD_NONE && (c->d_head_hidden <= 0 || c->d_head_hidden % 64 != 0 || c->d_out % 32 != 0))
    return fail(EAS_ERR_UNSUPPORTED, "connector widths must be multiples of 64 (hidden) and 32 (out)");
  if (c->head == EAS_HEAD_NONE && c->d_out != c->d_model) return fail(EAS_ERR_INVALID_ARG, "d_out must equal d_model without a head");
  if (c->head == EAS_HEAD_MLP_PROJECTOR && c->final_norm) return fail(EAS_ERR_UNSUPPORTED, "projector after a final norm");
  if (c->out_dtype != EAS_OUT_BF16 && c->out_dtype != EAS_OUT_FP32) return fail(EAS_ERR_INVALID_ARG, "unknown out_dtype %d", c->out_dtype);
  return EAS_OK;
}

static int embed_k_of(const eas_arch_config* c) { return c->in_channels * c->temporal_patch * c->patch * c->patch; }

extern "C" size_t eas_encoder_weight_arena_bytes(const eas_arch_config* c) {
  if (check_cfg(c) != EAS_OK) return 0;
  size_t total = 1024;
  const size_t d = c->d_model, I = c->d_mlp;
  if (c->family != EAS_FAMILY_AUDIO_CONV)   // padded patch matrix + the embedding kernel's pair table
    total += align_up(d * align_up(embed_k_of(c), 64) * 2, 1024) + align_up(align_up(embed_k_of(c), 64) * 2, 1024);
  if (c->pos == EAS_POS_ROPE_2D) total += c->n_layers * (align_up(3 * d * d * 2, 1024) + align_up(3 * d * 2, 1024));
  if (c->mlp == EAS_MLP_SWIGLU) total += c->n_layers * (align_up(2 * I * d * 2, 1024) + align_up(2 * I * 2, 1024));
  // folded normalisation: two fp32 constants per output of the qkv and MLP-up layers
  const size_t n1 = c->mlp == EAS_MLP_SWIGLU ? 2 * I : I;
  total += c->n_layers * (2 * align_up(3 * d * 4, 1024) + 2 * align_up(n1 * 4, 1024));
  return total;
}

namespace {
struct WeightIndex {
  std::map<std::string, const eas_tensor*> by_name;
  eas_status get(const std::string& name, std::initializer_list<int64_t> shape, const bf16** out) const {
    auto it = by_name.find(name);
    if (it == by_name.end()) return fail(EAS_ERR_INVALID_ARG, "weight '%s' is missing", name.c_str());
    const eas_tensor* t = it->second;
    if (t->dev_ptr == nullptr || (reinterpret_cast<uintptr_t>(t->dev_ptr) & 15) != 0)
      return fail(EAS_ERR_INVALID_ARG, "weight '%s' has a null or unaligned pointer", name.c_str());
    if (t->ndim != static_cast<int>(shape.size())) return fail(EAS_ERR_INVALID_ARG, "weight '%s' has rank %d", name.c_str(), t->ndim);
    int i = 0;
    for (int64_t s : shape) {
      if (t->shape[i] != s)
        return fail(EAS_ERR_INVALID_ARG, "weight '%s' dim %d is %lld, expected %lld", name.c_str(), i,
                    static_cast<long long>(t->shape[i]), static_cast<long long>(s));
      ++i;
    }
    *out = static_cast<const bf16*>(t->dev_ptr);
    return EAS_OK;
  }
};

struct Arena {
  uint8_t* base; size_t size; size_t used = 0;
  void* take(size_t bytes) {
    const size_t off = align_up(used, 1024);
    if (off + bytes > size) return nullptr;
    used = off + bytes;
    return base + off;
  }
};
}  // namespace

static eas_status relayout(bf16* dst, const bf16* src, const bf16* src2, long long rows, int k, int k_pad, int mode,
                           int head_dim, long long rope_rows) {
  RelayoutParams rp{src, src2, dst, rows, k, k_pad, mode, head_dim, rope_rows};
  const long long total = rows * k_pad;
  const int blocks = static_cast<int>(std::min<long long>((total + 255) / 256, 4096));
  relayout_kernel<<<blocks, 256>>>(rp);
  CUDA_TRY(cudaGetLastError());
  return EAS_OK;
}

#define EAS_TRY(expr)            \
  do {                           \
    eas_status s_ = (expr);      \
    if (s_ != EAS_OK) return s_; \
  } while (0)

// Kernel attributes (the dynamic shared-memory limit) belong to a device's context: they are set once per DEVICE, the
// first time a launch site is reached with that device current.
struct OncePerDevice {
  std::mutex m;
  bool done[64] = {};
  // true until settled() has been called with this device current (always true for ordinals past the table: the
  // attribute is then set every time).  A failed attribute call returns before settled(), so the next launch retries.
  bool first() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return true;
    std::lock_guard<std::mutex> lock(m);
    return !done[dev];
  }
  void settled() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return;
    std::lock_guard<std::mutex> lock(m);
    done[dev] = true;
  }
};

static eas_status finish_linear(Linear& L) {
  EAS_TRY(make_w_tmap(&L.tmap, L.w, L.N, L.K, kBN));
  EAS_TRY(make_w_tmap(&L.tmap_half, L.w, L.N, L.K, kBN / 2));
  EAS_TRY(make_w_tmap_deep(&L.tmap_deep, L.w, L.N, L.K, kBN));
  return make_w_tmap_deep(&L.tmap_half_deep, L.w, L.N, L.K, kBN / 2);
}

typedef void (*GemmKernel)(GemmParams);
// ctas: 1 = one CTA per 128x256 tile; 2 = CTA pair per 256x256 tile; 3 = CTA pair per 256x512 tile ("wide");
// deep (pair tiles only): two 64-wide k-blocks per stage and TMA operation
// out_fp32: 0 bf16, 1 fp32 (reduce-add when a residual is given), 2 the folding residual epilogue (OUT_F32_FOLD)
static GemmKernel gemm_kernel_for(int act, int out_fp32, int ctas, bool deep = false, bool split = false) {
  if (out_fp32 == 2) {
    if (act != ACT_NONE || split) return nullptr;
    if (ctas == 3) return gemm_kernel<ACT_NONE, OUT_F32_FOLD, 2, 2>;
    if (ctas == 2) return deep ? gemm_kernel<ACT_NONE, OUT_F32_FOLD, 2, 1, 2> : gemm_kernel<ACT_NONE, OUT_F32_FOLD, 2, 1>;
    return gemm_kernel<ACT_NONE, OUT_F32_FOLD, 1, 1>;
  }
  if (split) {             // split K: the fp32 residual GEMMs only
    if (act != ACT_NONE || !out_fp32) return nullptr;
    if (ctas == 3) return gemm_kernel<ACT_NONE, OUT_F32, 2, 2, 1, true>;
    if (ctas == 2) return deep ? gemm_kernel<ACT_NONE, OUT_F32, 2, 1, 2, true> : gemm_kernel<ACT_NONE, OUT_F32, 2, 1, 1, true>;
    return gemm_kernel<ACT_NONE, OUT_F32, 1, 1, 1, true>;
  }
  if (ctas == 3) {
    if (act == ACT_NONE && !out_fp32) return gemm_kernel<ACT_NONE, OUT_BF16, 2, 2>;
    if (act == ACT_GELU && !out_fp32) return gemm_kernel<ACT_GELU, OUT_BF16, 2, 2>;
    if (act == ACT_NONE && out_fp32) return gemm_kernel<ACT_NONE, OUT_F32, 2, 2>;
  } else if (ctas == 2 && deep) {
    if (act == ACT_NONE && !out_fp32) return gemm_kernel<ACT_NONE, OUT_BF16, 2, 1, 2>;
    if (act == ACT_GELU && !out_fp32) return gemm_kernel<ACT_GELU, OUT_BF16, 2, 1, 2>;
    if (act == ACT_SWIGLU && !out_fp32) return gemm_kernel<ACT_SWIGLU, OUT_BF16, 2, 1, 2>;
    if (act == ACT_NONE && out_fp32) return gemm_kernel<ACT_NONE, OUT_F32, 2, 1, 2>;
    if (act == ACT_GELU && out_fp32) return gemm_kernel<ACT_GELU, OUT_F32, 2, 1, 2>;
  } else if (ctas == 2) {
    if (act == ACT_NONE && !out_fp32) return gemm_kernel<ACT_NONE, OUT_BF16, 2, 1>;
    if (act == ACT_GELU && !out_fp32) return gemm_kernel<ACT_GELU, OUT_BF16, 2, 1>;
    if (act == ACT_SWIGLU && !out_fp32) return gemm_kernel<ACT_SWIGLU, OUT_BF16, 2, 1>;
    if (act == ACT_NONE && out_fp32) return gemm_kernel<ACT_NONE, OUT_F32, 2, 1>;
    if (act == ACT_GELU && out_fp32) return gemm_kernel<ACT_GELU, OUT_F32, 2, 1>;
  } else {
    if (act == ACT_NONE && !out_fp32) return gemm_kernel<ACT_NONE, OUT_BF16, 1, 1>;
    if (act == ACT_GELU && !out_fp32) return gemm_kernel<ACT_GELU, OUT_BF16, 1, 1>;
    if (act == ACT_SWIGLU && !out_fp32) return gemm_kernel<ACT_SWIGLU, OUT_BF16, 1, 1>;
    if (act == ACT_NONE && out_fp32) return gemm_kernel<ACT_NONE, OUT_F32, 1, 1>;
    if (act == ACT_GELU && out_fp32) return gemm_kernel<ACT_GELU, OUT_F32, 1, 1>;
  }
  return nullptr;
}
static eas_status set_kernel_attributes() {
  for (int deep = 0; deep < 2; ++deep)
    for (int ctas = 1; ctas <= 3; ++ctas)
      for (int act = 0; act < 3; ++act)
        for (int f32 = 0; f32 < 3; ++f32) {
          GemmKernel ks = gemm_kernel_for(act, f32, ctas, deep != 0, true);
          if (ks != nullptr) CUDA_TRY(cudaFuncSetAttribute(ks, cudaFuncAttributeMaxDynamicSharedMemorySize, kGemmSmemBytes));
          GemmKernel k = gemm_kernel_for(act, f32, ctas, deep != 0);
          if (k != nullptr)
            CUDA_TRY(cudaFuncSetAttribute(reinterpret_cast<const void*>(k), cudaFuncAttributeMaxDynamicSharedMemorySize, kGemmSmemBytes));
        }
  return EAS_OK;
}

// the GEMM kernels' attributes, once per device (create-time and the single-kernel entry point both come through here)
static eas_status set_kernel_attributes_once() {
  static OncePerDevice once;
  if (once.first()) {
    EAS_TRY(set_kernel_attributes());
    once.settled();
  }
  return EAS_OK;
}

// shared memory requested by the light kernels: more than half an SM's capacity, so that a second CTA
// can never be co-resident and a grid of B CTAs occupies B SMs
constexpr int kOnePerSmSmem = 120 * 1024;

static eas_status device_check(int* sm_count, int* device = nullptr) {
  int dev = 0;
  CUDA_TRY(cudaGetDevice(&dev));
  if (device != nullptr) *device = dev;
  int major = 0, minor = 0, sms = 0;
  CUDA_TRY(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
  CUDA_TRY(cudaDeviceGetAttribute(&minor, cudaDevAttrComputeCapabilityMinor, dev));
  CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  if (major != 10) return fail(EAS_ERR_ARCH, "device is compute capability %d.%d; this library is built for 10.x", major, minor);
  *sm_count = sms;
  return EAS_OK;
}

// the constants of a linear layer that follows a normalisation (gamma, beta; beta == nullptr for RMSNorm)
static eas_status fold_linear(Arena& arena, const Linear& src, const bf16* gamma, const bf16* beta, const float** c0, const float** c1) {
  float* k0 = static_cast<float*>(arena.take(static_cast<size_t>(src.N) * 4));
  float* k1 = static_cast<float*>(arena.take(static_cast<size_t>(src.N) * 4));
  if (k0 == nullptr || k1 == nullptr) return fail(EAS_ERR_WORKSPACE, "weight arena exhausted");
  FoldWeightsParams fp{src.w, src.b, gamma, beta, k0, k1, src.N, src.K};
  fold_weights_kernel<<<std::min((src.N + 7) / 8, 2048), 256>>>(fp);
  CUDA_TRY(cudaGetLastError());
  *c0 = k0;
  *c1 = k1;
  return EAS_OK;
}

extern "C" eas_status eas_encoder_create(const eas_arch_config* arch, const eas_weights* weights, eas_encoder** out) {
  if (out == nullptr) return fail(EAS_ERR_INVALID_ARG, "out is null");
  *out = nullptr;
  EAS_TRY(check_cfg(arch));
  if (weights == nullptr || weights->tensors == nullptr || weights->n_tensors <= 0)
    return fail(EAS_ERR_INVALID_ARG, "weights are null or empty");
  const size_t need = eas_encoder_weight_arena_bytes(arch);
  if (weights->arena == nullptr || weights->arena_bytes < need)
    return fail(EAS_ERR_WORKSPACE, "weight arena too small: %zu bytes given, %zu needed", weights->arena_bytes, need);
  int sm_count = 0, device = 0;
  EAS_TRY(device_check(&sm_count, &device));
  EAS_TRY(set_kernel_attributes_once());

  WeightIndex wi;
  for (int i = 0; i < weights->n_tensors; ++i) {
    if (weights->tensors[i].name == nullptr) return fail(EAS_ERR_INVALID_ARG, "tensor %d has no name", i);
    wi.by_name[weights->tensors[i].name] = &weights->tensors[i];
  }
  eas_encoder* e = new eas_encoder();
  std::unique_ptr<eas_encoder> guard(e);
  e->cfg = *arch;
  e->device = device;
  e->sm_count = sm_count;
  const eas_arch_config& c = e->cfg;
  const int d = c.d_model, I = c.d_mlp;
  e->hd = d / c.n_heads;
  const bool ln = c.norm == EAS_NORM_LAYERNORM;
  Arena arena{static_cast<uint8_t*>(weights->arena), weights->arena_bytes};

  if (c.family == EAS_FAMILY_AUDIO_CONV) {
    EAS_TRY(wi.get("conv1.w", {d, 3, c.in_channels}, &e->conv1.w));
    EAS_TRY(wi.get("conv1.b", {d}, &e->conv1.b));
    e->conv1.N = d; e->conv1.K = 3 * c.in_channels;
    EAS_TRY(finish_linear(e->conv1));
    EAS_TRY(wi.get("conv2.w", {d, 3, d}, &e->conv2.w));
    EAS_TRY(wi.get("conv2.b", {d}, &e->conv2.b));
    e->conv2.N = d; e->conv2.K = 3 * d;
    EAS_TRY(finish_linear(e->conv2));
  } else {
    e->embed_k = embed_k_of(&c);
    e->embed_k_pad = static_cast<int>(align_up(e->embed_k, 64));
    if (e->embed_k_pad > 4096 || c.patch > 255 || c.temporal_patch > 255 || c.in_channels > 255)
      return fail(EAS_ERR_UNSUPPORTED, "patch vector of %d elements (at most %d; patch, temporal patch and channels at most 255)", e->embed_k, 4096);
    const bf16* w = nullptr;
    EAS_TRY(wi.get("embed.w", {d, e->embed_k}, &w));
    EAS_TRY(wi.get("embed.b", {d}, &e->embed.b));
    bf16* dst = static_cast<bf16*>(arena.take(static_cast<size_t>(d) * e->embed_k_pad * 2));
    if (dst == nullptr) return fail(EAS_ERR_WORKSPACE, "weight arena exhausted");
    EAS_TRY(relayout(dst, w, nullptr, d, e->embed_k, e->embed_k_pad, 0, 0, 0));
    e->embed.w = dst; e->embed.N = d; e->embed.K = e->embed_k_pad;
    EAS_TRY(finish_linear(e->embed));
    uint32_t* table = static_cast<uint32_t*>(arena.take(static_cast<size_t>(e->embed_k_pad) * 2));
    if (table == nullptr) return fail(EAS_ERR_WORKSPACE, "weight arena exhausted");
    embed_table_kernel<<<4, 256>>>(table, e->embed_k, e->embed_k_pad, c.patch, c.temporal_patch);
    CUDA_TRY(cudaGetLastError());
    e->embed_table = table;
  }
  if (c.has_cls) EAS_TRY(wi.get("cls", {d}, &e->cls));
  if (c.pos == EAS_POS_TABLE) EAS_TRY(wi.get("pos", {c.max_pos, d}, &e->pos));
  if (c.embed_norm) {
    EAS_TRY(wi.get("embed_norm.g", {d}, &e->eng));
    if (ln) EAS_TRY(wi.get("embed_norm.b", {d}, &e->enb));
  }
  e->layers.resize(c.n_layers);
  for (int i = 0; i < c.n_layers; ++i) {
    Layer& L = e->layers[i];
    const std::string p = "blk" + std::to_string(i) + ".";
    EAS_TRY(wi.get(p + "norm1.g", {d}, &L.n1g));
    if (ln) EAS_TRY(wi.get(p + "norm1.b", {d}, &L.n1b));
    EAS_TRY(wi.get(p + "norm2.g", {d}, &L.n2g));
    if (ln) EAS_TRY(wi.get(p + "norm2.b", {d}, &L.n2b));
    const bf16 *qw = nullptr, *qb = nullptr;
    EAS_TRY(wi.get(p + "qkv.w", {3 * d, d}, &qw));
    EAS_TRY(wi.get(p + "qkv.b", {3 * d}, &qb));
    if (c.pos == EAS_POS_ROPE_2D) {
      // rows of every Q and K head re-ordered so that the two halves of a rotary pair are adjacent
      bf16* w2 = static_cast<bf16*>(arena.take(static_cast<size_t>(3) * d * d * 2));
      bf16* b2 = static_cast<bf16*>(arena.take(static_cast<size_t>(3) * d * 2));
      if (w2 == nullptr || b2 == nullptr) return fail(EAS_ERR_WORKSPACE, "weight arena exhausted");
      EAS_TRY(relayout(w2, qw, nullptr, 3LL * d, d, d, 1, e->hd, 2LL * d));
      EAS_TRY(relayout(b2, qb, nullptr, 3LL * d, 1, 1, 1, e->hd, 2LL * d));
      qw = w2; qb = b2;
    }
    L.qkv.w = qw; L.qkv.b = qb; L.qkv.N = 3 * d; L.qkv.K = d;
    EAS_TRY(finish_linear(L.qkv));
    EAS_TRY(wi.get(p + "proj.w", {d, d}, &L.proj.w));
    EAS_TRY(wi.get(p + "proj.b", {d}, &L.proj.b));
    L.proj.N = d; L.proj.K = d;
    EAS_TRY(finish_linear(L.proj));
    if (c.mlp == EAS_MLP_SWIGLU) {
      const bf16 *gw, *gb, *uw, *ub;
      EAS_TRY(wi.get(p + "gate.w", {I, d}, &gw));
      EAS_TRY(wi.get(p + "gate.b", {I}, &gb));
      EAS_TRY(wi.get(p + "up.w", {I, d}, &uw));
      EAS_TRY(wi.get(p + "up.b", {I}, &ub));
      bf16* w2 = static_cast<bf16*>(arena.take(static_cast<size_t>(2) * I * d * 2));
      bf16* b2 = static_cast<bf16*>(arena.take(static_cast<size_t>(2) * I * 2));
      if (w2 == nullptr || b2 == nullptr) return fail(EAS_ERR_WORKSPACE, "weight arena exhausted");
      EAS_TRY(relayout(w2, gw, uw, 2LL * I, d, d, 2, 0, 0));
      EAS_TRY(relayout(b2, gb, ub, 2LL * I, 1, 1, 2, 0, 0));
      L.fc1.w = w2; L.fc1.b = b2; L.fc1.N = 2 * I; L.fc1.K = d;
    } else {
      EAS_TRY(wi.get(p + "fc1.w", {I, d}, &L.fc1.w));
      EAS_TRY(wi.get(p + "fc1.b", {I}, &L.fc1.b));
      L.fc1.N = I; L.fc1.K = d;
    }
    EAS_TRY(finish_linear(L.fc1));
    EAS_TRY(wi.get(p + "fc2.w", {d, I}, &L.fc2.w));
    EAS_TRY(wi.get(p + "fc2.b", {d}, &L.fc2.b));
    L.fc2.N = d; L.fc2.K = I;
    EAS_TRY(finish_linear(L.fc2));
    EAS_TRY(fold_linear(arena, L.qkv, L.n1g, ln ? L.n1b : nullptr, &L.qkv_c0, &L.qkv_c1));
    EAS_TRY(fold_linear(arena, L.fc1, L.n2g, ln ? L.n2b : nullptr, &L.fc1_c0, &L.fc1_c1));
  }
  if (c.final_norm) {
    EAS_TRY(wi.get("final_norm.g", {d}, &e->fng));
    if (ln) EAS_TRY(wi.get("final_norm.b", {d}, &e->fnb));
  }
  if (c.head != EAS_HEAD_NONE) {
    const int kin = c.head == EAS_HEAD_MERGER_2X2 ? 4 * d : d;
    if (c.head == EAS_HEAD_MERGER_2X2) EAS_TRY(wi.get("head.norm.g", {d}, &e->hng));
    EAS_TRY(wi.get("head.fc1.w", {c.d_head_hidden, kin}, &e->head1.w));
    EAS_TRY(wi.get("head.fc1.b", {c.d_head_hidden}, &e->head1.b));
    e->head1.N = c.d_head_hidden; e->head1.K = kin;
    EAS_TRY(finish_linear(e->head1));
    EAS_TRY(wi.get("head.fc2.w", {c.d_out, c.d_head_hidden}, &e->head2.w));
    EAS_TRY(wi.get("head.fc2.b", {c.d_out}, &e->head2.b));
    e->head2.N = c.d_out; e->head2.K = c.d_head_hidden;
    EAS_TRY(finish_linear(e->head2));
  }
  CUDA_TRY(cudaDeviceSynchronize());   // re-layout kernels ran on the default stream
  *out = guard.release();
  return EAS_OK;
}

extern "C" void eas_encoder_destroy(eas_encoder* enc) { delete enc; }

extern "C" eas_status eas_encoder_set_attention_impl(eas_encoder* enc, int32_t impl) {
  if (enc == nullptr || impl < 0 || impl > 2) return fail(EAS_ERR_INVALID_ARG, "bad attention impl");
  enc->attn_impl = impl;
  return EAS_OK;
}

extern "C" eas_status eas_encoder_set_split_k(eas_encoder* enc, int32_t on) {
  if (enc == nullptr) return fail(EAS_ERR_INVALID_ARG, "encoder is null");
  enc->split_k = on != 0 ? 1 : 0;
  return EAS_OK;
}

extern "C" eas_status eas_encoder_set_norm_fold(eas_encoder* enc, int32_t on) {
  if (enc == nullptr) return fail(EAS_ERR_INVALID_ARG, "encoder is null");
  enc->fold = on != 0;
  return EAS_OK;
}

extern "C" int32_t eas_encoder_last_launch_count(const eas_encoder* enc) { return enc ? enc->last_launches : 0; }

// ------------------------------------------------------------------------------------ workspace plan
namespace {
struct Plan {
  size_t status, x, n, qkv, o, a, row_map, pos_idx, head_src, rope, mel_pad, h1_pad, conv1_map, part, stats, total;
  int splits_proj, splits_fc2;     // split-K factors of the two residual GEMMs of a block (1: off)
  int64_t part_rows;               // rows of one split's region of the partial-sum scratch
  int64_t T, embed_rows, padded_rows, out_rows;
};
}  // namespace

// Split-K factor of a residual GEMM x[M, N] += A[M, K] W^T with few tiles (small micro-batches: the K loop of one tile is
// the whole kernel, and most SMs have no tile).  A function of the shape and the device only, never of the SM budget, so
// that results do not depend on the budget; every split is a whole number of 128-wide k-steps, so that they do not
// depend on the tile shape either.
static int pick_splits(int64_t M, int64_t N, int64_t K, int sm_count) {
  const int64_t items = ((M + kBM - 1) / kBM) * ((N + kBN - 1) / kBN);
  for (int s = 4; s >= 2; s >>= 1)
    if (items * s <= sm_count && K % (s * 2 * kBK) == 0 && K / s >= 1024) return s;
  return 1;
}

static Plan make_plan(const eas_encoder* e, int64_t T, int n_items) {
  const eas_arch_config& c = e->cfg;
  Plan p{};
  p.T = T;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 1024); return o; };
  const size_t d = c.d_model;
  const bool audio = c.family == EAS_FAMILY_AUDIO_CONV;
  p.padded_rows = audio ? 2 * T + 2 * n_items : 0;
  p.embed_rows = audio ? T + n_items : T - (c.has_cls ? n_items : 0);
  p.out_rows = c.head == EAS_HEAD_MLP_PROJECTOR ? T - (c.has_cls ? n_items : 0) : (c.head == EAS_HEAD_MERGER_2X2 ? T / 4 : T);
  p.status = take(1024);
  p.x = take(T * d * 4);
  p.n = take(T * d * 2);
  p.qkv = take(T * 3 * d * 2);
  p.o = take(T * d * 2);
  const size_t a_elems = std::max<size_t>(T * static_cast<size_t>(c.d_mlp), static_cast<size_t>(p.out_rows) * std::max(c.d_head_hidden, 0));
  p.a = take(a_elems * 2);
  p.row_map = take(static_cast<size_t>(p.embed_rows) * 4);
  p.pos_idx = take(static_cast<size_t>(p.embed_rows) * 4);
  p.head_src = take(static_cast<size_t>(T) * 4);
  p.rope = take(c.pos == EAS_POS_ROPE_2D ? static_cast<size_t>(T) * (e->hd / 2) * 8 : 0);
  p.mel_pad = take(static_cast<size_t>(p.padded_rows) * c.in_channels * 2);
  p.h1_pad = take(static_cast<size_t>(p.padded_rows) * d * 2);
  p.conv1_map = take(static_cast<size_t>(p.padded_rows) * 4);
  p.splits_proj = e->split_k ? pick_splits(T, c.d_model, c.d_model, e->sm_count) : 1;
  p.splits_fc2 = e->split_k ? pick_splits(T, c.d_model, c.d_mlp, e->sm_count) : 1;
  p.part_rows = (T + 2 * kBM - 1) / (2 * kBM) * (2 * kBM);
  p.part = take(static_cast<size_t>(std::max(p.splits_proj, p.splits_fc2) - 1) * p.part_rows * d * 4);
  p.stats = take(static_cast<size_t>(T) * (d / kFoldGroup) * 8);    // (mean, M2) per row and group of 128 columns
  p.total = off;
  return p;
}

extern "C" size_t eas_encoder_workspace_bytes(const eas_encoder* enc, int64_t total_tokens, int32_t n_items, int32_t /*max_seqlen*/) {
  if (enc == nullptr || total_tokens <= 0 || n_items <= 0) return 0;
  return make_plan(enc, total_tokens, n_items).total;
}

static int64_t out_rows_of(const eas_encoder* e, int64_t S) {
  if (e->cfg.head == EAS_HEAD_MLP_PROJECTOR) return S - (e->cfg.has_cls ? 1 : 0);
  if (e->cfg.head == EAS_HEAD_MERGER_2X2) return S / 4;
  return S;
}

extern "C" int64_t eas_encoder_out_rows(const eas_encoder* enc, const int32_t* cu, int32_t n_items) {
  if (enc == nullptr || cu == nullptr || n_items <= 0) return -1;
  int64_t r = 0;
  for (int i = 0; i < n_items; ++i) r += out_rows_of(enc, cu[i + 1] - cu[i]);
  return r;
}

// ------------------------------------------------------------------------------------ launch helpers
// A call that owns the whole device launches its kernels with programmatic stream serialization: a kernel may be set
// up while its predecessor in the stream drains, and waits (griddepcontrol.wait) before touching any data.  A call on
// a SHARE of the SMs (Section 3.4) must not: its grids are persistent (all CTAs resident at once), so a dependent
// kernel would be released the moment its predecessor started, its CTAs would settle on SMs outside the share and
// sit there holding shared memory and tensor memory while they wait -- exactly the SMs the co-resident worker was
// promised.  Without the attribute a kernel starts when its predecessor has finished, and at most `sm_budget` SMs
// hold a CTA of this call at any time.  Set by every entry point before its first launch (per host thread).
static thread_local bool g_overlap_launches = true;
template <typename Params>
static eas_status launch_kernel(void (*kern)(Params), int grid, int block, size_t smem, cudaStream_t stream, const Params& params,
                                int cluster = 1) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(static_cast<unsigned>(grid), 1, 1);
  cfg.blockDim = dim3(static_cast<unsigned>(block), 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  int n = 0;
  if (g_overlap_launches) {
    attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
  }
  if (cluster > 1) {
    attr[n].id = cudaLaunchAttributeClusterDimension;
    attr[n].val.clusterDim.x = static_cast<unsigned>(cluster);
    attr[n].val.clusterDim.y = 1;
    attr[n].val.clusterDim.z = 1;
    ++n;
  }
  cfg.attrs = attr;
  cfg.numAttrs = n;
  CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, params));
  return EAS_OK;
}

namespace {
struct GemmCall {
  const void* A = nullptr;   // bf16
  int64_t a_run = 0;         // K per tap (elements)
  int64_t a_row_elems = 0;   // elements between consecutive rows of A
  int conv_stride = 1;       // 1: plain GEMM
  int taps = 1;
  int64_t a_rows = 0;        // rows addressable in A
  int M = 0;                 // rows walked
  const Linear* lin = nullptr;
  int act = ACT_NONE;
  int out_fp32 = 0;
  void* out = nullptr;
  int64_t ldo = 0;
  const float* resid = nullptr;
  const int* row_map = nullptr;
  const int* pos_idx = nullptr;
  const bf16* pos = nullptr;
  const float2* rope_cs = nullptr;
  int reverse = 0;             // walk the tiles last to first
  int w_const = 1;             // the weights are constant (set at create time): their loads may start before the stream's earlier work ends
  int force_tile = 0;          // 0: the launcher picks; 1 one CTA per 128x256 tile, 2 CTA pair per 256x256, 3 pair per 256x512 (tests)
  int splits = 1;              // split K (see GemmParams::splits); the partial sums of splits 1.. go to `part`
  float* part = nullptr;       // [(splits - 1) * part_rows, N] fp32
  int64_t part_rows = 0;
  long long rope_stride = 0;   // rows of the [pair][row] table
  int rope_pairs = 0, rope_ncols = 0, head_dim = 0;
  // folded normalisation (GemmParams::fold_stats).  Consumer: fold_stats with fold_c0 / fold_c1 of the folded weights in
  // `lin`.  Producer (an in-place fp32 residual GEMM): fold_stats_out, fold_xb and fold_gamma.
  const float2* fold_stats = nullptr;
  const float *fold_c0 = nullptr, *fold_c1 = nullptr;
  int fold_rms = 0;
  float fold_eps = 0.f;
  int64_t fold_rows = 0;
  float2* fold_stats_out = nullptr;
  bf16* fold_xb = nullptr;
  const bf16* fold_gamma = nullptr;
};
}  // namespace

static eas_status launch_gemm(const GemmCall& g, int budget, cudaStream_t stream, uint32_t* status) {
  const Linear& L = *g.lin;
  if (g.M <= 0) return EAS_OK;
  if (L.N % 32 != 0 || g.a_run % kBK != 0) return fail(EAS_ERR_UNSUPPORTED, "GEMM needs N %% 32 == 0 and K %% 64 == 0 (N=%d, K=%lld)", L.N, static_cast<long long>(g.a_run));
  // Tile shape: one CTA per 128x256 tile, a CTA pair per 256x256 tile, or a pair per wide 256x512 tile.  All three
  // accumulate every output element over K in the same order, so the results are bit-identical and this is a pure
  // speed choice: estimated time = waves x time of one tile.  The per-k-block times are measured on B200 with each
  // shape forced over the encoder's GEMM shapes (M = 1154 ... 24000): a 64-wide k-block takes 0.47 us (single CTA),
  // 0.40 us (pair, deep stages; 0.43 for the convolutions' shallow ones) or 0.75 us for twice the columns (wide
  // pair); the wide tile's epilogue (about 4 us) does not overlap the next main loop.  What decides in practice is
  // the wave count: at M = 4616 (c1, micro-batch 8) the out-projection is 2 half-empty waves of
  // pair tiles but exactly 1 wave of single-CTA tiles.
  const bool tma_out = g.row_map == nullptr && g.pos == nullptr && (g.resid == nullptr || g.resid == g.out);
  const int64_t k_total = g.a_run * g.taps;
  const double kb = static_cast<double>(k_total / kBK);
  auto waves = [](long long tiles, long long slots) { return static_cast<double>((tiles + slots - 1) / slots); };
  const long long n256 = (L.N + kBN - 1) / kBN;
  int ctas = 1;
  bool wide = false;
  if (budget >= 2) {
    const long long pairs = budget / 2;
    const long long m128 = (g.M + kBM - 1) / kBM, m256 = (g.M + 2 * kBM - 1) / (2 * kBM);
    const double cost_single = waves(m128 * n256 * g.splits, budget) * kb / g.splits * 0.47;
    const double cost_pair = waves(m256 * n256 * g.splits, pairs) * kb / g.splits * (g.conv_stride == 1 && g.taps == 1 ? 0.40 : 0.43);
    ctas = cost_single < cost_pair ? 1 : 2;
    // wide tiles: long reductions whose output splits evenly into 512-column blocks, plain TMA-stored epilogue
    if (tma_out && g.act != ACT_SWIGLU && k_total >= 2048 && L.N % 512 == 0 && gemm_kernel_for(g.act, g.out_fp32, 3) != nullptr) {
      const double cost_wide = waves(m256 * (L.N / (2 * kBN)) * g.splits, pairs) * (kb / g.splits * 0.75 + 4.0);
      if (cost_wide < std::min(cost_single, cost_pair)) { ctas = 2; wide = true; }
    }
    if (g.force_tile != 0) {
      const bool wide_ok = tma_out && g.act != ACT_SWIGLU && L.N % 512 == 0 && gemm_kernel_for(g.act, g.out_fp32, 3) != nullptr;
      if (g.force_tile == 3 && !wide_ok) return fail(EAS_ERR_UNSUPPORTED, "no wide (256x512) tile for this GEMM: it needs N %% 512 == 0, a plain or GELU epilogue and row-aligned output");
      ctas = g.force_tile == 1 ? 1 : 2;
      wide = g.force_tile == 3;
    }
#ifdef EAS_GEMM_FORCE_TILE   // calibration builds only: 1 single CTA, 2 pair, 3 wide pair (where a wide kernel exists)
    ctas = EAS_GEMM_FORCE_TILE == 1 ? 1 : 2;
    wide = EAS_GEMM_FORCE_TILE == 3 && tma_out && g.act != ACT_SWIGLU && L.N % 512 == 0 && gemm_kernel_for(g.act, g.out_fp32, 3) != nullptr;
#endif
  }
  const bool fold_out = g.fold_stats_out != nullptr;
  if (fold_out && (!tma_out || !g.out_fp32 || g.resid != g.out || g.splits != 1 || g.act != ACT_NONE || g.fold_xb == nullptr || g.fold_gamma == nullptr || L.N % kFoldGroup != 0))
    return fail(EAS_ERR_UNSUPPORTED, "the folding epilogue needs an in-place fp32 residual GEMM with N %% %d == 0", kFoldGroup);
  if (g.fold_stats != nullptr && (!tma_out || g.fold_c0 == nullptr || g.a_run % kFoldGroup != 0 || g.taps != 1))
    return fail(EAS_ERR_UNSUPPORTED, "a folded normalisation needs a plain GEMM with row-aligned output and K %% %d == 0", kFoldGroup);
  const int out_mode = fold_out ? 2 : (g.out_fp32 ? 1 : 0);
  const int tile_n = wide ? 2 * kBN : kBN;
  // pair tiles of plain GEMMs run the deep kernel (two k-blocks per stage and TMA operation: 8 % faster at K = 1024);
  // single-CTA and wide tiles would be left with two 96 KB stages and measured no better, and convolutions walk their
  // taps as 64-wide k-blocks
  const bool deep = g.conv_stride == 1 && g.taps == 1 && ctas == 2 && !wide;
  GemmParams p{};
  if (deep) EAS_TRY(make_a_tmap_deep(&p.tma_a, g.A, g.a_run, g.a_row_elems, g.a_rows));
  else EAS_TRY(make_a_tmap(&p.tma_a, g.A, g.a_run, g.a_row_elems, g.conv_stride, g.a_rows));
  p.tma_b = deep ? (ctas == 2 ? L.tmap_half_deep : L.tmap_deep) : (ctas == 2 ? L.tmap_half : L.tmap);
  p.M = g.M; p.N = L.N;
  p.kb_per_tap = static_cast<int>(g.a_run / kBK);
  p.k_blocks = deep ? (p.kb_per_tap + 1) / 2 : p.kb_per_tap * g.taps;
  p.conv_stride = g.conv_stride;
  p.reverse = g.reverse;
  p.w_const = g.w_const;
  p.splits = 1;
  p.kb_per_split = p.k_blocks;
  if (g.splits > 1) {
    if (!tma_out || !g.out_fp32 || g.resid != g.out || g.taps != 1 || g.conv_stride != 1 || g.part == nullptr ||
        g.a_run % (g.splits * 2 * kBK) != 0 || g.part_rows % (2 * kBM) != 0 || g.part_rows < g.M)
      return fail(EAS_ERR_UNSUPPORTED, "split K needs an in-place fp32 residual GEMM whose K is a multiple of %d", g.splits * 2 * kBK);
    p.splits = g.splits;
    p.kb_per_split = p.k_blocks / g.splits;
    p.part_rows = static_cast<int>(g.part_rows);
    EAS_TRY(make_out_tmap(&p.tma_part, g.part, true, L.N, L.N, static_cast<int64_t>(g.splits - 1) * g.part_rows));
  }
  p.m_blocks = (g.M + kBM * ctas - 1) / (kBM * ctas);
  p.n_blocks = (L.N + tile_n - 1) / tile_n;
  p.bias = L.b;
  p.out = g.out; p.ldo = g.ldo; p.resid = g.resid;
  p.row_map = g.row_map; p.pos_idx = g.pos_idx; p.pos = g.pos;
  p.rope_cs = g.rope_cs; p.rope_stride = g.rope_stride; p.rope_pairs = g.rope_pairs; p.rope_ncols = g.rope_ncols; p.head_dim = g.head_dim > 0 ? g.head_dim : 64;
  p.status = status;
  p.fold_stats = g.fold_stats; p.fold_c0 = g.fold_c0; p.fold_c1 = g.fold_c1; p.fold_rows = g.fold_rows;
  p.fold_parts = static_cast<int>(g.a_run / kFoldGroup); p.fold_rms = g.fold_rms; p.fold_eps = g.fold_eps;
  p.fold_stats_out = g.fold_stats_out; p.fold_xb = g.fold_xb; p.fold_gamma = g.fold_gamma;
  // TMA-store epilogue whenever output rows are the A rows and any residual is accumulated in place
  p.use_tma_out = tma_out ? 1 : 0;
  if (p.use_tma_out) {
    const int64_t out_cols = g.act == ACT_SWIGLU ? L.N / 2 : L.N;
    EAS_TRY(make_out_tmap(&p.tma_out, g.out, g.out_fp32 != 0, out_cols, g.ldo, g.M));
  }
  const int tiles = p.m_blocks * p.n_blocks * p.splits;
  GemmKernel kern = gemm_kernel_for(g.act, out_mode, wide ? 3 : ctas, deep, p.splits > 1);
  if (kern == nullptr) return fail(EAS_ERR_UNSUPPORTED, "no GEMM epilogue for act=%d out_fp32=%d", g.act, g.out_fp32);
  return launch_kernel(kern, std::min(budget / ctas, tiles) * ctas, kGemmThreads, kGemmSmemBytes, stream, p, ctas);
}

template <int KIND, bool F32, bool PART = false>
static eas_status launch_norm_nv(const NormParams& p, int budget, cudaStream_t stream) {
  const int nv = p.d / 128;
#define EAS_NORM_CASE(NV_)                                                                                         \
  case NV_: {                                                                                                      \
    static OncePerDevice once;                                                                                     \
    if (once.first()) {                                                                                            \
      CUDA_TRY(cudaFuncSetAttribute(norm_kernel<NV_, KIND, F32, PART>, cudaFuncAttributeMaxDynamicSharedMemorySize, kOnePerSmSmem)); \
      once.settled();                                                                                              \
    }                                                                                                              \
    EAS_TRY(launch_kernel(norm_kernel<NV_, KIND, F32, PART>, std::min(budget, (p.rows + 15) / 16), 512, kOnePerSmSmem, stream, p)); \
    break;                                                                                                         \
  }
  switch (nv) {
    EAS_NORM_CASE(1) EAS_NORM_CASE(2) EAS_NORM_CASE(3) EAS_NORM_CASE(4) EAS_NORM_CASE(5) EAS_NORM_CASE(6)
    EAS_NORM_CASE(7) EAS_NORM_CASE(8) EAS_NORM_CASE(9) EAS_NORM_CASE(10) EAS_NORM_CASE(11) EAS_NORM_CASE(12)
    EAS_NORM_CASE(13) EAS_NORM_CASE(14) EAS_NORM_CASE(15) EAS_NORM_CASE(16)
    default: return fail(EAS_ERR_UNSUPPORTED, "norm width %d", p.d);
  }
#undef EAS_NORM_CASE
  CUDA_TRY(cudaGetLastError());
  return EAS_OK;
}

static eas_status launch_fold_stats(const FoldStatsParams& p, int budget, cudaStream_t stream) {
  if (p.rows <= 0) return EAS_OK;
#define EAS_FOLD_CASE(NV_)                                                                                         \
  case NV_: {                                                                                                      \
    static OncePerDevice once;                                                                                     \
    if (once.first()) {                                                                                            \
      CUDA_TRY(cudaFuncSetAttribute(fold_stats_kernel<NV_>, cudaFuncAttributeMaxDynamicSharedMemorySize, kOnePerSmSmem)); \
      once.settled();                                                                                              \
    }                                                                                                              \
    EAS_TRY(launch_kernel(fold_stats_kernel<NV_>, std::min(budget, (p.rows + 15) / 16), 512, kOnePerSmSmem, stream, p)); \
    break;                                                                                                         \
  }
  switch (p.d / 128) {
    EAS_FOLD_CASE(1) EAS_FOLD_CASE(2) EAS_FOLD_CASE(3) EAS_FOLD_CASE(4) EAS_FOLD_CASE(5) EAS_FOLD_CASE(6)
    EAS_FOLD_CASE(7) EAS_FOLD_CASE(8) EAS_FOLD_CASE(9) EAS_FOLD_CASE(10) EAS_FOLD_CASE(11) EAS_FOLD_CASE(12)
    EAS_FOLD_CASE(13) EAS_FOLD_CASE(14) EAS_FOLD_CASE(15) EAS_FOLD_CASE(16)
    default: return fail(EAS_ERR_UNSUPPORTED, "row width %d", p.d);
  }
#undef EAS_FOLD_CASE
  return EAS_OK;
}

static eas_status launch_norm(int kind, bool out_fp32, const NormParams& p, int budget, cudaStream_t stream) {
  if (p.rows <= 0) return EAS_OK;
  if (p.d % 128 != 0 || p.d > 2048) return fail(EAS_ERR_UNSUPPORTED, "norm width %d (need a multiple of 128, at most 2048)", p.d);
  if (p.n_part > 0) {        // split-K partial sums to add first: the residual blocks' bf16 normalisations only
    if (out_fp32 || p.src_rows != nullptr || p.x_rw == nullptr || p.part == nullptr || kind == NORM_CAST)
      return fail(EAS_ERR_UNSUPPORTED, "partial sums are added by LayerNorm / RMSNorm with bf16 output only");
    return kind == NORM_LN ? launch_norm_nv<NORM_LN, false, true>(p, budget, stream) : launch_norm_nv<NORM_RMS, false, true>(p, budget, stream);
  }
  if (kind == NORM_LN) return out_fp32 ? launch_norm_nv<NORM_LN, true>(p, budget, stream) : launch_norm_nv<NORM_LN, false>(p, budget, stream);
  if (kind == NORM_RMS) return out_fp32 ? launch_norm_nv<NORM_RMS, true>(p, budget, stream) : launch_norm_nv<NORM_RMS, false>(p, budget, stream);
  if (kind == NORM_CAST) return out_fp32 ? launch_norm_nv<NORM_CAST, true>(p, budget, stream) : launch_norm_nv<NORM_CAST, false>(p, budget, stream);
  return fail(EAS_ERR_INVALID_ARG, "unknown norm kind %d", kind);
}

// schedule order: longest items first (stable), so the tail of the static round-robin is short work
// dual_head: the tcgen05 kernel's unit order for head_dim 64 (see decode_unit): per item H x (full pairs of query
// tiles), then one unit per two heads for an odd last tile.
// reverse: items of equal length are taken last to first (the producer of qkv wrote the last rows most recently: L2).
static void attention_schedule(const int32_t* cu, int n_items, int rows_per_unit, int H, int* item_start, int* item_len,
                               int* unit_prefix, int* total_units, bool dual_head = false, bool reverse = false) {
  std::vector<int> order(n_items);
  for (int i = 0; i < n_items; ++i) order[i] = reverse ? n_items - 1 - i : i;
  std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return (cu[a + 1] - cu[a]) > (cu[b + 1] - cu[b]); });
  int units = 0;
  for (int k = 0; k < n_items; ++k) {
    const int i = order[k];
    item_start[k] = cu[i];
    item_len[k] = cu[i + 1] - cu[i];
    unit_prefix[k] = units;
    if (dual_head) {
      const int tiles = (item_len[k] + rows_per_unit / 2 - 1) / (rows_per_unit / 2);
      units += (tiles / 2) * H + (tiles % 2) * ((H + 1) / 2);
    } else {
      units += ((item_len[k] + rows_per_unit - 1) / rows_per_unit) * H;
    }
  }
  unit_prefix[n_items] = units;
  *total_units = units;
}

static eas_status launch_attention_mma(const bf16* qkv, bf16* out, const int32_t* cu, int n_items, int H, int hd, int budget,
                                       cudaStream_t stream) {
  AttnParams ap{};
  const int d = H * hd;
  ap.qkv = qkv; ap.out = out; ap.ld = 3LL * d; ap.ldo = d; ap.d_model = d; ap.n_heads = H;
  ap.scale_log2 = static_cast<float>(1.4426950408889634 / std::sqrt(static_cast<double>(hd)));
  ap.n_items = n_items;
  attention_schedule(cu, n_items, kAttnBQ, H, ap.item_start, ap.item_len, ap.unit_prefix, &ap.total_units);
  if (ap.total_units == 0) return EAS_OK;
  const int grid = std::min(budget, ap.total_units);
  static OncePerDevice once;
  if (once.first()) {
    CUDA_TRY(cudaFuncSetAttribute(attn_mma_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, kOnePerSmSmem));
    CUDA_TRY(cudaFuncSetAttribute(attn_mma_kernel<80>, cudaFuncAttributeMaxDynamicSharedMemorySize, kOnePerSmSmem));
    once.settled();
  }
  static_assert(attn_mma_smem_bytes<80>() <= kOnePerSmSmem, "attention tile does not fit");
  if (hd == 64) return launch_kernel(attn_mma_kernel<64>, grid, kAttnThreads, kOnePerSmSmem, stream, ap);
  if (hd == 80) return launch_kernel(attn_mma_kernel<80>, grid, kAttnThreads, kOnePerSmSmem, stream, ap);
  return fail(EAS_ERR_UNSUPPORTED, "head_dim %d", hd);
}

template <bool PT>
static eas_status launch_attention_tc(const bf16* qkv, bf16* out, const int32_t* cu, int n_items, int H, int hd, int budget,
                                      cudaStream_t stream, uint32_t* status, bool reverse) {
  AttnTcParams ap{};
  const int d = H * hd;
  const int64_t T = cu[n_items];
  {
    const uint64_t dims[2] = {static_cast<uint64_t>(3 * d), static_cast<uint64_t>(T)};
    const uint64_t strides[1] = {static_cast<uint64_t>(3 * d) * 2};
    const uint32_t box_lo[2] = {64, kTcTile};
    EAS_TRY(make_tmap(&ap.map_lo, qkv, 2, dims, strides, box_lo, CU_TENSOR_MAP_SWIZZLE_128B));
    const uint32_t box_hi[2] = {16, kTcTile};
    EAS_TRY(make_tmap(&ap.map_hi, qkv, 2, dims, strides, box_hi, CU_TENSOR_MAP_SWIZZLE_32B));
    // K and V tiles: the kernel's keys per tile (head_dim 80 with P in tensor memory: 112)
    const uint32_t keys = hd == 64 ? AttnTcSmem<64, PT>::kKeys : AttnTcSmem<80, PT>::kKeys;
    const uint32_t box_klo[2] = {64, keys};
    EAS_TRY(make_tmap(&ap.map_klo, qkv, 2, dims, strides, box_klo, CU_TENSOR_MAP_SWIZZLE_128B));
    const uint32_t box_khi[2] = {16, keys};
    EAS_TRY(make_tmap(&ap.map_khi, qkv, 2, dims, strides, box_khi, CU_TENSOR_MAP_SWIZZLE_32B));
    const uint64_t odims[2] = {static_cast<uint64_t>(d), static_cast<uint64_t>(T)};
    const uint64_t ostrides[1] = {static_cast<uint64_t>(d) * 2};
    const uint32_t obox[2] = {64, 32};
    EAS_TRY(make_tmap(&ap.map_out, out, 2, odims, ostrides, obox, CU_TENSOR_MAP_SWIZZLE_128B));
  }
  ap.out = out; ap.ldo = d; ap.d_model = d; ap.n_heads = H;
  ap.scale_log2 = static_cast<float>(1.4426950408889634 / std::sqrt(static_cast<double>(hd)));
  ap.n_items = n_items;
  ap.status = status;
  // dual-head units (two heads' odd last query tiles in one unit) when some item has an odd number of 128-row tiles
  bool dual = false;
  if (hd == 64 && AttnTcSmem<64, PT>::kDualHeadOk && H >= 2)
    for (int i = 0; i < n_items; ++i) dual = dual || (((cu[i + 1] - cu[i] + kTcTile - 1) / kTcTile) & 1) != 0;
  attention_schedule(cu, n_items, 2 * kTcTile, H, ap.item_start, ap.item_len, ap.unit_prefix, &ap.total_units, dual, reverse);
  if (ap.total_units == 0) return EAS_OK;
  const int grid = std::min(budget, ap.total_units);
  static OncePerDevice once;
  if (once.first()) {
    CUDA_TRY(cudaFuncSetAttribute(attn_tc_kernel<64, PT>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttnTcSmem<64, PT>::kBytes));
    CUDA_TRY(cudaFuncSetAttribute(attn_tc_kernel<80, PT>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttnTcSmem<80, PT>::kBytes));
    if (AttnTcSmem<64, PT>::kDualHeadOk)
      CUDA_TRY(cudaFuncSetAttribute(attn_tc_kernel<64, PT, AttnTcSmem<64, PT>::kDualHeadOk>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttnTcSmem<64, PT>::kBytes));
    once.settled();
  }
  if (hd == 64 && dual)
    return launch_kernel(attn_tc_kernel<64, PT, AttnTcSmem<64, PT>::kDualHeadOk>, grid, kTcThreads, AttnTcSmem<64, PT>::kBytes, stream, ap);
  if (hd == 64) return launch_kernel(attn_tc_kernel<64, PT>, grid, kTcThreads, AttnTcSmem<64, PT>::kBytes, stream, ap);
  if (hd == 80) return launch_kernel(attn_tc_kernel<80, PT>, grid, kTcThreads, AttnTcSmem<80, PT>::kBytes, stream, ap);
  return fail(EAS_ERR_UNSUPPORTED, "head_dim %d", hd);
}

static eas_status launch_attention(const bf16* qkv, bf16* out, const int32_t* cu, int n_items, int H, int hd, int budget,
                                   cudaStream_t stream, int impl, uint32_t* status, bool reverse = false) {
  if (impl == 1) return launch_attention_mma(qkv, out, cu, n_items, H, hd, budget, stream);
  if (impl == 2) return launch_attention_tc<false>(qkv, out, cu, n_items, H, hd, budget, stream, status, reverse);
  return launch_attention_tc<true>(qkv, out, cu, n_items, H, hd, budget, stream, status, reverse);
}

// ------------------------------------------------------------------------------------ the forward pass
// The forward pass.  `workspace` / `workspace_bytes` override the fields of `in` (the entry points differ only in
// where the scratch comes from).
static eas_status encode_impl(eas_encoder* e, const eas_packed_inputs* in, void* workspace, size_t workspace_bytes,
                              const int32_t* cu_dev, int32_t sm_budget, void* stream_v, void* out_embeddings) {
  if (e == nullptr || in == nullptr) return fail(EAS_ERR_INVALID_ARG, "encoder or inputs are null");
  if (in->data == nullptr || in->item_shape == nullptr || in->item_offset == nullptr || in->cu_seqlens_host == nullptr ||
      workspace == nullptr || cu_dev == nullptr || out_embeddings == nullptr)
    return fail(EAS_ERR_INVALID_ARG, "a required pointer is null");
  {
    // the handle's weights, tensor maps and kernel attributes belong to the device it was created on
    int dev = -1;
    CUDA_TRY(cudaGetDevice(&dev));
    if (dev != e->device)
      return fail(EAS_ERR_INVALID_ARG, "the encoder was created on device %d but device %d is current", e->device, dev);
  }
  const int n = in->n_items;
  if (n < 1 || n > EAS_MAX_ITEMS) return fail(EAS_ERR_INVALID_ARG, "n_items %d outside 1..%d", n, static_cast<int>(EAS_MAX_ITEMS));
  if (sm_budget < 0 || sm_budget > e->sm_count) return fail(EAS_ERR_INVALID_ARG, "sm_budget %d outside 0..%d", sm_budget, e->sm_count);
  if ((reinterpret_cast<uintptr_t>(workspace) & 1023) != 0) return fail(EAS_ERR_INVALID_ARG, "workspace is not 1024-byte aligned");
  if ((reinterpret_cast<uintptr_t>(in->data) & 15) != 0 || (reinterpret_cast<uintptr_t>(out_embeddings) & 15) != 0)
    return fail(EAS_ERR_INVALID_ARG, "data / out_embeddings must be 16-byte aligned");
  const int budget = sm_budget == 0 ? e->sm_count : sm_budget;
  g_overlap_launches = budget == e->sm_count;
  const eas_arch_config& c = e->cfg;
  const int32_t* cu = in->cu_seqlens_host;
  const int d = c.d_model;
  const bool audio = c.family == EAS_FAMILY_AUDIO_CONV;
  if (cu[0] != 0) return fail(EAS_ERR_INVALID_ARG, "cu_seqlens must start at 0");

  ItemTable items{};
  items.n_items = n;
  int aux = 0;
  for (int i = 0; i < n; ++i) {
    const int f = in->item_shape[3 * i], h = in->item_shape[3 * i + 1], w = in->item_shape[3 * i + 2];
    const int S = cu[i + 1] - cu[i];
    if (S <= 0) return fail(EAS_ERR_INVALID_ARG, "cu_seqlens is not strictly increasing at item %d", i);
    if (f <= 0 || h <= 0 || w <= 0 || in->item_offset[i] < 0) return fail(EAS_ERR_INVALID_ARG, "item %d has a non-positive shape or negative offset", i);
    int expect;
    items.tok_start[i] = cu[i];
    items.aux_start[i] = aux;
    items.frames[i] = f; items.height[i] = h; items.width[i] = w;
    items.offset[i] = in->item_offset[i];
    if (audio) {
      if (h != c.in_channels || w != 1) return fail(EAS_ERR_INVALID_ARG, "audio item %d must be (frames, %d, 1)", i, c.in_channels);
      if ((in->item_offset[i] * 2) % 16 != 0) return fail(EAS_ERR_INVALID_ARG, "item %d offset is not 16-byte aligned", i);
      // the stride-2 convolution (k = 3, padding 1) yields ceil(f / 2) tokens; the staging rows of an item are one zero
      // row, its f frames, and one zero row (two when f is odd, so that every item starts on an even staging row)
      expect = (f + 1) / 2;
      aux += f + 2 + (f & 1);
    } else {
      const int unit = c.patch * (c.head == EAS_HEAD_MERGER_2X2 ? 2 : 1);
      if (h % unit != 0 || w % unit != 0) return fail(EAS_ERR_INVALID_ARG, "item %d: height/width must be multiples of %d", i, unit);
      if (f % c.temporal_patch != 0) return fail(EAS_ERR_INVALID_ARG, "item %d: frames must be a multiple of %d", i, c.temporal_patch);
      if (c.temporal_patch == 1 && f != 1) return fail(EAS_ERR_INVALID_ARG, "item %d: an image encoder takes one frame", i);
      if (static_cast<long long>(f) * c.in_channels * h * w >= (1LL << 31))
        return fail(EAS_ERR_UNSUPPORTED, "item %d has 2^31 or more elements", i);
      const int patches = (f / c.temporal_patch) * (h / c.patch) * (w / c.patch);
      expect = patches + (c.has_cls ? 1 : 0);
      aux += patches;
    }
    if (S != expect) return fail(EAS_ERR_INVALID_ARG, "item %d: cu_seqlens says %d tokens, its shape gives %d", i, S, expect);
    if (c.pos == EAS_POS_TABLE && S > c.max_pos) return fail(EAS_ERR_INVALID_ARG, "item %d has %d tokens, position table has %d rows", i, S, c.max_pos);
  }
  items.tok_start[n] = cu[n];
  items.aux_start[n] = aux;
  const int64_t T = cu[n];
  const Plan pl = make_plan(e, T, n);
  if (workspace_bytes < pl.total) return fail(EAS_ERR_WORKSPACE, "workspace too small: %zu bytes available, %zu needed", workspace_bytes, pl.total);

  cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  uint32_t* status = reinterpret_cast<uint32_t*>(ws + pl.status);
  float* x = reinterpret_cast<float*>(ws + pl.x);
  bf16* nbuf = reinterpret_cast<bf16*>(ws + pl.n);
  bf16* qkv = reinterpret_cast<bf16*>(ws + pl.qkv);
  bf16* obuf = reinterpret_cast<bf16*>(ws + pl.o);
  bf16* abuf = reinterpret_cast<bf16*>(ws + pl.a);
  int* row_map = reinterpret_cast<int*>(ws + pl.row_map);
  int* pos_idx = reinterpret_cast<int*>(ws + pl.pos_idx);
  int* head_src = reinterpret_cast<int*>(ws + pl.head_src);
  float2* rope = reinterpret_cast<float2*>(ws + pl.rope);
  bf16* mel_pad = reinterpret_cast<bf16*>(ws + pl.mel_pad);
  bf16* h1_pad = reinterpret_cast<bf16*>(ws + pl.h1_pad);
  int* conv1_map = reinterpret_cast<int*>(ws + pl.conv1_map);
  float* part = reinterpret_cast<float*>(ws + pl.part);
  float2* stats = reinterpret_cast<float2*>(ws + pl.stats);
  // Folded normalisation: the blocks' norm1 / norm2 run inside the GEMMs around them (GemmParams::fold_stats) unless the
  // residual GEMMs split K, whose partial sums a normalisation kernel has to add.
  const bool fold = e->fold != 0 && c.n_layers > 0 && pl.splits_proj == 1 && pl.splits_fc2 == 1;
  int pending_parts = 0;      // split-K partial sums of the last residual GEMM, to be added by the next normalisation
  int launches = 0;
  e->last_status = status;

  CUDA_TRY(cudaMemsetAsync(status, 0, 16, stream));
  e->tcls.clear();
  EAS_TRY(mark(e, EAS_KC_PREP, stream));

  // ---- tables: row maps, rotary (cos, sin), CLS rows
  {
    PrepParams pp{};
    pp.items = items;
    pp.family = c.family; pp.has_cls = c.has_cls; pp.patch = c.patch; pp.d_model = d;
    pp.total_tokens = static_cast<int>(T); pp.n_embed_rows = static_cast<int>(pl.embed_rows);
    pp.rope_pairs = e->hd / 2; pp.rope_theta = c.rope_theta;
    pp.cu_seqlens_dev = cu_dev;
    pp.embed_row_map = row_map; pp.embed_pos_idx = pos_idx;
    pp.head_src_rows = c.head == EAS_HEAD_MLP_PROJECTOR ? head_src : nullptr;
    pp.rope_cs = rope; pp.x = x; pp.cls = e->cls; pp.pos = e->pos;
    pp.conv1_row_map = conv1_map; pp.n_conv1_rows = static_cast<int>(pl.padded_rows);
    pp.status = status;
    EAS_TRY(launch_kernel(prep_kernel, budget, 256, 0, stream, pp));
    ++launches;
  }

  // ---- embedding
  const int ln_kind = c.norm == EAS_NORM_LAYERNORM ? NORM_LN : NORM_RMS;
  if (audio) {
    AudioStageParams sp{};
    sp.data = static_cast<const bf16*>(in->data); sp.mel_pad = mel_pad; sp.h1_pad = h1_pad;
    sp.n_mel = c.in_channels; sp.d_model = d; sp.padded_rows = static_cast<int>(pl.padded_rows); sp.items = items;
    static OncePerDevice once;
    if (once.first()) {
      CUDA_TRY(cudaFuncSetAttribute(audio_stage_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kOnePerSmSmem));
      once.settled();
    }
    EAS_TRY(mark(e, EAS_KC_EMBED_GATHER, stream));
    EAS_TRY(launch_kernel(audio_stage_kernel, budget, 512, kOnePerSmSmem, stream, sp));
    ++launches;
    GemmCall g1;   // conv1 (k=3, stride 1) + GELU -> padded h1
    g1.A = mel_pad; g1.a_run = c.in_channels; g1.a_row_elems = c.in_channels; g1.conv_stride = 1; g1.taps = 3;
    g1.a_rows = pl.padded_rows; g1.M = static_cast<int>(pl.padded_rows); g1.lin = &e->conv1; g1.act = ACT_GELU;
    g1.out = h1_pad; g1.ldo = d; g1.row_map = conv1_map;
    EAS_TRY(mark(e, EAS_KC_GEMM_EMBED, stream));
    EAS_TRY(launch_gemm(g1, budget, stream, status)); ++launches;
    GemmCall g2;   // conv2 (k=3, stride 2) + GELU + position table -> residual stream
    g2.A = h1_pad; g2.a_run = d; g2.a_row_elems = d; g2.conv_stride = 2; g2.taps = 3;
    g2.a_rows = pl.padded_rows; g2.M = static_cast<int>(pl.embed_rows); g2.lin = &e->conv2; g2.act = ACT_GELU; g2.out_fp32 = 1;
    g2.out = x; g2.ldo = d; g2.row_map = row_map; g2.pos_idx = pos_idx; g2.pos = e->pos;
    EAS_TRY(mark(e, EAS_KC_GEMM_EMBED, stream));
    EAS_TRY(launch_gemm(g2, budget, stream, status)); ++launches;
  } else {
    // patch embedding: the im2col gather is the GEMM's A producer (no patch matrix in global memory)
    EmbedGemmParams gp{};
    gp.tma_w = e->embed.tmap;
    gp.data = static_cast<const bf16*>(in->data); gp.bias = e->embed.b; gp.x = x;
    gp.row_map = row_map;
    if (c.pos == EAS_POS_TABLE) { gp.pos_idx = pos_idx; gp.pos = e->pos; }
    gp.n_patches = static_cast<int>(pl.embed_rows); gp.N = d; gp.k = e->embed_k; gp.k_pad = e->embed_k_pad;
    gp.channels = c.in_channels; gp.patch = c.patch; gp.tpatch = c.temporal_patch;
    gp.merge_order = c.family == EAS_FAMILY_VIT_ROPE_MERGER ? 1 : 0;
    gp.pairs_ok = (c.patch % 2 == 0 && (reinterpret_cast<uintptr_t>(in->data) & 3) == 0) ? 1 : 0;
    for (int i = 0; i < n && gp.pairs_ok; ++i)
      if ((in->item_offset[i] & 1) != 0 || (in->item_shape[3 * i + 2] & 1) != 0) gp.pairs_ok = 0;
    gp.table = e->embed_table;
    gp.status = status;
    gp.items = items;
    static OncePerDevice once;
    if (once.first()) {
      CUDA_TRY(cudaFuncSetAttribute(embed_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kEgSmemBytes));
      once.settled();
    }
    const int tiles = static_cast<int>((pl.embed_rows + 127) / 128);     // a CTA owns whole blocks of 128 patches
    EAS_TRY(mark(e, EAS_KC_GEMM_EMBED, stream));
    EAS_TRY(launch_kernel(embed_gemm_kernel, std::min(budget, tiles), kEgThreads, kEgSmemBytes, stream, gp));
    ++launches;
  }
  if (c.embed_norm) {
    NormParams np{x, x, e->eng, e->enb, nullptr, static_cast<int>(T), d, c.norm_eps};
    EAS_TRY(mark(e, EAS_KC_NORM, stream));
    EAS_TRY(launch_norm(ln_kind, true, np, budget, stream)); ++launches;
  }

  // ---- transformer blocks
  // Consecutive kernels walk the token rows in alternating directions (`dir`): each starts with the rows its producer
  // wrote last, which are the ones still in L2.  Every row, tile and attention unit is independent of the order.
  int dir = 0;
  if (fold) {
    // the first block's rows come from the embedding: their bf16 copy and group statistics from a kernel of its own
    FoldStatsParams fp{x, nbuf, stats, e->layers[0].n1g, static_cast<int>(T), d};
    EAS_TRY(mark(e, EAS_KC_NORM, stream));
    EAS_TRY(launch_fold_stats(fp, budget, stream)); ++launches;
  }
  auto fold_in = [&](GemmCall& g, const float* c0, const float* c1) {    // a GEMM on rows scaled by gamma only
    g.fold_stats = stats; g.fold_c0 = c0; g.fold_c1 = ln_kind == NORM_LN ? c1 : nullptr;
    g.fold_rms = ln_kind == NORM_RMS ? 1 : 0; g.fold_eps = c.norm_eps; g.fold_rows = T;
  };
  for (int li = 0; li < c.n_layers; ++li) {
    const Layer& L = e->layers[li];
    if (!fold) {
      NormParams np{x, nbuf, L.n1g, L.n1b, nullptr, static_cast<int>(T), d, c.norm_eps};
      np.part = part; np.part_stride = pl.part_rows * d; np.n_part = pending_parts; np.x_rw = x; pending_parts = 0;
      np.reverse = dir; dir ^= 1;
      EAS_TRY(mark(e, EAS_KC_NORM, stream));
      EAS_TRY(launch_norm(ln_kind, false, np, budget, stream)); ++launches;
    }
    {
      GemmCall g;
      g.A = nbuf; g.a_run = d; g.a_row_elems = d; g.a_rows = T; g.M = static_cast<int>(T); g.lin = &L.qkv;
      if (fold) fold_in(g, L.qkv_c0, L.qkv_c1);
      g.out = qkv; g.ldo = 3LL * d;
      if (c.pos == EAS_POS_ROPE_2D) { g.rope_cs = rope; g.rope_stride = T; g.rope_pairs = e->hd / 2; g.rope_ncols = 2 * d; g.head_dim = e->hd; }
      g.reverse = dir; dir ^= 1;
      EAS_TRY(mark(e, EAS_KC_GEMM_QKV, stream));
      EAS_TRY(launch_gemm(g, budget, stream, status)); ++launches;
    }
    EAS_TRY(mark(e, EAS_KC_ATTENTION, stream));
    EAS_TRY(launch_attention(qkv, obuf, cu, n, c.n_heads, e->hd, budget, stream, e->attn_impl, status, dir != 0)); ++launches;
    dir ^= 1;
    {
      GemmCall g;
      g.A = obuf; g.a_run = d; g.a_row_elems = d; g.a_rows = T; g.M = static_cast<int>(T); g.lin = &L.proj;
      g.out_fp32 = 1; g.out = x; g.ldo = d; g.resid = x;
      g.splits = pl.splits_proj; g.part = part; g.part_rows = pl.part_rows; pending_parts = g.splits - 1;   // norm2 follows
      if (fold) { g.fold_stats_out = stats; g.fold_xb = nbuf; g.fold_gamma = L.n2g; g.fold_rows = T; }
      g.reverse = dir; dir ^= 1;
      EAS_TRY(mark(e, EAS_KC_GEMM_PROJ, stream));
      EAS_TRY(launch_gemm(g, budget, stream, status)); ++launches;
    }
    if (!fold) {
      NormParams np{x, nbuf, L.n2g, L.n2b, nullptr, static_cast<int>(T), d, c.norm_eps};
      np.part = part; np.part_stride = pl.part_rows * d; np.n_part = pending_parts; np.x_rw = x; pending_parts = 0;
      np.reverse = dir; dir ^= 1;
      EAS_TRY(mark(e, EAS_KC_NORM, stream));
      EAS_TRY(launch_norm(ln_kind, false, np, budget, stream)); ++launches;
    }
    {
      GemmCall g;
      g.A = nbuf; g.a_run = d; g.a_row_elems = d; g.a_rows = T; g.M = static_cast<int>(T); g.lin = &L.fc1;
      g.act = c.mlp == EAS_MLP_SWIGLU ? ACT_SWIGLU : ACT_GELU;
      if (fold) fold_in(g, L.fc1_c0, L.fc1_c1);
      g.out = abuf; g.ldo = c.d_mlp;
      g.reverse = dir; dir ^= 1;
      EAS_TRY(mark(e, EAS_KC_GEMM_FC1, stream));
      EAS_TRY(launch_gemm(g, budget, stream, status)); ++launches;
    }
    {
      GemmCall g;
      g.A = abuf; g.a_run = c.d_mlp; g.a_row_elems = c.d_mlp; g.a_rows = T; g.M = static_cast<int>(T); g.lin = &L.fc2;
      g.out_fp32 = 1; g.out = x; g.ldo = d; g.resid = x;
      if (li + 1 < c.n_layers) {      // the next block's first normalisation adds the partial sums
        g.splits = pl.splits_fc2; g.part = part; g.part_rows = pl.part_rows; pending_parts = g.splits - 1;
        if (fold) { g.fold_stats_out = stats; g.fold_xb = nbuf; g.fold_gamma = e->layers[li + 1].n1g; g.fold_rows = T; }
      }
      g.reverse = dir; dir ^= 1;
      EAS_TRY(mark(e, EAS_KC_GEMM_FC2, stream));
      EAS_TRY(launch_gemm(g, budget, stream, status)); ++launches;
    }
  }

  // ---- connector
  EAS_TRY(mark(e, EAS_KC_NORM, stream));
  const bool out_f32 = c.out_dtype == EAS_OUT_FP32;
  if (c.head == EAS_HEAD_NONE) {
    if (c.final_norm) {
      NormParams np{x, out_embeddings, e->fng, e->fnb, nullptr, static_cast<int>(T), d, c.norm_eps};
      EAS_TRY(launch_norm(ln_kind, out_f32, np, budget, stream)); ++launches;
    } else {
      NormParams np{x, out_embeddings, nullptr, nullptr, nullptr, static_cast<int>(T), d, c.norm_eps};
      EAS_TRY(launch_norm(NORM_CAST, out_f32, np, budget, stream)); ++launches;
    }
  } else {
    int64_t rows_in;   // rows of the connector's first GEMM
    int64_t k_in;
    if (c.head == EAS_HEAD_MLP_PROJECTOR) {
      rows_in = pl.out_rows; k_in = d;
      NormParams np{x, nbuf, nullptr, nullptr, c.has_cls ? head_src : nullptr, static_cast<int>(rows_in), d, c.norm_eps};
      EAS_TRY(launch_norm(NORM_CAST, false, np, budget, stream)); ++launches;
    } else {
      // RMSNorm per token; four consecutive tokens (one 2x2 group) then form one row of width 4d
      rows_in = T / 4; k_in = 4LL * d;
      NormParams np{x, nbuf, e->hng, nullptr, nullptr, static_cast<int>(T), d, c.norm_eps};
      EAS_TRY(launch_norm(NORM_RMS, false, np, budget, stream)); ++launches;
    }
    GemmCall g1;
    g1.A = nbuf; g1.a_run = k_in; g1.a_row_elems = k_in; g1.a_rows = rows_in; g1.M = static_cast<int>(rows_in); g1.lin = &e->head1;
    g1.act = ACT_GELU; g1.out = abuf; g1.ldo = c.d_head_hidden;
    EAS_TRY(mark(e, EAS_KC_GEMM_HEAD, stream));
    EAS_TRY(launch_gemm(g1, budget, stream, status)); ++launches;
    GemmCall g2;
    g2.A = abuf; g2.a_run = c.d_head_hidden; g2.a_row_elems = c.d_head_hidden; g2.a_rows = rows_in; g2.M = static_cast<int>(rows_in); g2.lin = &e->head2;
    g2.out = out_embeddings; g2.ldo = c.d_out; g2.out_fp32 = out_f32 ? 1 : 0;
    EAS_TRY(mark(e, EAS_KC_GEMM_HEAD, stream));
    EAS_TRY(launch_gemm(g2, budget, stream, status)); ++launches;
  }
  EAS_TRY(mark(e, -1, stream));
  e->last_launches = launches;
  return EAS_OK;
}

// The forward pass through the graph cache.  A micro-batch is identified by everything the launches depend on:
// item shapes and offsets, cu_seqlens, the SM budget, the attention variant and every pointer.  A hit replays the
// captured launches (one driver call instead of one per kernel); a miss captures them from the ordinary code path,
// so the kernels and their arguments are the same either way.
static eas_status encode_cached(eas_encoder* e, const eas_packed_inputs* in, void* workspace, size_t workspace_bytes,
                                const int32_t* cu_dev, int32_t sm_budget, void* stream_v, void* out_embeddings) {
  cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
  const bool usable = e != nullptr && e->graph_mode != 0 && !e->timing && in != nullptr && in->item_shape != nullptr &&
                      in->item_offset != nullptr && in->cu_seqlens_host != nullptr && in->n_items >= 1 &&
                      in->n_items <= EAS_MAX_ITEMS && stream != nullptr && stream != cudaStreamLegacy &&
                      stream != cudaStreamPerThread;
  if (!usable) return encode_impl(e, in, workspace, workspace_bytes, cu_dev, sm_budget, stream_v, out_embeddings);
  const int n = in->n_items;
  std::vector<int64_t> key;
  key.reserve(8 + 5 * static_cast<size_t>(n) + 1);
  key.push_back(n); key.push_back(sm_budget); key.push_back(e->attn_impl * 4 + e->split_k * 2 + e->fold);
  key.push_back(static_cast<int64_t>(reinterpret_cast<uintptr_t>(in->data)));
  key.push_back(static_cast<int64_t>(reinterpret_cast<uintptr_t>(workspace)));
  key.push_back(static_cast<int64_t>(workspace_bytes));
  key.push_back(static_cast<int64_t>(reinterpret_cast<uintptr_t>(cu_dev)));
  key.push_back(static_cast<int64_t>(reinterpret_cast<uintptr_t>(out_embeddings)));
  for (int i = 0; i < 3 * n; ++i) key.push_back(in->item_shape[i]);
  for (int i = 0; i < n; ++i) key.push_back(in->item_offset[i]);
  for (int i = 0; i <= n; ++i) key.push_back(in->cu_seqlens_host[i]);
  ++e->graph_clock;
  for (GraphEntry& g : e->graphs) {
    if (g.key == key) {
      g.last_use = e->graph_clock;
      e->last_launches = g.launches;
      e->last_status = g.status;
      ++e->graph_hits;
      CUDA_TRY(cudaGraphLaunch(g.exec, stream));
      return EAS_OK;
    }
  }
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  CUDA_TRY(cudaStreamIsCapturing(stream, &cap));
  if (cap != cudaStreamCaptureStatusNone)     // the caller is capturing this stream itself: just add the launches
    return encode_impl(e, in, workspace, workspace_bytes, cu_dev, sm_budget, stream_v, out_embeddings);
  CUDA_TRY(cudaStreamBeginCapture(stream, cudaStreamCaptureModeRelaxed));
  const eas_status st = encode_impl(e, in, workspace, workspace_bytes, cu_dev, sm_budget, stream_v, out_embeddings);
  cudaGraph_t graph = nullptr;
  const cudaError_t end = cudaStreamEndCapture(stream, &graph);
  if (st != EAS_OK) {                         // nothing was launched; the message of the failed step stands
    if (graph) cudaGraphDestroy(graph);
    (void)cudaGetLastError();
    return st;
  }
  if (end != cudaSuccess || graph == nullptr) {
    if (graph) cudaGraphDestroy(graph);
    return fail(EAS_ERR_CUDA, "stream capture of the forward pass failed: %s", cudaGetErrorString(end));
  }
  GraphEntry g;
  const cudaError_t inst = cudaGraphInstantiate(&g.exec, graph, 0);
  cudaGraphDestroy(graph);
  if (inst != cudaSuccess) return fail(EAS_ERR_CUDA, "cudaGraphInstantiate failed: %s", cudaGetErrorString(inst));
  g.key = std::move(key);
  g.launches = e->last_launches;
  g.status = e->last_status;
  g.last_use = e->graph_clock;
  if (e->graphs.size() >= kMaxGraphs) {       // evict the least recently used capture
    size_t victim = 0;
    for (size_t i = 1; i < e->graphs.size(); ++i) if (e->graphs[i].last_use < e->graphs[victim].last_use) victim = i;
    cudaGraphExecDestroy(e->graphs[victim].exec);
    e->graphs[victim] = std::move(g);
    ++e->graph_captures;
    CUDA_TRY(cudaGraphLaunch(e->graphs[victim].exec, stream));
    return EAS_OK;
  }
  e->graphs.push_back(std::move(g));
  ++e->graph_captures;
  CUDA_TRY(cudaGraphLaunch(e->graphs.back().exec, stream));
  return EAS_OK;
}

extern "C" eas_status eas_encode_microbatch(eas_encoder* e, const eas_packed_inputs* in, const int32_t* cu_dev,
                                            int32_t sm_budget, void* stream_v, void* out_embeddings) {
  if (in == nullptr) return fail(EAS_ERR_INVALID_ARG, "encoder or inputs are null");
  return encode_cached(e, in, in->workspace, in->workspace_bytes, cu_dev, sm_budget, stream_v, out_embeddings);
}

extern "C" eas_status eas_encoder_set_graph_mode(eas_encoder* e, int32_t mode) {
  if (e == nullptr) return fail(EAS_ERR_INVALID_ARG, "encoder is null");
  if (mode != 0 && mode != 1) return fail(EAS_ERR_INVALID_ARG, "graph mode %d (0 = off, 1 = on)", mode);
  e->graph_mode = mode;
  if (mode == 0) {
    for (GraphEntry& g : e->graphs) if (g.exec) cudaGraphExecDestroy(g.exec);
    e->graphs.clear();
  }
  return EAS_OK;
}

extern "C" eas_status eas_encoder_graph_stats(const eas_encoder* e, int64_t* hits, int64_t* captures, int32_t* cached) {
  if (e == nullptr) return fail(EAS_ERR_INVALID_ARG, "encoder is null");
  if (hits) *hits = e->graph_hits;
  if (captures) *captures = e->graph_captures;
  if (cached) *cached = static_cast<int32_t>(e->graphs.size());
  return EAS_OK;
}

// ------------------------------------------------------------------------------------ scratch baked into the library
// Scratch for callers that must not allocate: it lives in the library image, so every GPU that loads the
// library carries it until the process exits.  In host code the array's name is only a host-side stand-in, never
// a device address: the address is obtained per device with cudaGetSymbolAddress and handed to the kernels.
static __device__ __align__(256) unsigned char g_static_scratch[EAS_STATIC_WORKSPACE_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
unsigned char* g_static_ptr[kMaxDevices] = {};   // device address of g_static_scratch on each device, once known
}  // namespace

extern "C" eas_status eas_encode_microbatch_static(eas_encoder* e, const eas_packed_inputs* in, const int32_t* cu_dev,
                                                   int32_t sm_budget, void* stream_v, void* out_embeddings) {
  int dev = 0;
  CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return fail(EAS_ERR_UNSUPPORTED, "device ordinal %d", dev);
  if (e != nullptr && dev != e->device)
    return fail(EAS_ERR_INVALID_ARG, "the encoder was created on device %d but device %d is current", e->device, dev);
  unsigned char* base = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (g_static_ptr[dev] == nullptr) {
      // first call on this device (the device is current): look the symbol's device address up once
      void* sym = nullptr;
      CUDA_TRY(cudaGetSymbolAddress(&sym, g_static_scratch));
      if (sym == nullptr) return fail(EAS_ERR_CUDA, "cudaGetSymbolAddress returned a null address");
      g_static_ptr[dev] = static_cast<unsigned char*>(sym);
    }
    base = g_static_ptr[dev];
  }
  // the forward pass wants its scratch on a 1024-byte boundary; the array itself is only 256-byte aligned
  const uintptr_t aligned = (reinterpret_cast<uintptr_t>(base) + 1023) & ~uintptr_t(1023);
  const size_t usable = EAS_STATIC_WORKSPACE_BYTES - (aligned - reinterpret_cast<uintptr_t>(base));
  if (e != nullptr && in != nullptr && in->cu_seqlens_host != nullptr && in->n_items >= 1 && in->n_items <= EAS_MAX_ITEMS) {
    const int64_t T = in->cu_seqlens_host[in->n_items];
    if (T > 0) {
      const size_t need = make_plan(e, T, in->n_items).total;
      if (need > usable)
        return fail(EAS_ERR_WORKSPACE,
                    "micro-batch needs %zu bytes of scratch but the built-in scratch holds %zu: use eas_encode_microbatch "
                    "with a caller-allocated workspace, or send fewer / smaller items", need, usable);
    }
  }
  return encode_cached(e, in, reinterpret_cast<void*>(aligned), usable, cu_dev, sm_budget, stream_v, out_embeddings);
}

extern "C" eas_status eas_encoder_enable_timing(eas_encoder* e, int32_t on) {
  if (e == nullptr) return fail(EAS_ERR_INVALID_ARG, "encoder is null");
  e->timing = on != 0;
  e->tcls.clear();
  return EAS_OK;
}

extern "C" int32_t eas_encoder_timing_read(eas_encoder* e, int32_t capacity, int32_t* kernel_class, float* ms) {
  if (e == nullptr || e->tcls.size() < 2) return 0;
  const int n = static_cast<int>(e->tcls.size()) - 1;
  if (kernel_class == nullptr || ms == nullptr) return n;
  if (cudaEventSynchronize(e->tev[n]) != cudaSuccess) return -1;
  const int m = std::min(n, capacity);
  for (int i = 0; i < m; ++i) {
    kernel_class[i] = e->tcls[i];
    if (cudaEventElapsedTime(&ms[i], e->tev[i], e->tev[i + 1]) != cudaSuccess) return -1;
  }
  return m;
}

extern "C" eas_status eas_encoder_status(eas_encoder* e, void* stream_v) {
  if (e == nullptr) return fail(EAS_ERR_INVALID_ARG, "encoder is null");
  cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
  CUDA_TRY(cudaStreamSynchronize(stream));
  if (e->last_status == nullptr) return EAS_OK;
  uint32_t v = 0;
  CUDA_TRY(cudaMemcpy(&v, e->last_status, 4, cudaMemcpyDeviceToHost));
  if (v != DEV_OK) CUDA_TRY(cudaMemset(e->last_status, 0, 4));
  if (v == DEV_ERR_WAIT_TIMEOUT) return fail(EAS_ERR_DEVICE_TIMEOUT, "a bounded device-side wait expired");
  if (v == DEV_ERR_CU_SEQLENS_MISMATCH) return fail(EAS_ERR_DEVICE_CHECK, "device cu_seqlens differs from cu_seqlens_host");
  if (v != DEV_OK) return fail(EAS_ERR_DEVICE_CHECK, "device status %u", v);
  return EAS_OK;
}

// ------------------------------------------------------------------------------------ SM partition (Section 3.4)
// Two green contexts over disjoint sets of SMs, one stream in each.  The driver calls are looked up at run time (the
// library does not link libcuda).
namespace {
template <typename Fn>
Fn driver_fn(const char* name) {
  void* p = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint(name, &p, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess) return nullptr;
  return reinterpret_cast<Fn>(p);
}
struct GreenApi {
  CUresult (*device_get)(CUdevice*, int) = nullptr;
  CUresult (*get_resource)(CUdevice, CUdevResource*, CUdevResourceType) = nullptr;
  CUresult (*split)(CUdevResource*, unsigned int*, const CUdevResource*, CUdevResource*, unsigned int, unsigned int) = nullptr;
  CUresult (*gen_desc)(CUdevResourceDesc*, CUdevResource*, unsigned int) = nullptr;
  CUresult (*ctx_create)(CUgreenCtx*, CUdevResourceDesc, CUdevice, unsigned int) = nullptr;
  CUresult (*ctx_destroy)(CUgreenCtx) = nullptr;
  CUresult (*stream_create)(CUstream*, CUgreenCtx, unsigned int, int) = nullptr;
  bool load() {
    device_get = driver_fn<decltype(device_get)>("cuDeviceGet");
    get_resource = driver_fn<decltype(get_resource)>("cuDeviceGetDevResource");
    split = driver_fn<decltype(split)>("cuDevSmResourceSplitByCount");
    gen_desc = driver_fn<decltype(gen_desc)>("cuDevResourceGenerateDesc");
    ctx_create = driver_fn<decltype(ctx_create)>("cuGreenCtxCreate");
    ctx_destroy = driver_fn<decltype(ctx_destroy)>("cuGreenCtxDestroy");
    stream_create = driver_fn<decltype(stream_create)>("cuGreenCtxStreamCreate");
    return device_get && get_resource && split && gen_desc && ctx_create && ctx_destroy && stream_create;
  }
};
}  // namespace

struct eas_sm_partition {
  GreenApi api;
  CUgreenCtx ctx[2] = {nullptr, nullptr};
  CUstream stream[2] = {nullptr, nullptr};
  int32_t sm_count[2] = {0, 0};
};

extern "C" void eas_sm_partition_destroy(eas_sm_partition* p) {
  if (p == nullptr) return;
  for (int s = 0; s < 2; ++s) {
    if (p->stream[s] != nullptr) { cudaStreamSynchronize(p->stream[s]); cudaStreamDestroy(p->stream[s]); }
    if (p->ctx[s] != nullptr) p->api.ctx_destroy(p->ctx[s]);
  }
  delete p;
}

extern "C" eas_status eas_sm_partition_create(int32_t sm_encode, eas_sm_partition** out) {
  if (out == nullptr) return fail(EAS_ERR_INVALID_ARG, "eas_sm_partition_create: out is NULL");
  *out = nullptr;
  if (sm_encode <= 0) return fail(EAS_ERR_INVALID_ARG, "eas_sm_partition_create: sm_encode = %d", sm_encode);
  int dev = 0;
  CUDA_TRY(cudaGetDevice(&dev));
  CUDA_TRY(cudaFree(nullptr));                       // the primary context exists from here on
  std::unique_ptr<eas_sm_partition, void (*)(eas_sm_partition*)> p(new eas_sm_partition, eas_sm_partition_destroy);
  if (!p->api.load()) return fail(EAS_ERR_UNSUPPORTED, "this driver has no green contexts");
  CUdevice cudev;
  CUdevResource all, part[2];
  CUresult r = p->api.device_get(&cudev, dev);
  if (r == CUDA_SUCCESS) r = p->api.get_resource(cudev, &all, CU_DEV_RESOURCE_TYPE_SM);
  if (r != CUDA_SUCCESS) return fail(EAS_ERR_CUDA, "cuDeviceGetDevResource failed with code %d", static_cast<int>(r));
  if (sm_encode >= static_cast<int32_t>(all.sm.smCount))
    return fail(EAS_ERR_INVALID_ARG, "eas_sm_partition_create: sm_encode = %d leaves nothing of %u SMs", sm_encode, all.sm.smCount);
  unsigned int groups = 1;
  r = p->api.split(&part[0], &groups, &all, &part[1], 0, static_cast<unsigned int>(sm_encode));
  if (r != CUDA_SUCCESS || groups != 1)
    return fail(EAS_ERR_CUDA, "cuDevSmResourceSplitByCount(%d) failed with code %d (%u groups)", sm_encode, static_cast<int>(r), groups);
  if (part[1].sm.smCount == 0)
    return fail(EAS_ERR_INVALID_ARG, "eas_sm_partition_create: %d SMs round up to %u and leave none", sm_encode, part[0].sm.smCount);
  for (int s = 0; s < 2; ++s) {
    CUdevResourceDesc desc;
    r = p->api.gen_desc(&desc, &part[s], 1);
    if (r == CUDA_SUCCESS) r = p->api.ctx_create(&p->ctx[s], desc, cudev, CU_GREEN_CTX_DEFAULT_STREAM);
    if (r == CUDA_SUCCESS) r = p->api.stream_create(&p->stream[s], p->ctx[s], CU_STREAM_NON_BLOCKING, 0);
    if (r != CUDA_SUCCESS) return fail(EAS_ERR_CUDA, "creating the green context of side %d failed with code %d", s, static_cast<int>(r));
    p->sm_count[s] = static_cast<int32_t>(part[s].sm.smCount);
  }
  *out = p.release();
  return EAS_OK;
}

extern "C" int32_t eas_sm_partition_sm_count(const eas_sm_partition* p, int32_t side) {
  return (p != nullptr && (side == 0 || side == 1)) ? p->sm_count[side] : 0;
}

extern "C" void* eas_sm_partition_stream(const eas_sm_partition* p, int32_t side) {
  return (p != nullptr && (side == 0 || side == 1)) ? static_cast<void*>(p->stream[side]) : nullptr;
}

// ------------------------------------------------------------------------------------ single-kernel entry points
static eas_status resolve_budget(int32_t sm_budget, int* budget) {
  int sm_count = 0;
  EAS_TRY(device_check(&sm_count));
  if (sm_budget < 0 || sm_budget > sm_count) return fail(EAS_ERR_INVALID_ARG, "sm_budget %d outside 0..%d", sm_budget, sm_count);
  *budget = sm_budget == 0 ? sm_count : sm_budget;
  g_overlap_launches = *budget == sm_count;
  return EAS_OK;
}

extern "C" eas_status eas_kernel_gemm(const void* A, const void* W, const void* bias, void* out, const float* resid,
                                      int32_t M, int32_t N, int32_t K, int32_t act, int32_t out_fp32, int32_t sm_budget,
                                      void* stream, uint32_t* status_dev) {
  return eas_kernel_gemm_tile(A, W, bias, out, resid, M, N, K, act, out_fp32, sm_budget, stream, status_dev, 0);
}

extern "C" eas_status eas_kernel_gemm_tile(const void* A, const void* W, const void* bias, void* out, const float* resid,
                                           int32_t M, int32_t N, int32_t K, int32_t act, int32_t out_fp32, int32_t sm_budget,
                                           void* stream, uint32_t* status_dev, int32_t tile_shape) {
  if (tile_shape < 0 || tile_shape > 3) return fail(EAS_ERR_INVALID_ARG, "tile_shape %d outside 0..3", tile_shape);
  if (A == nullptr || W == nullptr || bias == nullptr || out == nullptr || status_dev == nullptr)
    return fail(EAS_ERR_INVALID_ARG, "a required pointer is null");
  if (M <= 0 || N <= 0 || K <= 0 || K % 64 != 0 || N % 32 != 0) return fail(EAS_ERR_INVALID_ARG, "need M,N,K > 0, K %% 64 == 0, N %% 32 == 0");
  if (act < 0 || act > 2 || (act == ACT_SWIGLU && out_fp32)) return fail(EAS_ERR_INVALID_ARG, "bad epilogue selection");
  int budget = 0;
  EAS_TRY(resolve_budget(sm_budget, &budget));
  EAS_TRY(set_kernel_attributes_once());
  Linear L;
  L.w = static_cast<const bf16*>(W); L.b = static_cast<const bf16*>(bias); L.N = N; L.K = K;
  EAS_TRY(finish_linear(L));
  GemmCall g;
  g.A = A; g.a_run = K; g.a_row_elems = K; g.a_rows = M; g.M = M; g.lin = &L; g.act = act; g.out_fp32 = out_fp32;
  g.out = out; g.ldo = act == ACT_SWIGLU ? N / 2 : N; g.resid = out_fp32 ? resid : nullptr;
  g.w_const = 0;             // W is the caller's tensor: work earlier in the stream may have produced it
  g.force_tile = budget >= 2 ? tile_shape : 0;
  return launch_gemm(g, budget, static_cast<cudaStream_t>(stream), status_dev);
}

extern "C" eas_status eas_kernel_norm(const float* x, void* y, const void* gamma, const void* beta, int32_t rows, int32_t d,
                                      int32_t kind, float eps, int32_t out_fp32, int32_t sm_budget, void* stream) {
  if (x == nullptr || y == nullptr || rows <= 0) return fail(EAS_ERR_INVALID_ARG, "bad arguments");
  if ((kind == NORM_LN && (gamma == nullptr || beta == nullptr)) || (kind == NORM_RMS && gamma == nullptr))
    return fail(EAS_ERR_INVALID_ARG, "gamma/beta missing");
  int budget = 0;
  EAS_TRY(resolve_budget(sm_budget, &budget));
  NormParams np{x, y, static_cast<const bf16*>(gamma), static_cast<const bf16*>(beta), nullptr, rows, d, eps};
  return launch_norm(kind, out_fp32 != 0, np, budget, static_cast<cudaStream_t>(stream));
}

extern "C" eas_status eas_kernel_attention(const void* qkv, void* out, const int32_t* cu, int32_t n_items, int32_t n_heads,
                                           int32_t head_dim, int32_t sm_budget, void* stream, int32_t impl, uint32_t* status_dev) {
  if (qkv == nullptr || out == nullptr || cu == nullptr || status_dev == nullptr) return fail(EAS_ERR_INVALID_ARG, "a required pointer is null");
  if (n_items < 1 || n_items > EAS_MAX_ITEMS || n_heads <= 0) return fail(EAS_ERR_INVALID_ARG, "bad sizes");
  if (head_dim != 64 && head_dim != 80) return fail(EAS_ERR_UNSUPPORTED, "head_dim %d", head_dim);
  for (int i = 0; i < n_items; ++i)
    if (cu[i + 1] <= cu[i]) return fail(EAS_ERR_INVALID_ARG, "cu_seqlens is not strictly increasing");
  int budget = 0;
  EAS_TRY(resolve_budget(sm_budget, &budget));
  return launch_attention(static_cast<const bf16*>(qkv), static_cast<bf16*>(out), cu, n_items, n_heads, head_dim, budget,
                          static_cast<cudaStream_t>(stream), impl, status_dev);
}

#ifdef EAS_GEMM_PROFILE
extern "C" int eas_debug_gemm_stamps(unsigned long long* host_out /* [32*16] */) {
  return cudaMemcpyFromSymbol(host_out, eas::g_gemm_dbg, sizeof(unsigned long long) * 32 * 16) == cudaSuccess ? 0 : 1;
}
#endif
#ifdef EAS_ATTN_PROFILE
extern "C" int eas_debug_attn_stamps(unsigned long long* host_out /* [2*64*12] */) {
  return cudaMemcpyFromSymbol(host_out, eas::g_attn_dbg, sizeof(unsigned long long) * 2 * 64 * 12) == cudaSuccess ? 0 : 1;
}
#endif
