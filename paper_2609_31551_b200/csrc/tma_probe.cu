// Stand-alone probe: what bounds the L2 -> shared-memory path of a CTA that streams GEMM operand tiles with TMA?
//
// Every CTA (one per SM, 148 of them) walks the tiles of an 18432 x 4096 x 1024 GEMM in the encoder's panel order and
// loads, per k-step, the A and W boxes a GEMM CTA would load into a shared-memory ring; a second thread hands each
// stage straight back (no MMA).  Variants differ in the number of TMA operations per step, their size, whether tiles
// are shared between CTAs, and whether one or two threads issue the operations.  Findings on B200 (the numbers the
// GEMM kernel's "deep" stages and its two producer warps are built on):
//   * a step costs about 290 ns + 70 ns per operation, almost independent of the operation's size up to 64 KB:
//     two 16 KB boxes 458 ns (10.6 TB/s over 148 SMs), two 32 KB boxes 476 ns (20.4 TB/s), eight 4 KB boxes 845 ns;
//   * whether the CTAs read the same tiles or private ones makes no difference (no hot spots in L2);
//   * the ~70 ns per operation are spent by the ISSUING THREAD: with one thread per operand the two-box step takes
//     380 ns instead of 458.
// Every wait is bounded; a wait that expires is reported and the kernel returns.
// Build and run:  python -m paper_2609_31551_b200.tma_probe
#include <cuda.h>
#include <cuda_runtime.h>
#include <cstdio>
#include <cstdint>
#include <cstdlib>
#include <vector>
#define CK(x) do { cudaError_t e = (x); if (e != cudaSuccess) { printf("cuda error %s at %d\n", cudaGetErrorString(e), __LINE__); exit(1); } } while (0)
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void mbar_init(uint64_t* b, uint32_t c) { asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(b)), "r"(c)); }
__device__ __forceinline__ void mbar_expect(uint64_t* b, uint32_t bytes) { asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(b)), "r"(bytes) : "memory"); }
__device__ __forceinline__ void mbar_arrive(uint64_t* b) { asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(b)) : "memory"); }
__device__ __forceinline__ bool mbar_wait(uint64_t* b, uint32_t parity, volatile int* abort_flag) {
  const long long t0 = clock64();
  while (true) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(ok) : "r"(smem_u32(b)), "r"(parity) : "memory");
    if (ok) return true;
    if (*abort_flag || clock64() - t0 > 2000000000LL) { *abort_flag = 1; return false; }
  }
}
__device__ __forceinline__ void tma2(void* dst, const CUtensorMap* m, uint64_t* bar, int x, int y) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
               ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(m)), "r"(smem_u32(bar)), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void tma3(void* dst, const CUtensorMap* m, uint64_t* bar, int x, int y, int z) {
  asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
               ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(m)), "r"(smem_u32(bar)), "r"(x), "r"(y), "r"(z) : "memory");
}
struct P {
  CUtensorMap a, b;
  int a_rows_box, b_rows_box;   // rows per box
  int katoms;                   // 64-column atoms per op (1: 2-D box; 2 or 4: 3-D box {64, katoms, rows})
  int a_ops, b_ops;             // ops per k-step for A and B (each op loads rows_box rows, consecutive row blocks)
  int k_steps;                  // steps over K
  int m_blocks, n_blocks;       // tile grid
  int stage_bytes, stages;
  int split;                   // 1: a second producer thread issues the B operations
  int priv;                    // 1: every CTA streams its own rows of A and B (no tile shared between CTAs)
  int* fail;
};
__global__ void __launch_bounds__(128, 1) tma_bw_kernel(const __grid_constant__ P p) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  __shared__ uint64_t full[8], empty[8];
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) { mbar_init(&full[s], p.split ? 2 : 1); mbar_init(&empty[s], 1); }
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const int tiles = p.m_blocks * p.n_blocks;
  const int a_bytes = p.a_rows_box * 128 * p.katoms, b_bytes = p.b_rows_box * 128 * p.katoms;
  if (threadIdx.x == 0 || (p.split && threadIdx.x == 64)) {
    const bool do_a = threadIdx.x == 0, do_b = p.split ? threadIdx.x == 64 : true;
    uint32_t it = 0;
    for (int t = blockIdx.x; t < tiles; t += gridDim.x) {
      const int per_panel = 8 * p.n_blocks, panel = t / per_panel, within = t - panel * per_panel;
      const int rows_here = min(8, p.m_blocks - panel * 8);
      int nb = within / rows_here, mb = panel * 8 + (within - nb * rows_here);
      if (p.priv) { mb = blockIdx.x % p.m_blocks; nb = blockIdx.x % p.n_blocks; }
      for (int k = 0; k < p.k_steps; ++k, ++it) {
        const int s = it % p.stages;
        if (!mbar_wait(&empty[s], ((it / p.stages) & 1u) ^ 1u, &abort_flag)) return;
        uint8_t* dst = smem + s * p.stage_bytes;
        if (do_a) mbar_expect(&full[s], (do_b ? p.a_ops * a_bytes + p.b_ops * b_bytes : p.a_ops * a_bytes));
        else mbar_expect(&full[s], p.b_ops * b_bytes);
        if (do_a) for (int o = 0; o < p.a_ops; ++o) {
          const int y = (mb * p.a_ops + o) * p.a_rows_box;
          if (p.katoms == 1) tma2(dst + o * a_bytes, &p.a, &full[s], k * 64, y); else tma3(dst + o * a_bytes, &p.a, &full[s], 0, y, k * p.katoms);
        }
        dst += p.a_ops * a_bytes;
        if (do_b) for (int o = 0; o < p.b_ops; ++o) {
          const int y = (nb * p.b_ops + o) * p.b_rows_box;
          if (p.katoms == 1) tma2(dst + o * b_bytes, &p.b, &full[s], k * 64, y); else tma3(dst + o * b_bytes, &p.b, &full[s], 0, y, k * p.katoms);
        }
      }
    }
  } else if (threadIdx.x == 32) {
    uint32_t it = 0;
    for (int t = blockIdx.x; t < tiles; t += gridDim.x)
      for (int k = 0; k < p.k_steps; ++k, ++it) {
        const int s = it % p.stages;
        if (!mbar_wait(&full[s], (it / p.stages) & 1u, &abort_flag)) { *p.fail = 1; return; }
        mbar_arrive(&empty[s]);
      }
  }
}
typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeFn get_fn() {
  void* fn = nullptr; cudaDriverEntryPointQueryResult q;
  CK(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q));
  return reinterpret_cast<EncodeFn>(fn);
}
static void make_map(CUtensorMap* m, void* base, long rows, long K, int rows_box, int katoms) {
  EncodeFn fn = get_fn();
  cuuint32_t es[3] = {1, 1, 1};
  CUresult r;
  if (katoms == 1) {
    cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows}; cuuint64_t str[1] = {(cuuint64_t)K * 2}; cuuint32_t box[2] = {64, (cuuint32_t)rows_box};
    r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, dims, str, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  } else {
    cuuint64_t dims[3] = {64, (cuuint64_t)rows, (cuuint64_t)(K / 64)}; cuuint64_t str[2] = {(cuuint64_t)K * 2, 128}; cuuint32_t box[3] = {64, (cuuint32_t)rows_box, (cuuint32_t)katoms};
    r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, base, dims, str, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  }
  if (r != CUDA_SUCCESS) { printf("encode failed %d\n", (int)r); exit(1); }
}
int main() {
  const long M = 18432, N = 4096, K = 1024;
  void *A, *B; int* fail;
  CK(cudaMalloc(&A, M * K * 2)); CK(cudaMalloc(&B, N * K * 2)); CK(cudaMalloc(&fail, 4));
  CK(cudaMemset(A, 0, M * K * 2)); CK(cudaMemset(B, 0, N * K * 2)); CK(cudaMemset(fail, 0, 4));
  struct V { const char* name; int a_rows, b_rows, katoms, a_ops, b_ops, tile_m, tile_n; int priv; int split; };
  const V vs[] = {
    {"shared  1 op  16 KB (A 128r x 64)", 128, 128, 1, 1, 0, 128, 128, 0},
    {"shared  1 op  32 KB (A 128r x 128 deep)", 128, 128, 2, 1, 0, 128, 128, 0},
    {"shared  1 op  64 KB (A 128r x 256 deep)", 128, 128, 4, 1, 0, 128, 128, 0},
    {"shared  2 ops 16 KB (A + B)", 128, 128, 1, 1, 1, 128, 128, 0},
    {"shared  2 ops 32 KB (A + B deep)", 128, 128, 2, 1, 1, 128, 128, 0},
    {"shared  4 ops 16 KB (2A + 2B)", 128, 128, 1, 2, 2, 256, 256, 0},
    {"shared  8 ops 4 KB (4A + 4B 32r)", 32, 32, 1, 4, 4, 128, 128, 0},
    {"private 1 op  16 KB", 128, 128, 1, 1, 0, 128, 128, 1},
    {"private 2 ops 16 KB", 128, 128, 1, 1, 1, 128, 128, 1},
    {"private 2 ops 32 KB deep", 128, 128, 2, 1, 1, 128, 128, 1},
    {"private 4 ops 16 KB", 128, 128, 1, 2, 2, 256, 256, 1},
    {"private 8 ops 4 KB", 32, 32, 1, 4, 4, 128, 128, 1},
    {"shared  2 ops 16 KB, two producer threads", 128, 128, 1, 1, 1, 128, 128, 0, 1},
    {"shared  2 ops 32 KB deep, two producer threads", 128, 128, 2, 1, 1, 128, 128, 0, 1},
    {"shared  4 ops 16 KB, two producer threads", 128, 128, 1, 2, 2, 256, 256, 0, 1},
  };

  for (const V& v : vs) {
    P p{};
    make_map(&p.a, A, M, K, v.a_rows, v.katoms); make_map(&p.b, B, N, K, v.b_rows, v.katoms);
    p.a_rows_box = v.a_rows; p.b_rows_box = v.b_rows; p.katoms = v.katoms; p.a_ops = v.a_ops; p.b_ops = v.b_ops;
    p.k_steps = K / (64 * v.katoms); p.m_blocks = M / v.tile_m; p.n_blocks = N / v.tile_n;
    p.stage_bytes = (v.a_ops * v.a_rows + v.b_ops * v.b_rows) * 128 * v.katoms;
    p.stages = 196608 / p.stage_bytes; if (p.stages > 8) p.stages = 8; if (p.stages < 1) { printf("%s: stage too large\n", v.name); continue; }
    p.fail = fail; p.priv = v.priv; p.split = v.split;
    const int smem = p.stages * p.stage_bytes + 1024;
    CK(cudaFuncSetAttribute(tma_bw_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    cudaEvent_t e0, e1; CK(cudaEventCreate(&e0)); CK(cudaEventCreate(&e1));
    tma_bw_kernel<<<148, 128, smem>>>(p); CK(cudaDeviceSynchronize());
    CK(cudaEventRecord(e0));
    for (int i = 0; i < 5; ++i) tma_bw_kernel<<<148, 128, smem>>>(p);
    CK(cudaEventRecord(e1)); CK(cudaDeviceSynchronize());
    float ms; CK(cudaEventElapsedTime(&ms, e0, e1)); ms /= 5;
    const double bytes = (double)p.m_blocks * p.n_blocks * p.k_steps * p.stage_bytes;
    int f; CK(cudaMemcpy(&f, fail, 4, cudaMemcpyDeviceToHost));
    printf("%-62s stages %d: %.1f us, %.2f TB/s into the SMs, %.0f ns per k-step and CTA%s\n", v.name, p.stages, ms * 1e3, bytes / ms / 1e9,
           ms * 1e6 / ((double)p.m_blocks * p.n_blocks / 148.0 * p.k_steps), f ? "  [WAIT EXPIRED]" : "");
  }
  return 0;
}
