// Block-diagonal (variable-length) softmax attention on tcgen05 tensor cores.
//
// One work unit = (item, head, 256 query rows) = two 128-row query tiles A and B that share every
// K/V tile.  Keys and values come from the same item only: the key loop stops at the item's last
// 128-key tile and the keys past the item's end are masked to -inf (probability exactly 0).
// An item with an odd number of query tiles (577 tokens = 4.5 tiles) would leave tile B empty in every
// head's last unit; for head_dim 64 those last tiles of two adjacent heads share a unit instead
// (dual-head unit: A on head h, B on head h + 1, each with its own K/V tiles).
//
//   warp 0       TMA producer: Q tiles (double buffered across units), K/V tiles through a ring
//   warp 1       UMMA issuer:  S = Q K^T (128 x keys x {64|80}) into TMEM, O += P V (128 x {64|80} x keys) in TMEM;
//                keys per K/V tile: 128 for head_dim 64, 112 for head_dim 80 (see AttnTcSmem); head_dim 80 has an
//                issuer thread per warpgroup (warp 1 for tile A, warp 2 for tile B)
//   warps 2, 3   idle (they complete the first warpgroup, whose registers are handed to the softmax warps)
//   warps 4..7   softmax warpgroup of tile A: one thread per query row
//   warps 8..11  softmax warpgroup of tile B
//
// A softmax thread reads its row of S from TMEM, keeps a running reference maximum m and sum l, and writes
// P = exp2((s - m) * scale) as bf16 back into tensor memory (columns of its own: the A operand of P V is read from
// there; the PT = false instantiation, kept as a cross-check, stages P in shared memory instead, K-major with
// 128-byte swizzle).  The reference maximum only moves when the row maximum grows by more than 2^8 in the exponent;
// then the thread rescales its O row in TMEM.  Final O / l is written as bf16.
// Persistent: gridDim.x = sm_budget CTAs; the units are dealt to them in rounds of gridDim.x, alternate rounds in
// opposite directions (the host sorts the units by decreasing cost: a fixed direction would hand CTA 0 the costliest
// unit of every round).
#pragma once
#include "ptx.cuh"

namespace eas {

constexpr int kTcThreads = 384;
constexpr int kTcTile = 128;            // query rows per tile and keys per K/V tile
constexpr float kRescaleThreshold = 8.0f;

struct AttnTcParams {
  CUtensorMap map_lo;   // qkv [T, 3d], box {64 columns, 128 rows}, 128-byte swizzle
  CUtensorMap map_hi;   // box {16 columns, 128 rows}, 32-byte swizzle (head_dim 80: columns 64..79)
  CUtensorMap map_klo;  // qkv, box {64 columns, keys per K/V tile}, 128-byte swizzle (K and V tiles)
  CUtensorMap map_khi;  // box {16 columns, keys per K/V tile}, 32-byte swizzle
  CUtensorMap map_out;  // out [T, d], box {64 columns, 32 rows}, 128-byte swizzle (store of a warp's 32 output rows)
  bf16* out;
  long long ldo;
  int d_model, n_heads;
  float scale_log2;     // log2(e) / sqrt(head_dim)
  int n_items, total_units;
  int item_start[128];
  int item_len[128];
  int unit_prefix[129];
  uint32_t* status;
};

// PT: the probabilities P live in tensor memory (the A operand of P V is read from there); otherwise they are
// staged in shared memory.  With PT the 64 KB of P staging become extra K/V stages.
#ifndef EAS_ATTN_KEYS_HD80
#define EAS_ATTN_KEYS_HD80 112     // keys per K/V tile for head_dim 80 with P in tensor memory (128: the former layout)
#endif
template <int HD, bool PT>
struct AttnTcSmem {
  static constexpr int HI = HD - 64;                       // 0 or 16 extra columns
  // Keys per K/V tile.  head_dim 80 with P in tensor memory takes 112: then S (2 x 112 columns), O (2 x 80) and
  // dedicated P columns (2 x 56) fit the 512 columns of tensor memory together (496), P no longer has to re-use S's
  // columns, and the next scores can be computed while P V of the current tile is still running, as for head_dim 64.
  // With 128 keys the three would need 544 columns.
  static constexpr int kKeys = (PT && HD != 64) ? EAS_ATTN_KEYS_HD80 : kTcTile;
  static constexpr bool kNarrowO = PT && HD != 64 && kKeys < kTcTile;   // O is HD columns wide, P has its own columns
  static constexpr int kLoBytes = kTcTile * 128;           // Q tile: 128 rows x 64 bf16
  static constexpr int kHiBytes = kTcTile * HI * 2;        // 128 rows x 16 bf16
  static constexpr int kTileBytes = kLoBytes + kHiBytes;   // one Q tile
  static constexpr int kKLoBytes = kKeys * 128;            // K or V tile: keys x 64 bf16
  static constexpr int kKHiBytes = kKeys * HI * 2;         // keys x 16 bf16
  static constexpr int kKHiPad = (kKHiBytes + 1023) / 1024 * 1024;   // the next tile starts on a swizzle-atom boundary
  static constexpr int kKTileBytes = kKLoBytes + kKHiPad;  // shared memory of one K tile
  static constexpr int kKTxBytes = kKLoBytes + kKHiBytes;  // bytes its loads deliver
  static constexpr bool kStagedOut = PT && HD == 64;       // output rows leave through shared memory and TMA stores
  // With P in tensor memory and head_dim 80, V is loaded 128 columns wide (two 64-column boxes; the extra 48 columns
  // belong to the next head, or are zero past the last one) so that P V is ONE UMMA per 16 keys (N = 80 across the
  // two swizzle atoms; N = 128 with 128-key tiles, whose surplus output columns are never read) instead of an N = 64
  // plus an N = 16 one: the issuer is the bottleneck there and every UMMA costs about the same.
  static constexpr bool kWideV = PT && HD != 64;
  static constexpr int kVBytes = kWideV ? 2 * kKLoBytes : kKTileBytes;
  static constexpr int kVTxBytes = kWideV ? 2 * kKLoBytes : kKTxBytes;
  static constexpr int kStageBytes = kKTileBytes + kVBytes;  // K then V
  static constexpr int kStages = PT ? (HD == 64 ? 4 : (kNarrowO ? 3 : 2)) : (HD == 64 ? 3 : 2);
  static constexpr int kQOff = 0;                          // [2 buffers][2 tiles]
  static constexpr int kKvOff = kQOff + 4 * kTileBytes;    // [stages][K, V]
  static constexpr int kPOff = kKvOff + kStages * kStageBytes;   // [2 tiles][2 k-blocks of 16 KB] (shared-memory P only)
  static constexpr int kOutOff = kPOff + (PT ? 0 : 2 * 32768);      // [8 softmax warps][32 rows x 128 bytes]
  static constexpr int kBarOff = kOutOff + (kStagedOut ? 8 * 4096 : 0);
  static constexpr int kBytes = kBarOff + 512 + 1024;      // barriers + alignment slack
  static_assert(kBytes <= 232448, "exceeds the shared memory of an SM");
  static_assert(kKeys % 16 == 0 && kKeys % 8 == 0 && kKeys <= kTcTile, "key tile: whole UMMA k-steps and swizzle-atom rows");
  static_assert(kStageBytes % 1024 == 0 && kTileBytes % 1024 == 0, "tiles start on swizzle-atom boundaries");
  // TMEM columns: S_A [0, keys) S_B [keys, 2 keys), then O_A, O_B, then (if P has columns of its own) P_A, P_B.
  // head_dim 64: 128 + 128 + 64 + 64 + 64 + 64 = 512.  head_dim 80 with 112 keys: 224 + 160 + 112 = 496.
  // head_dim 80 with 128 keys: S 256 + O 2 x 128 (wide) = 512, and P re-uses the first 64 columns of S (dead once
  // the row sits in registers), which obliges the issuer to run P V before the next S.
  // Dual-head units: an item whose query rows end in a single 128-row tile would leave warpgroup B idle for that
  // tile's whole key loop (c1: 577 tokens = 4.5 tiles, one unit in three).  With four K/V stages such tiles of TWO
  // adjacent heads form one unit instead: A works on head h, B on head h + 1, each with its own K/V tiles (two ring
  // stages per key tile).
  static constexpr bool kDualHeadOk = PT && HD == 64;   // the kernel's DUAL template argument may be set
  static constexpr int kSStride = kKeys;
  static constexpr int kOCol0 = 2 * kKeys, kOStride = HD == 64 ? 64 : (kNarrowO ? HD : 128);
  static constexpr bool kPAliasesS = PT && HD != 64 && !kNarrowO;
  static constexpr int kPCol0 = kPAliasesS ? 0 : kOCol0 + 2 * kOStride, kPStride = kPAliasesS ? kSStride : kKeys / 2;
  static_assert(kPAliasesS || !PT || kPCol0 + 2 * kPStride <= 512, "tensor memory columns");
  static_assert(kOCol0 + 2 * kOStride <= 512, "tensor memory columns");
};

__device__ __forceinline__ void tmem_st_32x32_from(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
        "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
        "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}

__device__ __forceinline__ void tmem_ld_32x16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st_32x16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

template <int OFF, int N>
__device__ __forceinline__ void tmem_ld_32x16_at(uint32_t taddr, uint32_t (&r)[N]) {
  static_assert(OFF + 16 <= N, "row buffer too short");
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[OFF + 0]), "=r"(r[OFF + 1]), "=r"(r[OFF + 2]), "=r"(r[OFF + 3]), "=r"(r[OFF + 4]), "=r"(r[OFF + 5]),
        "=r"(r[OFF + 6]), "=r"(r[OFF + 7]), "=r"(r[OFF + 8]), "=r"(r[OFF + 9]), "=r"(r[OFF + 10]), "=r"(r[OFF + 11]),
        "=r"(r[OFF + 12]), "=r"(r[OFF + 13]), "=r"(r[OFF + 14]), "=r"(r[OFF + 15])
      : "r"(taddr + OFF)
      : "memory");
}
__device__ __forceinline__ void tmem_st_32x16_from(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
__device__ __forceinline__ void tmem_st_32x8_from(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
      : "memory");
}
template <int OFF, int N>
__device__ __forceinline__ void tmem_ld_32x32_at(uint32_t taddr, uint32_t (&r)[N]) {
  static_assert(OFF + 32 <= N, "row buffer too short");
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[OFF + 0]), "=r"(r[OFF + 1]), "=r"(r[OFF + 2]), "=r"(r[OFF + 3]), "=r"(r[OFF + 4]), "=r"(r[OFF + 5]),
        "=r"(r[OFF + 6]), "=r"(r[OFF + 7]), "=r"(r[OFF + 8]), "=r"(r[OFF + 9]), "=r"(r[OFF + 10]), "=r"(r[OFF + 11]),
        "=r"(r[OFF + 12]), "=r"(r[OFF + 13]), "=r"(r[OFF + 14]), "=r"(r[OFF + 15]), "=r"(r[OFF + 16]), "=r"(r[OFF + 17]),
        "=r"(r[OFF + 18]), "=r"(r[OFF + 19]), "=r"(r[OFF + 20]), "=r"(r[OFF + 21]), "=r"(r[OFF + 22]), "=r"(r[OFF + 23]),
        "=r"(r[OFF + 24]), "=r"(r[OFF + 25]), "=r"(r[OFF + 26]), "=r"(r[OFF + 27]), "=r"(r[OFF + 28]), "=r"(r[OFF + 29]),
        "=r"(r[OFF + 30]), "=r"(r[OFF + 31])
      : "r"(taddr + OFF)
      : "memory");
}
// 2^x for a pair of arguments on the FMA pipe instead of the special-function unit: x = n + f with n = rint(x)
// (magic-number rounding), 2^f by a cubic fitted on [-0.5, 0.5] (relative error below 8e-5, far under the bf16
// rounding of P), then n is added to the exponent field.  Arguments are clamped at -126 (result ~1e-38 instead of 0).
#ifndef EAS_ATTN_MAX_CHAINS
#define EAS_ATTN_MAX_CHAINS 4      // independent chains of the row-maximum reduction (a power of two)
#endif
#ifndef EAS_ATTN_POLY_OF_4
#define EAS_ATTN_POLY_OF_4 1      // of every 4 pairs of probabilities, this many take the polynomial path
#endif
__device__ __forceinline__ void exp2_poly_pair(uint64_t x2, float& p0, float& p1) {
  float x0, x1;
  unpack2(x2, x0, x1);
  x2 = pack2(fmaxf(x0, -126.0f), fmaxf(x1, -126.0f));
  const uint64_t magic = pack2(12582912.0f, 12582912.0f);            // 1.5 * 2^23
  const uint64_t nmagic = pack2(-12582912.0f, -12582912.0f);
  const uint64_t t2 = fadd2(x2, magic);                              // low mantissa bits hold rint(x)
  const uint64_t n2 = fadd2(t2, nmagic);
  const uint64_t f2 = ffma2(n2, pack2(-1.0f, -1.0f), x2);            // f = x - n in [-0.5, 0.5]
  uint64_t r2 = ffma2(pack2(0.05508868f, 0.05508868f), f2, pack2(0.24260405f, 0.24260405f));
  r2 = ffma2(r2, f2, pack2(0.69327623f, 0.69327623f));
  r2 = ffma2(r2, f2, pack2(0.99992895f, 0.99992895f));
  float r0, r1, t0, t1;
  unpack2(r2, r0, r1);
  unpack2(t2, t0, t1);
  p0 = __uint_as_float(__float_as_uint(r0) + (__float_as_uint(t0) << 23));
  p1 = __uint_as_float(__float_as_uint(r1) + (__float_as_uint(t1) << 23));
}
__device__ __forceinline__ float fmax3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
// Register re-balancing between warpgroups.  The pool is the CTA's launch allocation (168 x 384 registers): the
// sum over warpgroups of 128 x their limit must stay BELOW it, or setmaxnreg.inc waits forever.
constexpr int kRegsLight = 112, kRegsSoftmax = 192;
static_assert(128 * kRegsLight + 256 * kRegsSoftmax < 168 * 384, "setmaxnreg budget exceeds the CTA's register allocation");
template <int N>
__device__ __forceinline__ void setmaxnreg_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N>
__device__ __forceinline__ void setmaxnreg_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }

#ifdef EAS_ATTN_PROFILE
// phase timestamps of the first softmax warp of each warpgroup in CTA 0 (profiling builds only)
__device__ unsigned long long g_attn_dbg[2 * 64 * 12];
#define ATTN_STAMP(k) do { if (blockIdx.x == 0 && quarter == 0 && lane == 0 && n < 64) g_attn_dbg[(w * 64 + n) * 12 + (k)] = clock64(); } while (0)
#define ATTN_STAMP_PREV(k) do { if (blockIdx.x == 0 && quarter == 0 && lane == 0 && n >= 1 && n <= 64) g_attn_dbg[(w * 64 + n - 1) * 12 + (k)] = clock64(); } while (0)
#else
#define ATTN_STAMP(k) do { } while (0)
#define ATTN_STAMP_PREV(k) do { } while (0)
#endif

struct UnitInfo {
  int head, q0, S, n_kv, n_q;
  int dual;             // 1: tile A belongs to `head`, tile B to `head + 1`, same query rows, separate K/V tiles
  long long row0;
};
// `cursor` is the caller's item index of its previous unit: units are visited in increasing order, so the item is
// found by stepping forward (usually zero or one step) instead of searching.
// Unit order inside an item (the host's attention_schedule counts the same way).  Without dual-head units:
// (head, pair of query tiles), the pair index fastest, the last pair possibly a single tile.  With them: first the
// (head, FULL pair) units, then one unit per two heads for the odd last query tile.
template <bool DUAL, int KEYS>
__device__ __forceinline__ UnitInfo decode_unit(const AttnTcParams& p, int unit, int& cursor) {
  static_assert(!DUAL || KEYS == kTcTile, "dual-head units count query tiles as key tiles");
  int lo = cursor;
  while (lo + 1 < p.n_items && p.unit_prefix[lo + 1] <= unit) ++lo;
  cursor = lo;
  UnitInfo u;
  u.S = p.item_len[lo];
  u.row0 = p.item_start[lo];
  u.n_kv = (u.S + KEYS - 1) / KEYS;
  const int r = unit - p.unit_prefix[lo];
  if (DUAL) {
    const int full = u.n_kv >> 1;                  // query tiles == key tiles
    const int n_full = p.n_heads * full;
    if (r < n_full) {
      u.head = r / full;
      u.q0 = (r - u.head * full) * 2 * kTcTile;
      u.n_q = 2;
      u.dual = 0;
    } else {
      u.head = 2 * (r - n_full);
      u.q0 = full * 2 * kTcTile;
      u.dual = u.head + 1 < p.n_heads ? 1 : 0;
      u.n_q = 1 + u.dual;
    }
    return u;
  }
  const int pairs = (u.S + 2 * kTcTile - 1) / (2 * kTcTile);
  u.head = r / pairs;
  u.q0 = (r - u.head * pairs) * 2 * kTcTile;       // pair index varies fastest: neighbours share K and V in L2
  u.n_q = (u.q0 + kTcTile < u.S) ? 2 : 1;
  u.dual = 0;
  return u;
}

// DUAL: the launch's unit order contains dual-head units (the host sets it only when some item has an odd number of
// query tiles; without it every `dual` test below folds away).
template <int HD, bool PT, bool DUAL = false>
__global__ void __launch_bounds__(kTcThreads, 1) attn_tc_kernel(const __grid_constant__ AttnTcParams p) {
  using L = AttnTcSmem<HD, PT>;
  static_assert(!DUAL || L::kDualHeadOk, "dual-head units need four K/V stages and dedicated P columns");
  constexpr int HI = L::HI;
  constexpr int NST = L::kStages;
  // head_dim 80: the single issuer thread (12 UMMAs per tile and warpgroup, about 90 cycles each) is what the softmax
  // warpgroups wait for, so each warpgroup gets an issuer thread of its own (warps 1 and 2).  Not for head_dim 64: there
  // the fixed order of one issuer keeps the two warpgroups' exponential phases apart, which is worth more.
  constexpr bool kTwoIssuers = PT && HD != 64 && !L::kPAliasesS;
  static_assert(!kTwoIssuers || (!DUAL && !L::kPAliasesS), "the two-issuer path has no dual-head units and needs dedicated P columns");
  extern __shared__ uint8_t smem_raw_attn[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw_attn) + 1023) & ~uintptr_t(1023));
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::kBarOff);
  uint64_t* q_full = bars;                 // [2]
  uint64_t* q_empty = bars + 2;            // [2]
  uint64_t* k_full = bars + 4;             // [NST]
  uint64_t* v_full = bars + 4 + NST;       // [NST]
  uint64_t* kv_empty = bars + 4 + 2 * NST; // [NST]
  uint64_t* s_full = bars + 4 + 3 * NST;   // [2]
  uint64_t* p_ready = s_full + 2;          // [2]
  uint64_t* pv_done = s_full + 4;          // [2]
  uint64_t* s_free = s_full + 6;           // [2] two-issuer kernels: the warpgroup has read its scores out of tensor memory
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(s_full + 8);
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    // with one issuer thread per warpgroup both threads hand every K/V stage and Q buffer back
    for (int i = 0; i < 2; ++i) {
      mbar_init(&q_full[i], 1); mbar_init(&q_empty[i], kTwoIssuers ? 2 : 1);
      mbar_init(&s_full[i], 1); mbar_init(&p_ready[i], 4); mbar_init(&pv_done[i], 1); mbar_init(&s_free[i], 4);
    }
    for (int i = 0; i < NST; ++i) { mbar_init(&k_full[i], 1); mbar_init(&v_full[i], 1); mbar_init(&kv_empty[i], kTwoIssuers ? 2 : 1); }
    *abort_flag = 0;
    mbar_fence_init();
    tma_prefetch_desc(&p.map_lo);
    if (HI) tma_prefetch_desc(&p.map_hi);
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, 512);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;
  pdl_launch_dependents();
  pdl_wait();

  // this CTA's unit of a round; increasing in `round`
  auto unit_at = [&](uint32_t round) -> int {
    const int g = static_cast<int>(gridDim.x), b = static_cast<int>(blockIdx.x);
    return static_cast<int>(round) * g + ((round & 1u) ? g - 1 - b : b);
  };
  auto q_tile = [&](int buf, int t) { return smem + L::kQOff + (buf * 2 + t) * L::kTileBytes; };
  auto k_tile = [&](int s) { return smem + L::kKvOff + s * L::kStageBytes; };
  auto v_tile = [&](int s) { return smem + L::kKvOff + s * L::kStageBytes + L::kKTileBytes; };
  auto p_tile = [&](int w) { return smem + L::kPOff + w * 32768; };

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    setmaxnreg_dec<kRegsLight>();
    if (lane == 0) {
      uint32_t kv_it = 0, u_cnt = 0;
      bool ok = true;
      int cursor = 0;
      for (int unit = unit_at(0); unit < p.total_units && ok; unit = unit_at(++u_cnt)) {
        const UnitInfo u = decode_unit<DUAL, L::kKeys>(p, unit, cursor);
        const int qb = u_cnt & 1;
        if (!mbar_wait(&q_empty[qb], ((u_cnt >> 1) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
        mbar_expect_tx(&q_full[qb], u.n_q * L::kTileBytes);
        for (int t = 0; t < u.n_q; ++t) {
          const int xq = (u.head + (u.dual ? t : 0)) * HD;
          const int y = static_cast<int>(u.row0) + u.q0 + (u.dual ? 0 : t * kTcTile);
          tma_load_2d(q_tile(qb, t), &p.map_lo, &q_full[qb], xq, y);
          if (HI) tma_load_2d(q_tile(qb, t) + L::kLoBytes, &p.map_hi, &q_full[qb], xq + 64, y);
        }
        const int kv_tiles = u.n_kv * (1 + u.dual);      // dual-head units: key tile j of head h, then of head h + 1
        for (int jj = 0; jj < kv_tiles; ++jj, ++kv_it) {
          const int j = u.dual ? (jj >> 1) : jj;
          const int xq = (u.head + (u.dual ? (jj & 1) : 0)) * HD;
          const int s = kv_it % NST;
          if (!mbar_wait(&kv_empty[s], ((kv_it / NST) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
          const int y = static_cast<int>(u.row0) + j * L::kKeys;
          mbar_expect_tx(&k_full[s], L::kKTxBytes);
          tma_load_2d(k_tile(s), &p.map_klo, &k_full[s], p.d_model + xq, y);
          if (HI) tma_load_2d(k_tile(s) + L::kKLoBytes, &p.map_khi, &k_full[s], p.d_model + xq + 64, y);
          mbar_expect_tx(&v_full[s], L::kVTxBytes);
          tma_load_2d(v_tile(s), &p.map_klo, &v_full[s], 2 * p.d_model + xq, y);
          if (L::kWideV) tma_load_2d(v_tile(s) + L::kKLoBytes, &p.map_klo, &v_full[s], 2 * p.d_model + xq + 64, y);
          else if (HI) tma_load_2d(v_tile(s) + L::kKLoBytes, &p.map_khi, &v_full[s], 2 * p.d_model + xq + 64, y);
        }
      }
      if (!ok) {
        const long long t0 = clock64();
        while (clock64() - t0 < 4000000) {}     // let loads in flight land before the CTA retires
      }
    }
  } else if (warp == 1 || (kTwoIssuers && warp == 2)) {
    // ------------------------------------------------------------------ UMMA issuer(s)
    setmaxnreg_dec<kRegsLight>();
    if (lane == 0) {
      constexpr uint32_t idesc_s = make_idesc_bf16(128, L::kKeys, 0, 0);     // S = Q K^T, both K-major
      constexpr uint32_t idesc_o_lo = make_idesc_bf16(128, 64, 0, 1);   // O[:, 0:64] += P V, V is MN-major
      constexpr uint32_t idesc_o_hi = make_idesc_bf16(128, 16, 0, 1);   // O[:, 64:80]
      constexpr uint32_t idesc_o_wide = make_idesc_bf16(128, L::kNarrowO ? HD : 128, 0, 1); // O from the 128-column V tile
      uint32_t kv_it = 0, u_cnt = 0;
      uint32_t n_tiles[2] = {0, 0};            // S tiles issued per warpgroup (phase counters)
      uint32_t n_pv[2] = {0, 0};
      bool ok = true;

      auto issue_s = [&](int w, int qb, int s) {
        const uint32_t qa = smem_u32(q_tile(qb, w));
        const uint32_t ka = smem_u32(k_tile(s));
        const uint64_t ad = make_smem_desc(qa, 16, 1024, kSwizzle128B);
        const uint64_t bd = make_smem_desc(ka, 16, 1024, kSwizzle128B);
        const uint32_t d = tmem_base + w * L::kSStride;
#pragma unroll
        for (int k = 0; k < 4; ++k) umma_bf16_ss(d, ad + 2 * k, bd + 2 * k, idesc_s, k != 0);
        if (HI) {
          const uint64_t ah = make_smem_desc(qa + L::kLoBytes, 16, 256, kSwizzle32B);
          const uint64_t bh = make_smem_desc(ka + L::kKLoBytes, 16, 256, kSwizzle32B);
          umma_bf16_ss(d, ah, bh, idesc_s, 1);
        }
        umma_commit(&s_full[w]);
        ++n_tiles[w];
      };
      auto issue_pv = [&](int w, int s, bool accumulate) {
        const uint32_t va = smem_u32(v_tile(s));
        const uint32_t d = tmem_base + L::kOCol0 + w * L::kOStride;
#pragma unroll
        for (int ks = 0; ks < L::kKeys / 16; ++ks) {       // 16 keys per step
          const uint64_t bd = make_smem_desc(va + ks * 2048, 1024, 1024, kSwizzle128B);
          const uint32_t acc = (accumulate || ks != 0) ? 1u : 0u;
          if (L::kWideV) {
            // two 64-column swizzle atoms 16 KB apart (leading byte offset), 8-key groups 1 KB apart
            const uint32_t pt = tmem_base + L::kPCol0 + w * L::kPStride + ks * 8;
            const uint64_t bw = make_smem_desc(va + ks * 2048, L::kKLoBytes, 1024, kSwizzle128B);
            umma_bf16_ts(d, pt, bw, idesc_o_wide, acc);
          } else if (PT) {
            const uint32_t pt = tmem_base + L::kPCol0 + w * L::kPStride + ks * 8;   // 16 bf16 = 8 columns
            umma_bf16_ts(d, pt, bd, idesc_o_lo, acc);
            if (HI) {
              const uint64_t bh = make_smem_desc(va + L::kKLoBytes + ks * 512, 256, 256, kSwizzle32B);
              umma_bf16_ts(d + 64, pt, bh, idesc_o_hi, acc);
            }
          } else {
            const uint32_t pa = smem_u32(p_tile(w));
            const uint64_t ad = make_smem_desc(pa + (ks >> 2) * 16384 + (ks & 3) * 32, 16, 1024, kSwizzle128B);
            umma_bf16_ss(d, ad, bd, idesc_o_lo, acc);
            if (HI) {
              const uint64_t bh = make_smem_desc(va + L::kKLoBytes + ks * 512, 256, 256, kSwizzle32B);
              umma_bf16_ss(d + 64, ad, bh, idesc_o_hi, acc);
            }
          }
        }
        umma_commit(&pv_done[w]);
        ++n_pv[w];
      };

      if constexpr (kTwoIssuers) {
        // One issuer thread per warpgroup (w = warp - 1), so every wait is in that warpgroup's own deterministic order:
        //   S(next tile)  as soon as the warpgroup has read its previous scores out of tensor memory (s_free): the
        //                 next scores are computed while the warpgroup works on the exponentials;
        //   PV(tile)      when the warpgroup has stored P (p_ready).
        // The thread walks EVERY tile of every unit of the CTA in order, also those of units its warpgroup has no part
        // in: it waits until such a tile (or Q buffer) has landed and hands it back with a plain arrival, so that both
        // issuers see every phase of every barrier and a parity can never be mistaken for an earlier phase.
        const int w = warp - 1;
        struct Pos {                                 // a tile position in the CTA's sequence, with its unit's facts
          int unit, j, n_kv, hint;
          uint32_t ucnt, g;                          // units before it (Q buffer), tiles before it (ring stage)
          bool active, end;
        };
        auto enter_unit = [&](Pos& c) {              // c.unit / c.ucnt / c.g are set; fills the unit's facts
          if (c.unit >= p.total_units) { c.end = true; return; }
          const UnitInfo u = decode_unit<DUAL, L::kKeys>(p, c.unit, c.hint);
          c.n_kv = u.n_kv;
          c.active = w < u.n_q;
          c.j = 0;
        };
        auto next_tile = [&](Pos& c) {
          ++c.j; ++c.g;
          if (c.j >= c.n_kv) { ++c.ucnt; c.unit = unit_at(c.ucnt); enter_unit(c); }
        };
        Pos pc;                                      // in-order position: every tile is visited
        pc.unit = unit_at(0); pc.ucnt = 0; pc.g = 0; pc.hint = 0; pc.end = false;
        enter_unit(pc);
        bool s_issued = false;                       // S of the own tile at pc is already in flight
        uint32_t q_seen = 0;                         // units before this one have had their Q seen landing by this thread
        while (!pc.end && ok) {
          const int qb = pc.ucnt & 1;
          if (pc.j == 0) {                           // entering a unit: see its Q land; hand it back at once if unused
            if (pc.ucnt >= q_seen) {                 // (a look-ahead S may have seen it already, and handed it back)
              if (!mbar_wait(&q_full[qb], (pc.ucnt >> 1) & 1u, abort_flag)) { ok = false; break; }
              q_seen = pc.ucnt + 1;
            }
            if (!pc.active) mbar_arrive(&q_empty[qb]);
          }
          const int s = pc.g % NST;
          const uint32_t ph = (pc.g / NST) & 1u;
          if (!pc.active) {
            if (!mbar_wait(&k_full[s], ph, abort_flag) || !mbar_wait(&v_full[s], ph, abort_flag)) { ok = false; break; }
            mbar_arrive(&kv_empty[s]);
            next_tile(pc);
            continue;
          }
          if (!s_issued) {                           // first own tile, or the look-ahead below was not possible
            if (!mbar_wait(&k_full[s], ph, abort_flag)) { ok = false; break; }
            tc_fence_after_sync();
            issue_s(w, qb, s);
            if (pc.j + 1 >= pc.n_kv) umma_commit(&q_empty[qb]);
          }
          s_issued = false;
          // the next own tile, if it is close enough that its barriers' previous phases have been seen by this thread
          // (strictly inside the ring: the stage of tile pc.g + NST is the one this thread still holds)
          Pos nx = pc;
          next_tile(nx);
          while (!nx.end && !nx.active && nx.g - pc.g + 1 < static_cast<uint32_t>(NST) && nx.ucnt <= pc.ucnt + 1) next_tile(nx);
          const bool ahead = !nx.end && nx.active && nx.g - pc.g < static_cast<uint32_t>(NST) && nx.ucnt <= pc.ucnt + 1;
          if (ahead) {
            if (!mbar_wait(&s_free[w], (n_tiles[w] - 1) & 1u, abort_flag)) { ok = false; break; }
            const int nqb = nx.ucnt & 1;
            if (nx.ucnt >= q_seen) {
              if (!mbar_wait(&q_full[nqb], (nx.ucnt >> 1) & 1u, abort_flag)) { ok = false; break; }
              q_seen = nx.ucnt + 1;
            }
            const int sn = nx.g % NST;
            if (!mbar_wait(&k_full[sn], (nx.g / NST) & 1u, abort_flag)) { ok = false; break; }
            tc_fence_after_sync();
            issue_s(w, nqb, sn);
            if (nx.j + 1 >= nx.n_kv) umma_commit(&q_empty[nqb]);
            s_issued = true;
          }
          if (!mbar_wait(&p_ready[w], n_pv[w] & 1u, abort_flag)) { ok = false; break; }
          if (!mbar_wait(&v_full[s], ph, abort_flag)) { ok = false; break; }
          tc_fence_after_sync();
          issue_pv(w, s, pc.j != 0);
          umma_commit(&kv_empty[s]);                 // arrives when everything this thread has issued so far is complete
          next_tile(pc);
        }
      } else {
        bool pre_issued[2] = {false, false};       // S(w, 0) of this unit was already issued at the end of the previous one
        int cursor = 0;
        UnitInfo un = decode_unit<DUAL, L::kKeys>(p, min(static_cast<int>(blockIdx.x), p.total_units - 1), cursor);
        for (int unit = unit_at(0); unit < p.total_units && ok; unit = unit_at(++u_cnt)) {
          const UnitInfo u = un;
          const int qb = u_cnt & 1;
          const bool has_next = unit_at(u_cnt + 1) < p.total_units;
          if (has_next) un = decode_unit<DUAL, L::kKeys>(p, unit_at(u_cnt + 1), cursor);
          if (!mbar_wait(&q_full[qb], (u_cnt >> 1) & 1u, abort_flag)) { ok = false; break; }
          // K/V tile of warpgroup w at ring position kv_it: shared by both warpgroups, or (dual-head unit) one each
          const uint32_t step = 1 + u.dual;
#pragma unroll
          for (int w = 0; w < 2; ++w) {
            if (w < u.n_q && !pre_issued[w]) {
              const uint32_t g = kv_it + (u.dual ? w : 0);
              if (!mbar_wait(&k_full[g % NST], (g / NST) & 1u, abort_flag)) { ok = false; break; }
              tc_fence_after_sync();
              issue_s(w, qb, g % NST);
            }
          }
          if (!ok) break;
          pre_issued[0] = pre_issued[1] = false;
          bool next_q_ready = false;
          const int n_kv = u.n_kv, n_q = u.n_q, next_n_q = un.n_q;
          const uint32_t b_off = u.dual ? 1u : 0u, b_off_next = un.dual ? 1u : 0u;   // B's tile relative to A's
          for (int j = 0; j < n_kv && ok; ++j, kv_it += step) {
            const bool last = j + 1 == n_kv;
#pragma unroll
            for (int w = 0; w < 2; ++w) {
              if (w >= n_q) break;
              const uint32_t g = kv_it + (w ? b_off : 0u);                                          // this tile
              const uint32_t gn = kv_it + step + (w ? (last ? b_off_next : b_off) : 0u);            // the warpgroup's next one
              const int s = g % NST, sn = gn % NST;
              // warpgroup B shares A's tiles unless the unit is dual-head: A has already seen them land
              const bool own_tile = w == 0 || (b_off | (last ? b_off_next : 0u)) != 0u;
              // P(w, j) is in shared memory, S(w) has been read, O(w) has been rescaled if it had to be
              if (!mbar_wait(&p_ready[w], (n_pv[w]) & 1u, abort_flag)) { ok = false; break; }
              tc_fence_after_sync();
              // next scores first (the softmax of the next tile overlaps P V of this one); after the unit's last
              // tile the next scores are the first tile of the NEXT unit, so the pipeline never drains
              // next scores before P V, so that the next softmax overlaps it -- unless P re-uses S's columns
              if (!last && !L::kPAliasesS) {
                if (own_tile && !mbar_wait(&k_full[sn], (gn / NST) & 1u, abort_flag)) { ok = false; break; }
                tc_fence_after_sync();
                issue_s(w, qb, sn);
              }
              if (own_tile && !mbar_wait(&v_full[s], (g / NST) & 1u, abort_flag)) { ok = false; break; }
              tc_fence_after_sync();
              issue_pv(w, s, j != 0);
              if (!last && L::kPAliasesS) {
                if (own_tile && !mbar_wait(&k_full[sn], (gn / NST) & 1u, abort_flag)) { ok = false; break; }
                tc_fence_after_sync();
                issue_s(w, qb, sn);
              }
              if (last && has_next && w < next_n_q) {
                // the unit's output is waiting for this P V, so it went first; now the first scores of the next unit
                if (!next_q_ready) {
                  if (!mbar_wait(&q_full[qb ^ 1], ((u_cnt + 1) >> 1) & 1u, abort_flag)) { ok = false; break; }
                  next_q_ready = true;
                }
                if (own_tile && !mbar_wait(&k_full[sn], (gn / NST) & 1u, abort_flag)) { ok = false; break; }
                tc_fence_after_sync();
                issue_s(w, qb ^ 1, sn);
                pre_issued[w] = true;
              }
              // K and V of this tile are free once everything issued so far completes: after the last warpgroup that
              // uses them
              if (b_off != 0u || w + 1 == n_q) umma_commit(&kv_empty[s]);
            }
          }
          if (ok) umma_commit(&q_empty[qb]);
        }
      }
    }
  } else if (warp < 4) {
    setmaxnreg_dec<kRegsLight>();
  } else {
    // ------------------------------------------------------------------ softmax warpgroups
    setmaxnreg_inc<kRegsSoftmax>();
    const int w = (warp - 4) >> 2;                 // 0: tile A, 1: tile B
    const int quarter = warp & 3;                  // TMEM lane quarter of this warp
    const int row = quarter * 32 + lane;           // query row inside the tile == TMEM lane
    const uint32_t lane_addr = static_cast<uint32_t>(quarter * 32) << 16;
    const uint32_t s_addr = tmem_base + lane_addr + w * L::kSStride;
    const uint32_t o_addr = tmem_base + lane_addr + L::kOCol0 + w * L::kOStride;
    const uint32_t p_addr = tmem_base + lane_addr + L::kPCol0 + w * L::kPStride;
    uint8_t* p_row = p_tile(w) + row * 128;
    const int sw = row & 7;
    uint32_t n = 0;                                // tiles processed by this warpgroup
    bool ok = true;

    // The output of a unit is written while the NEXT unit's first tile is in flight: by then its last P V has
    // long finished, so the warpgroup never waits for it.
    bool pend = false;
    int pend_q0 = 0, pend_head = 0, pend_S = 0;
    long long pend_row0 = 0;
    float pend_l = 1.f;
    uint32_t pend_n = 0;
    uint8_t* out_stage = smem + L::kOutOff + (warp - 4) * 4096;
    auto flush_output = [&]() -> bool {
      if (!mbar_wait(&pv_done[w], pend_n & 1u, abort_flag)) return false;
      tc_fence_after_sync();
      ATTN_STAMP_PREV(7);
      const float inv = 1.0f / pend_l;
      const int warp_row0 = pend_q0 + quarter * 32;                    // first query row of this warp within the item
      const int qrow = warp_row0 + lane;
      uint32_t o[HD / 16][16];
      __syncwarp();
#pragma unroll
      for (int c = 0; c < HD / 16; ++c) tmem_ld_32x16(o_addr + c * 16, o[c]);
      tmem_ld_wait();
      ATTN_STAMP_PREV(8);
      uint32_t pkd[HD / 2];
#pragma unroll
      for (int c = 0; c < HD / 16; ++c)
#pragma unroll
        for (int i = 0; i < 8; ++i)
          pkd[c * 8 + i] = pack_bf16x2(__uint_as_float(o[c][2 * i]) * inv, __uint_as_float(o[c][2 * i + 1]) * inv);
      if (L::kStagedOut && warp_row0 + 32 <= pend_S) {
        // all 32 rows of this warp belong to the item: swizzled staging, one TMA store
        if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        __syncwarp();
        uint8_t* srow = out_stage + lane * 128;
#pragma unroll
        for (int q = 0; q < 8; ++q)
          *reinterpret_cast<uint4*>(srow + ((q ^ (lane & 7)) << 4)) = make_uint4(pkd[4 * q], pkd[4 * q + 1], pkd[4 * q + 2], pkd[4 * q + 3]);
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                       ::"l"(reinterpret_cast<uint64_t>(&p.map_out)), "r"(smem_u32(out_stage)), "r"(pend_head * HD),
                         "r"(static_cast<int>(pend_row0) + warp_row0) : "memory");
          asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        }
      } else if (qrow < pend_S) {
        // the warp straddles the item's end (or this head size has no staged path): per-row stores
        uint4* dst = reinterpret_cast<uint4*>(p.out + (pend_row0 + qrow) * p.ldo + pend_head * HD);
#pragma unroll
        for (int q = 0; q < HD / 8; ++q) dst[q] = make_uint4(pkd[4 * q], pkd[4 * q + 1], pkd[4 * q + 2], pkd[4 * q + 3]);
      }
      ATTN_STAMP_PREV(9);
      // the O reads above are complete before this warpgroup's next p_ready lets P V overwrite O
      tc_fence_before_sync();
      pend = false;
      return true;
    };

    int cursor = 0;
    UnitInfo u_next = decode_unit<DUAL, L::kKeys>(p, min(static_cast<int>(blockIdx.x), p.total_units - 1), cursor);
    uint32_t round = 0;
    for (int unit = unit_at(0); unit < p.total_units && ok; unit = unit_at(++round)) {
      const UnitInfo u = u_next;
      ATTN_STAMP_PREV(10);
      const bool has_next = unit_at(round + 1) < p.total_units;
      if (w >= u.n_q) {                             // this warpgroup has no tile in the unit
        if (has_next) u_next = decode_unit<DUAL, L::kKeys>(p, unit_at(round + 1), cursor);
        if (pend && !flush_output()) { ok = false; break; }
        continue;
      }
      float m_used = -INFINITY, l = 0.f;
      for (int j = 0; j < u.n_kv; ++j, ++n) {
        ATTN_STAMP(0);
        // The previous unit's output goes out here: its last P V was issued before this unit's first scores,
        // so it is complete while those are still being computed, and the write hides behind that wait.
        if (j == 0 && pend && !flush_output()) { ok = false; break; }
        if (!mbar_wait(&s_full[w], n & 1u, abort_flag)) { ok = false; break; }
        tc_fence_after_sync();
        ATTN_STAMP(1);
        constexpr int KEYS = L::kKeys;
        const int valid = min(KEYS, u.S - j * KEYS);           // keys of this tile that belong to the item
        // the whole score row (one fp32 per key) in registers: a few loads, one wait
        uint32_t sr[KEYS];
        __syncwarp();
        tmem_ld_32x32_at<0>(s_addr, sr);
        tmem_ld_32x32_at<32>(s_addr, sr);
        tmem_ld_32x32_at<64>(s_addr, sr);
        if constexpr (KEYS == 128) tmem_ld_32x32_at<96>(s_addr, sr); else tmem_ld_32x16_at<96>(s_addr, sr);
        static_assert(KEYS == 128 || KEYS == 112, "score row: 4 x 32 columns, or 3 x 32 + 16");
        tmem_ld_wait();
        if constexpr (kTwoIssuers) {      // the scores are in registers: the issuer may start the next S into these columns
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(&s_free[w]);
        }
        ATTN_STAMP(2);
        if (valid < KEYS) {                                     // last tile of the item: keys past its end
#pragma unroll
          for (int i = 0; i < KEYS; ++i) if (i >= valid) sr[i] = 0xff800000u;   // -inf
        }
        // row maximum: EAS_ATTN_MAX_CHAINS independent chains of 3-input maxima (a chain is a string of dependent
        // instructions: more, shorter chains hide their latency behind each other), folded at the end
        float mxc[EAS_ATTN_MAX_CHAINS];
#pragma unroll
        for (int c = 0; c < EAS_ATTN_MAX_CHAINS; ++c) mxc[c] = -INFINITY;
#pragma unroll
        for (int i = 0; i < KEYS; i += 2)
          mxc[(i / 2) % EAS_ATTN_MAX_CHAINS] = fmax3(mxc[(i / 2) % EAS_ATTN_MAX_CHAINS], __uint_as_float(sr[i]), __uint_as_float(sr[i + 1]));
#pragma unroll
        for (int w2 = EAS_ATTN_MAX_CHAINS / 2; w2 >= 1; w2 >>= 1)
#pragma unroll
          for (int c = 0; c < w2; ++c) mxc[c] = fmaxf(mxc[c], mxc[c + w2]);
        const float mx = mxc[0];
        ATTN_STAMP(3);
        // reference maximum: moves only when the row maximum grew by more than the threshold
        float corr = 1.0f;
        bool rescale = false;
        if (j == 0) {
          m_used = mx;
        } else if ((mx - m_used) * p.scale_log2 > kRescaleThreshold) {
          corr = fast_ex2((m_used - mx) * p.scale_log2);
          m_used = mx;
          rescale = true;
        }
        l *= corr;
        const float mb = m_used * p.scale_log2;
        const uint64_t scale2 = pack2(p.scale_log2, p.scale_log2);
        const uint64_t nmb2 = pack2(-mb, -mb);
        // probabilities, kept packed in registers until the P buffer is free
        uint32_t pk[KEYS / 2];
        uint64_t acc0 = 0, acc1 = 0, acc2 = 0, acc3 = 0;       // (0.f, 0.f) pairs
#pragma unroll
        for (int i = 0; i < KEYS / 2; i += 4) {
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const uint64_t t = ffma2(pack2(__uint_as_float(sr[2 * (i + q)]), __uint_as_float(sr[2 * (i + q) + 1])), scale2, nmb2);
            float p0, p1;
            if (q < EAS_ATTN_POLY_OF_4) {
              exp2_poly_pair(t, p0, p1);
            } else {
              float t0, t1;
              unpack2(t, t0, t1);
              p0 = fast_ex2(t0);
              p1 = fast_ex2(t1);
            }
            const uint64_t pp = pack2(p0, p1);
            if (q == 0) acc0 = fadd2(acc0, pp);
            if (q == 1) acc1 = fadd2(acc1, pp);
            if (q == 2) acc2 = fadd2(acc2, pp);
            if (q == 3) acc3 = fadd2(acc3, pp);
            pk[i + q] = pack_bf16x2(p0, p1);
          }
        }
        {
          const uint64_t a = fadd2(fadd2(acc0, acc1), fadd2(acc2, acc3));
          float a0, a1;
          unpack2(a, a0, a1);
          l += a0 + a1;
        }
        // S has been read: the issuer may overwrite it with the next tile's scores once p_ready fires.
        // The previous P V must be complete before P is overwritten or O is touched.
        ATTN_STAMP(4);
        if (n > 0 && !mbar_wait(&pv_done[w], (n - 1) & 1u, abort_flag)) { ok = false; break; }
        ATTN_STAMP(5);
        tc_fence_after_sync();
        if (__any_sync(0xffffffffu, rescale)) {
#pragma unroll 1
          for (int c = 0; c < HD / 16; ++c) {
            uint32_t o[16];
            __syncwarp();
            tmem_ld_32x16(o_addr + c * 16, o);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 16; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * corr);
            tmem_st_32x16(o_addr + c * 16, o);
          }
          tmem_st_wait();
        }
        if constexpr (PT) {
          // P row into tensor memory: two bf16 per column of this thread's lane
          __syncwarp();
          tmem_st_32x32_from(p_addr, pk);
          if constexpr (KEYS == 128) {
            tmem_st_32x32_from(p_addr + 32, pk + 32);
          } else {
            tmem_st_32x16_from(p_addr + 32, pk + 32);
            tmem_st_32x8_from(p_addr + 48, pk + 48);
          }
          tmem_st_wait();
        } else {
          // P row: 2 k-blocks of 64 keys, each row 128 bytes, 16-byte chunks XOR-swizzled by (row & 7)
#pragma unroll
          for (int cc = 0; cc < 16; ++cc) {
            const int kblk = cc >> 3, ch = cc & 7;
            uint4 v = make_uint4(pk[cc * 4], pk[cc * 4 + 1], pk[cc * 4 + 2], pk[cc * 4 + 3]);
            *reinterpret_cast<uint4*>(p_row + kblk * 16384 + ((ch ^ sw) << 4)) = v;
          }
          fence_proxy_async_smem();
        }
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive(&p_ready[w]);
        ATTN_STAMP(6);
        // decode the following unit here: the warp now waits for the issuer anyway
        if (j == 0 && has_next) u_next = decode_unit<DUAL, L::kKeys>(p, unit_at(round + 1), cursor);
      }
      if (!ok) break;
      pend = true;                                  // written later, see flush_output
      // this warpgroup's tile: the second 128 rows of the same head, or (dual-head unit) the same rows of the next head
      pend_q0 = u.q0 + (u.dual ? 0 : w * kTcTile); pend_head = u.head + (u.dual ? w : 0);
      pend_S = u.S; pend_row0 = u.row0; pend_l = l; pend_n = n - 1;
    }
    if (ok && pend) flush_output();
    if (L::kStagedOut && lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
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
