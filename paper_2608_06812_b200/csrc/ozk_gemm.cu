// Limb GEMM on the FP4 tensor cores (tcgen05.mma kind::mxf4, block-scaled E2M1, FP32 accumulators
// in tensor memory), with the recombination of the limb products in the epilogue.
//
//   DGEMM path   Section 5.1: ab = a0 b0 + 13 (a0 b1 + a1 b0) + 13^2 a1 b1 (mod m); Section 6.4: all
//                moduli in one launch, three accumulators per modulus, only residues reach memory;
//                Lemma 3: every FP32 partial sum is an exact integer.
//   INT8 path    Section 3 / Eq. 1 with p = q = 3: nine limb products in five groups i + j = g,
//                C = sum_g 13^g G_g as int32.
//
// One persistent CTA per SM walks a static list of work items (plane group l, tile of 128 columns
// of C, tile of W rows of C).  The tensor-core row side (TMEM lanes) holds the B-matrix limbs p_i
// (plane rows = columns j of C) and the column side the A-matrix limbs q_j (plane rows = rows i of
// C), so an epilogue thread owns one j and consecutive i: the column-major order of C.
//
// The limb tiles q_0 .. q_{NQ-1} of a stage are adjacent in shared memory, so ONE instruction per
// row-side limb does all its products:  D[W*i .. W*i + NQ*W) += p_i * [q_0 ; ... ; q_{NQ-1}].
// Group g = i + j therefore accumulates in TMEM columns [W*g, W*g + W): the cross terms that share
// a power of 13 land in the same accumulator (NP + NQ - 1 accumulators for NP * NQ products).
//
// Warp roles: 0 = TMA producer, 1 = MMA issuer (owns the TMEM allocation), 2.. = epilogue.
// Every wait is bounded; on expiry the CTA records OZK_ERR_DEVICE_TIMEOUT, drains and returns.
#include <stdio.h>
#include <stdlib.h>

#include <atomic>

#include "ozk_common.cuh"
#include "ozk_ptx.cuh"

namespace ozk {
namespace {

using namespace ptx;

constexpr int kPTileBytes = kTileRows * kTileKBytes;  // 16 KiB: 128 rows x 128 bytes
constexpr int kTmemCols = 512;
constexpr int kScaleCol = 496;  // scale-factor bytes live in TMEM columns 496..511
constexpr uint64_t kWaitLimitNs = 2000000000ull;
constexpr int kMaxStages = 4;

struct GemmCore {
  int L;        // plane groups (moduli); plane index = limbs * l + limb
  int tiles_p;  // tiles of 128 along the columns of C (B-matrix plane rows)
  int tiles_q;  // tiles of W along the rows of C (A-matrix plane rows)
  int kblocks;  // Kp / 256
  int group;    // rasterisation: this many column tiles share one sweep over the row tiles
  int skip_top_first;  // plane group 0 needs no p_{NP-1} q_{NQ-1} product (13^2 = 0 mod 169)
  int q_groups;        // 0: both operands use plane group l; n > 0: row side uses l / n, column side l % n
  unsigned int* wave_counter;  // optional: producers of all CTAs meet here before every wave of items
  int fast_combine;    // K <= 17476: D1 + 13 D2 stays below 2^24 and may be formed in FP32 before the release
  int count_cycles;    // measurement aid: the issuing thread of pair 0 records where its clocks went (status block)
  int karatsuba;       // CTA-pair kernel: moduli with karatsuba_modulus(l) run three products with sum-limb planes
  int sum_plane_base;  // plane index of the first sum-limb plane (2 L)
  StatusBlock* status;
  uint32_t scale_word;  // four copies of the UE8M0 scale byte
};

struct __align__(8) GemmShared {
  uint64_t full[kMaxStages];
  uint64_t empty[kMaxStages];
  uint64_t tmem_full;
  uint64_t tmem_empty;
  uint64_t drained;
  uint32_t tmem_base;
  volatile int abort;
};

// Bounded wait on an mbarrier phase.  Returns false after the time limit or when another role
// of this CTA has already given up.
__device__ __forceinline__ bool wait_bounded(uint32_t bar, uint32_t parity, volatile int* abort, StatusBlock* status, int where) {
  if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = global_timer_ns();
  for (uint32_t it = 1;; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 63u) == 0u) {
      if (*abort) return false;
      if (global_timer_ns() - t0 > kWaitLimitNs) {
        *abort = 1;
        atomicMin(&status->code, (int)OZK_ERR_DEVICE_TIMEOUT);
        atomicExch(&status->where, where);
        return false;
      }
    }
  }
}


// Producer-side wave barrier: before loading the operands of its n-th item a producer announces
// itself on a global counter and waits (bounded) until every producer that has an n-th item has
// done so.  It keeps the CTAs of a wave within one tile of each other, so that tiles requested by
// several CTAs are still in L2 when the last of them asks.  Needs all CTAs resident (persistent
// grid, cooperative launch).  Returns false on expiry.
__device__ __forceinline__ bool wave_barrier(unsigned int* counter, unsigned int target, volatile int* abort, StatusBlock* status) {
  atomicAdd(counter, 1u);
  const uint64_t t0 = global_timer_ns();
  for (uint32_t it = 0;; ++it) {
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(counter) : "memory");
    if (v >= target) return true;
    __nanosleep(64);
    if ((it & 63u) == 63u) {
      if (*abort) return false;
      if (global_timer_ns() - t0 > kWaitLimitNs) {
        *abort = 1;
        atomicMin(&status->code, (int)OZK_ERR_DEVICE_TIMEOUT);
        atomicExch(&status->where, 0x700);
        return false;
      }
    }
  }
}

// The same counter used for pacing only, in the two-accumulator kernel whose tiles are short: a producer announces each
// item and goes on as soon as the counter has reached `target`, which the caller sets to the arrivals of the wave before
// the previous one.  `seen` is the newest value this producer knows; wave_counter_probe() reads the counter without
// waiting for the answer (it is looked at one item later), so that in step no producer ever polls.
__device__ __forceinline__ unsigned int wave_counter_probe(const unsigned int* counter) {
  unsigned int v;
  asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(counter) : "memory");
  return v;
}
__device__ __forceinline__ bool wave_barrier_lagged(unsigned int* counter, unsigned int target, unsigned int& seen, volatile int* abort,
                                                    StatusBlock* status) {
  atomicAdd(counter, 1u);
  if (seen >= target) return true;
  const uint64_t t0 = global_timer_ns();
  for (uint32_t it = 0;; ++it) {
    seen = wave_counter_probe(counter);
    if (seen >= target) return true;
    __nanosleep(64);
    if ((it & 63u) == 63u) {
      if (*abort) return false;
      if (global_timer_ns() - t0 > kWaitLimitNs) {
        *abort = 1;
        atomicMin(&status->code, (int)OZK_ERR_DEVICE_TIMEOUT);
        atomicExch(&status->where, 0x701);
        return false;
      }
    }
  }
}

__device__ __forceinline__ void decode_item(const GemmCore& p, int item, int& l, int& tp, int& tq) {
  const int per_group = p.tiles_p * p.tiles_q;
  l = item / per_group;
  const int t = item - l * per_group;
  const int band = p.group * p.tiles_q;
  const int g = t / band;
  const int rem = t - g * band;
  const int gsize = min(p.group, p.tiles_p - g * p.group);
  tq = rem / gsize;
  tp = g * p.group + (rem - tq * gsize);
}

// Walks the items item, item + step, ... of one CTA pair in the order of decode_item without a division per item.
struct ItemCursor {
  int l, g, rem;           // modulus, band of column tiles, position inside the band (tq * gsize + column tile of the band)
  int gsize, band_items;   // column tiles and items of this band
  uint32_t inv_gsize;      // ceil(2^32 / gsize): rem / gsize by one multiply-high (rem < 2^29)
  __device__ __forceinline__ void set_band(const GemmCore& p) {
    gsize = min(p.group, p.tiles_p - g * p.group);
    band_items = gsize * p.tiles_q;
    inv_gsize = gsize > 1 ? 0xFFFFFFFFu / (uint32_t)gsize + 1u : 0u;
  }
  __device__ __forceinline__ void init(const GemmCore& p, int item) {
    const int per_group = p.tiles_p * p.tiles_q;
    l = item / per_group;
    const int t = item - l * per_group;
    const int band = p.group * p.tiles_q;
    g = t / band;
    rem = t - g * band;
    set_band(p);
  }
  __device__ __forceinline__ void advance(const GemmCore& p, int step) {
    rem += step;
    while (rem >= band_items) {
      rem -= band_items;
      if (++g * p.group >= p.tiles_p) g = 0, ++l;
      set_band(p);
    }
  }
  __device__ __forceinline__ void tile(const GemmCore& p, int& tp, int& tq) const {
    tq = gsize > 1 ? (int)__umulhi((uint32_t)rem, inv_gsize) : rem;
    tp = g * p.group + (rem - tq * gsize);
  }
};


// Drains the three accumulators of 64 columns (lanes of this warp's quadrant) and hands tensor memory
// back as early as possible.  With `fast` the only work before the release is one exact FP32
// multiply-add per element, u = D1 + 13 D2 (|u| <= 128 K + 13 * 64 K < 2^24 for K <= 17476); the
// conversions, the rest of the weighted sum and the reduction mod m run after the release and
// overlap the next tile's main loop.  Returns t = D0 + 13 D1 + 169 D2 + offset (non-negative).
// mode: 0 = modulus 169 (no 13^2 accumulator), 1 = the regular three accumulators [D0 | D1 | D2],
//       2 = Karatsuba accumulators [a0 b0 | (a0 + a1)(b0 + b1) | a1 b1]: t = D0 + 13 (Ds - D0 - D2) + 169 D2
//           = D0 + 13 (Ds - D0 + 12 D2), the inner sum below 976 K < 2^24 for K <= 17152.
template <bool kFast, bool kZeroTop, bool kKara = false>
__device__ __forceinline__ void drain_and_release(uint32_t base, int W, int mode, uint32_t offset, uint32_t release_bar,
                                                  bool release_remote, int lane, uint32_t (&t)[64]) {
  const bool top = mode != 0;
  uint32_t u[kFast ? 64 : 1];
  if constexpr (kFast && !kKara) {
    // 16 columns of each accumulator at a time; the loads of the next chunk are in flight while this chunk's
    // multiply-adds run (a wait covers every load issued before it, so it sits between the two)
    uint32_t d1[2][16], d2[2][16];
    auto issue = [&](int c) {
      tmem_ld_32x16(base + 1 * W + c * 16, d1[c & 1]);
      if (top) tmem_ld_32x16(base + 2 * W + c * 16, d2[c & 1]);
      tmem_ld_32x16(base + 0 * W + c * 16, *reinterpret_cast<uint32_t(*)[16]>(&t[c * 16]));  // raw FP32 bits until after the release
    };
    issue(0);
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      tmem_wait_ld();
      if (c < 3) issue(c + 1);
#pragma unroll
      for (int e = 0; e < 16; ++e)
        u[c * 16 + e] = top ? __float_as_uint(fmaf(__uint_as_float(d2[c & 1][e]), 13.0f, __uint_as_float(d1[c & 1][e]))) : d1[c & 1][e];
    }
  } else
#pragma unroll
  for (int c = 0; c < 2; ++c) {
    uint32_t d1[32], d2[32];
    tmem_ld_32x32(base + 1 * W + c * 32, d1);
    if (top) tmem_ld_32x32(base + 2 * W + c * 32, d2);
    if constexpr (kFast) {
      // D0 goes straight into t (raw FP32 bits until after the release): one wait covers all three loads
      tmem_ld_32x32(base + 0 * W + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&t[c * 32]));
      tmem_wait_ld();
      if (kKara && mode == 2) {
#pragma unroll
        for (int e = 0; e < 32; ++e)
          u[c * 32 + e] = __float_as_uint(fmaf(__uint_as_float(d2[e]), 12.0f, __uint_as_float(d1[e]) - __uint_as_float(t[c * 32 + e])));
      } else {
#pragma unroll
        for (int e = 0; e < 32; ++e)
          u[c * 32 + e] = top ? __float_as_uint(fmaf(__uint_as_float(d2[e]), 13.0f, __uint_as_float(d1[e]))) : d1[e];
      }
    } else {
      uint32_t d0[32];
      tmem_ld_32x32(base + 0 * W + c * 32, d0);
      tmem_wait_ld();
#pragma unroll
      for (int e = 0; e < 32; ++e) {
        const int a0 = __float2int_rn(__uint_as_float(d0[e]));
        const int a1 = __float2int_rn(__uint_as_float(d1[e]));
        const int a2 = top ? __float2int_rn(__uint_as_float(d2[e])) : 0;
        const int cross = (kKara && mode == 2) ? a1 - a0 - a2 : a1;
        t[c * 32 + e] = (uint32_t)(a0 + 13 * cross + 169 * a2) + offset;  // non-negative, < 2^32
      }
    }
  }
  if constexpr (kZeroTop) {
    tmem_st_32x32_const(base + 2 * W, 0u);
    tmem_st_32x32_const(base + 2 * W + 32, 0u);
    tmem_wait_st();
  }
  tc_fence_before();
  __syncwarp();
  if (lane == 0) {
    if (release_remote) mbar_arrive_cluster(release_bar); else mbar_arrive(release_bar);
  }
  if constexpr (kFast) {
#pragma unroll
    for (int e = 0; e < 64; ++e)
      t[e] = (uint32_t)(__float2int_rn(__uint_as_float(t[e])) + 13 * __float2int_rn(__uint_as_float(u[e]))) + offset;
  }
}

// Reduces 64 composed values mod m (one multiply-high each, result in [0, m)) and stores them as bytes.
__device__ __forceinline__ void reduce_and_store(const uint32_t (&t)[64], uint32_t m, uint32_t recip, uint4* dst) {
#pragma unroll
  for (int q4 = 0; q4 < 4; ++q4) {
    uint32_t w[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      uint32_t word = 0;
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        const uint32_t x = t[q4 * 16 + k * 4 + b];
        uint32_t r = x - __umulhi(x, recip) * m;  // in [0, 2m)
        r = min(r, r - m);
        word |= r << (8 * b);
      }
      w[k] = word;
    }
    dst[q4] = make_uint4(w[0], w[1], w[2], w[3]);
  }
}

// ------------------------------------------------------------------------------------
// Epilogue of the DGEMM path: r = (D0 + 13 D1 + 169 D2) mod m in [0, m), one byte per element.
// 8 warps: warp (quadrant q, half h) drains lanes 32q..32q+31, columns 64h..64h+63 of the three
// accumulators into 64 registers, releases tensor memory, then reduces and stores.
// ------------------------------------------------------------------------------------
struct ResidueParams {
    int m[kMaxModuli];
    uint32_t recip[kMaxModuli];   // floor(2^32 / m)
    uint32_t offset[kMaxModuli];  // multiple of m close to 2^31: makes the composed value non-negative
    uint8_t* res;                 // [L][Np][Mp] bytes
    int64_t res_ld;               // Mp
    size_t res_stride;            // Mp * Np
};
template <bool kFast>
struct ResidueEpilogue {
  static constexpr int kWarps = 8;
  using Params = ResidueParams;
  template <int W>
  __device__ static __forceinline__ void run(const Params& ep, const GemmCore& core, uint32_t tmem, int epi_warp, int lane, int l,
                                             int tp, int tq, uint32_t release_bar) {
    static_assert(W == 128, "residue epilogue is written for 128-wide tiles");
    // a warp can only touch the TMEM lanes of its own quadrant, (warp index in the CTA) mod 4
    const uint32_t quad = (uint32_t)((epi_warp + 2) & 3), half = (uint32_t)(epi_warp >> 2);
    const uint32_t base = tmem + ((quad * 32u) << 16) + half * 64u;
    const uint32_t m = (uint32_t)ep.m[l], recip = ep.recip[l], offset = ep.offset[l];
    const bool top = !(core.skip_top_first && l == 0);
    uint32_t t[64];
    drain_and_release<kFast, false>(base, W, top ? 1 : 0, offset, release_bar, false, lane, t);
    const int64_t j = (int64_t)tp * kTileRows + quad * 32 + lane;
    uint4* dst = reinterpret_cast<uint4*>(ep.res + (size_t)l * ep.res_stride + (size_t)j * (size_t)ep.res_ld +
                                          (size_t)tq * W + half * 64);
    reduce_and_store(t, m, recip, dst);
  }
};

// ------------------------------------------------------------------------------------
// Epilogue of the INT8 path: C = G0 + 13 G1 + 169 G2 + 2197 G3 + 28561 G4 as int32, written
// straight into the caller's column-major C.  4 warps, 16 columns at a time.
// ------------------------------------------------------------------------------------
struct Int32Epilogue {
  static constexpr int kWarps = 4;
  struct Params {
    int32_t* C;
    int64_t ldc, M, N;
  };
  template <int W>
  __device__ static __forceinline__ void run(const Params& ep, const GemmCore&, uint32_t tmem, int epi_warp, int lane, int,
                                             int tp, int tq, uint32_t release_bar) {
    const uint32_t quad = (uint32_t)((epi_warp + 2) & 3);  // TMEM lane quadrant = warp index mod 4
    const uint32_t base = tmem + ((quad * 32u) << 16);
    const int64_t j = (int64_t)tp * kTileRows + quad * 32 + lane;
    const int64_t i0 = (int64_t)tq * W;
    int32_t* col = ep.C + j * ep.ldc;
    const bool vec_ok = ((reinterpret_cast<uintptr_t>(ep.C) & 15) == 0) && ((ep.ldc & 3) == 0);
#pragma unroll 1
    for (int c = 0; c < W / 16; ++c) {
      uint32_t g0[16], g1[16], g2[16], g3[16], g4[16];
      tmem_ld_32x16(base + 0 * W + c * 16, g0);
      tmem_ld_32x16(base + 1 * W + c * 16, g1);
      tmem_ld_32x16(base + 2 * W + c * 16, g2);
      tmem_ld_32x16(base + 3 * W + c * 16, g3);
      tmem_ld_32x16(base + 4 * W + c * 16, g4);
      tmem_wait_ld();
      int32_t v[16];
#pragma unroll
      for (int e = 0; e < 16; ++e) {
        v[e] = __float2int_rn(__uint_as_float(g0[e])) + 13 * __float2int_rn(__uint_as_float(g1[e])) +
               169 * __float2int_rn(__uint_as_float(g2[e])) + 2197 * __float2int_rn(__uint_as_float(g3[e])) +
               28561 * __float2int_rn(__uint_as_float(g4[e]));
      }
      const int64_t i = i0 + c * 16;
      if (j < ep.N) {
        if (vec_ok && i + 16 <= ep.M) {
          int4* d = reinterpret_cast<int4*>(col + i);
#pragma unroll
          for (int k = 0; k < 4; ++k) d[k] = make_int4(v[4 * k], v[4 * k + 1], v[4 * k + 2], v[4 * k + 3]);
        } else {
#pragma unroll
          for (int e = 0; e < 16; ++e)
            if (i + e < ep.M) col[i + e] = v[e];
        }
      }
    }
    tc_fence_before();
    __syncwarp();
    if (lane == 0) mbar_arrive(release_bar);
  }
};


// ------------------------------------------------------------------------------------
// Epilogue of the scheme-I passes (Eq. 1): one pass multiplies NP = 4 row-side limbs with NQ = 3
// column-side limbs; its six accumulators G_0..G_5 (anti-diagonals of the 4 x 3 block) are combined
// as V = sum_g 13^g G_g in int64 (|G_g| <= 3 * 64 * K, 13^5 < 2^19) and stored per pass; a separate
// reduction kernel adds the passes with their powers of 13.  4 warps, 16 columns at a time.
// ------------------------------------------------------------------------------------
struct Int64BlockEpilogue {
  static constexpr int kWarps = 4;
  struct Params {
    long long* out;      // [passes][Np][ld] int64
    int64_t ld;          // rows per column of a pass (multiple of the tile width)
    size_t pass_stride;  // Np * ld
  };
  template <int W>
  __device__ static __forceinline__ void run(const Params& ep, const GemmCore&, uint32_t tmem, int epi_warp, int lane, int l,
                                             int tp, int tq, uint32_t release_bar) {
    const uint32_t quad = (uint32_t)((epi_warp + 2) & 3);  // TMEM lane quadrant = warp index mod 4
    const uint32_t base = tmem + ((quad * 32u) << 16);
    const int64_t j = (int64_t)tp * kTileRows + quad * 32 + lane;
    long long* col = ep.out + (size_t)l * ep.pass_stride + (size_t)j * (size_t)ep.ld + (size_t)tq * W;
#pragma unroll 1
    for (int c = 0; c < W / 16; ++c) {
      uint32_t g0[16], g1[16], g2[16], g3[16], g4[16], g5[16];
      tmem_ld_32x16(base + 0 * W + c * 16, g0);
      tmem_ld_32x16(base + 1 * W + c * 16, g1);
      tmem_ld_32x16(base + 2 * W + c * 16, g2);
      tmem_ld_32x16(base + 3 * W + c * 16, g3);
      tmem_ld_32x16(base + 4 * W + c * 16, g4);
      tmem_ld_32x16(base + 5 * W + c * 16, g5);
      tmem_wait_ld();
      longlong2* dst = reinterpret_cast<longlong2*>(col + c * 16);
#pragma unroll
      for (int e = 0; e < 16; e += 2) {
        long long v[2];
#pragma unroll
        for (int o = 0; o < 2; ++o) {
          const long long a0 = __float2int_rn(__uint_as_float(g0[e + o])), a1 = __float2int_rn(__uint_as_float(g1[e + o]));
          const long long a2 = __float2int_rn(__uint_as_float(g2[e + o])), a3 = __float2int_rn(__uint_as_float(g3[e + o]));
          const long long a4 = __float2int_rn(__uint_as_float(g4[e + o])), a5 = __float2int_rn(__uint_as_float(g5[e + o]));
          v[o] = a0 + 13ll * a1 + 169ll * a2 + 2197ll * a3 + 28561ll * a4 + 371293ll * a5;
        }
        dst[e / 2] = make_longlong2(v[0], v[1]);
      }
    }
    tc_fence_before();
    __syncwarp();
    if (lane == 0) mbar_arrive(release_bar);
  }
};

template <int NP, int NQ, int W, int STAGES, class Epi>
__global__ void __launch_bounds__(64 + 32 * Epi::kWarps, 1)
limb_gemm_kernel(const __grid_constant__ CUtensorMap map_p, const __grid_constant__ CUtensorMap map_q,
                 const __grid_constant__ GemmCore p, const __grid_constant__ typename Epi::Params ep) {
  constexpr int kQTileBytes = W * kTileKBytes;
  constexpr int kStageBytes = NP * kPTileBytes + NQ * kQTileBytes;
  constexpr int NG = NP + NQ - 1;
  static_assert(NG * W <= kScaleCol, "accumulators must leave room for the scale-factor columns");
  static_assert(NQ * W <= 256 && W % 16 == 0 && STAGES <= kMaxStages, "instruction shape limits");
  extern __shared__ uint8_t smem_raw[];
  // operand stages need 1024-byte alignment (128-byte swizzle atoms)
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  GemmShared* sh = reinterpret_cast<GemmShared*>(tiles + STAGES * kStageBytes);
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int total_items = p.L * p.tiles_p * p.tiles_q;

  if (threadIdx.x == 0) {
    prefetch_tensormap(&map_p);
    prefetch_tensormap(&map_q);
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(smem_u32(&sh->full[s]), 1);
      mbar_init(smem_u32(&sh->empty[s]), 1);
    }
    mbar_init(smem_u32(&sh->tmem_full), 1);
    mbar_init(smem_u32(&sh->tmem_empty), Epi::kWarps);
    mbar_init(smem_u32(&sh->drained), 1);
    sh->abort = 0;
    fence_barrier_init();
    fence_proxy_async();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&sh->tmem_base), kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sh->tmem_base;
  if (warp >= 2 && warp < 6) {  // constant UE8M0 scale bytes, identical for every row, column and K block
    const uint32_t quad = (uint32_t)(warp & 3);
    tmem_st_32x8_const(tmem + ((quad * 32u) << 16) + kScaleCol, p.scale_word);
    tmem_st_32x8_const(tmem + ((quad * 32u) << 16) + kScaleCol + 8, p.scale_word);
    tmem_wait_st();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      uint32_t armed_parity[STAGES];
      bool armed[STAGES];
      for (int s = 0; s < STAGES; ++s) armed[s] = false, armed_parity[s] = 0;
      bool ok = true;
      for (int item = blockIdx.x; item < total_items && ok; item += gridDim.x) {
        int l, tp, tq;
        decode_item(p, item, l, tp, tq);
        const int lp = p.q_groups ? l / p.q_groups : l, lq = p.q_groups ? l % p.q_groups : l;
        if (p.wave_counter) {
          const long long wave = item / (int)gridDim.x;
          const long long target = min((wave + 1) * (long long)gridDim.x, (long long)total_items);
          if (!wave_barrier(p.wave_counter, (unsigned int)target, &sh->abort, p.status)) break;
        }
        for (int kb = 0; kb < p.kblocks; ++kb) {
          if (!wait_bounded(smem_u32(&sh->empty[stage]), phase ^ 1u, &sh->abort, p.status, 0x000 + stage)) {
            ok = false;
            break;
          }
          const uint32_t bar = smem_u32(&sh->full[stage]);
          const uint32_t dst = smem_u32(tiles + stage * kStageBytes);
          mbar_arrive_expect_tx(bar, kStageBytes);
          armed[stage] = true;
          armed_parity[stage] = phase;
          const int x = kb * kTileKBytes;
#pragma unroll
          for (int i = 0; i < NP; ++i) tma_load_3d(dst + i * kPTileBytes, &map_p, bar, x, tp * kTileRows, NP * lp + i);
#pragma unroll
          for (int jq = 0; jq < NQ; ++jq)
            tma_load_3d(dst + NP * kPTileBytes + jq * kQTileBytes, &map_q, bar, x, tq * W, NQ * lq + jq);
          if (++stage == STAGES) stage = 0, phase ^= 1u;
        }
      }
      if (sh->abort) {  // let copies already in flight land before the CTA leaves
        for (int s = 0; s < STAGES; ++s)
          if (armed[s]) {
            const uint64_t t0 = global_timer_ns();
            while (!mbar_try_wait(smem_u32(&sh->full[s]), armed_parity[s]) && global_timer_ns() - t0 < kWaitLimitNs) {
            }
          }
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer --------------------------------
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0, acc_phase = 0;
      const uint32_t sf = tmem + kScaleCol;
      constexpr uint32_t kIdescOne = idesc_mxf4(W);
      constexpr uint32_t kIdescAll = idesc_mxf4(NQ * W);
      constexpr uint32_t kIdescButLast = idesc_mxf4(NQ > 1 ? (NQ - 1) * W : W);
      bool ok = true;
      for (int item = blockIdx.x; item < total_items && ok; item += gridDim.x) {
        int l, tp, tq;
        decode_item(p, item, l, tp, tq);
        const bool skip_top = p.skip_top_first && l == 0;
        if (!wait_bounded(smem_u32(&sh->tmem_empty), acc_phase ^ 1u, &sh->abort, p.status, 0x100)) break;
        tc_fence_after();
        for (int kb = 0; kb < p.kblocks; ++kb) {
          if (!wait_bounded(smem_u32(&sh->full[stage]), phase, &sh->abort, p.status, 0x110 + stage)) {
            ok = false;
            break;
          }
          tc_fence_after();
          const uint32_t pbase = smem_u32(tiles + stage * kStageBytes);
          const uint32_t qbase = pbase + NP * kPTileBytes;
#pragma unroll
          for (int ks = 0; ks < 4; ++ks) {
            if (kb == 0 && ks == 0) {
              // first step of a tile: overwrite instead of accumulate, group by group
              bool touched[NG];
#pragma unroll
              for (int g = 0; g < NG; ++g) touched[g] = false;
#pragma unroll
              for (int i = 0; i < NP; ++i) {
#pragma unroll
                for (int jq = 0; jq < NQ; ++jq) {
                  if (skip_top && i == NP - 1 && jq == NQ - 1) continue;
                  mma_mxf4(tmem + W * (i + jq), smem_desc_sw128(pbase + i * kPTileBytes),
                           smem_desc_sw128(qbase + jq * kQTileBytes), kIdescOne, sf, sf, touched[i + jq] ? 1u : 0u);
                  touched[i + jq] = true;
                }
              }
            } else {
#pragma unroll
              for (int i = 0; i < NP; ++i) {
                const bool shorten = skip_top && i == NP - 1;
                mma_mxf4(tmem + W * i, smem_desc_sw128(pbase + i * kPTileBytes + ks * 32), smem_desc_sw128(qbase + ks * 32),
                         shorten ? kIdescButLast : kIdescAll, sf, sf, 1u);
              }
            }
          }
          mma_commit(smem_u32(&sh->empty[stage]));
          if (++stage == STAGES) stage = 0, phase ^= 1u;
        }
        if (!ok) break;
        mma_commit(smem_u32(&sh->tmem_full));
        acc_phase ^= 1u;
      }
      if (sh->abort) {  // wait for the tensor pipe to go idle before TMEM is released
        mma_commit(smem_u32(&sh->drained));
        const uint64_t t0 = global_timer_ns();
        while (!mbar_try_wait(smem_u32(&sh->drained), 0u) && global_timer_ns() - t0 < kWaitLimitNs) {
        }
      }
    }
  } else {
    // ------------------------------ epilogue ----------------------------------
    uint32_t acc_phase = 0;
    for (int item = blockIdx.x; item < total_items; item += gridDim.x) {
      int l, tp, tq;
      decode_item(p, item, l, tp, tq);
      // the outcome must be warp-uniform: the TMEM loads below are warp-collective
      if (!__all_sync(0xFFFFFFFFu, wait_bounded(smem_u32(&sh->tmem_full), acc_phase, &sh->abort, p.status, 0x200 + warp))) break;
      tc_fence_after();
      Epi::template run<W>(ep, p, tmem, warp - 2, lane, l, tp, tq, smem_u32(&sh->tmem_empty));
      acc_phase ^= 1u;
    }
  }

  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 1) {
    __syncwarp();
    tmem_dealloc(tmem, kTmemCols);
  }
}


// ------------------------------------------------------------------------------------
// DGEMM path on CTA pairs (cta_group::2).  Two CTAs of a cluster (one TPC) work on a 256 x 128
// output tile: each holds 128 of the 256 TMEM lanes (columns j of C) and loads its own p0, p1 tiles;
// the 256 stacked column-side rows [q0 ; q1] are split between them, the leader keeps q0 and its
// peer q1, and the tensor core reads both halves.  Per stage a CTA therefore loads 48 KiB instead
// of 64 KiB and its shared memory feeds 64 instead of 96 bytes per clock to the MMA.
// The leader's MMA thread issues for the pair; byte counts of both CTAs' TMA loads arrive on the
// leader's "full" barrier; commits are multicast to the barriers of both CTAs.
// The first K step runs p0 with "overwrite" and p1 with "accumulate" (the cross-term columns
// 128..255 need both); the columns 256..383 of the 13^2 term are first overwritten with zeros by
// one extra instruction whose column-side operand is an all-zero tile in shared memory.
// For m = 169 (13^2 = 0) the p1 q1 product is not needed: those items run three 256 x 128 x 64
// instructions per K step instead, with each CTA supplying half the rows of q0 and of q1.
// ------------------------------------------------------------------------------------
constexpr int kPairStages = 4;
constexpr int kPairStageBytes = 3 * kPTileBytes;  // p0, p1 and this CTA's half of [q0 ; q1]
constexpr int kPairThreads = 64 + 32 * 8;
constexpr int kPairZeroBytes = 64 * kTileKBytes;  // this CTA's half of a 128-row all-zero column-side tile

template <bool kFast, bool kKara>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kPairThreads, 1)
residue_gemm_pair_kernel(const __grid_constant__ CUtensorMap map_p, const __grid_constant__ CUtensorMap map_q,
                         const __grid_constant__ CUtensorMap map_qh, const __grid_constant__ GemmCore p,
                         const __grid_constant__ ResidueParams ep) {
  constexpr int W = 128;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* zero_tile = tiles + kPairStages * kPairStageBytes;  // 64 rows x 128 bytes of E2M1 zeros
  GemmShared* sh = reinterpret_cast<GemmShared*>(zero_tile + kPairZeroBytes);
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  for (int i = threadIdx.x; i < kPairZeroBytes / 16; i += blockDim.x) reinterpret_cast<uint4*>(zero_tile)[i] = make_uint4(0, 0, 0, 0);
  fence_proxy_async();  // the tensor core reads this tile through the async proxy
  const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
  const int total_items = p.L * p.tiles_p * p.tiles_q;  // tiles_p counts 256-wide column tiles here

  if (threadIdx.x == 0) {
    prefetch_tensormap(&map_p);
    prefetch_tensormap(&map_q);
    for (int s = 0; s < kPairStages; ++s) {
      mbar_init(smem_u32(&sh->full[s]), 1);   // used in the leader only
      mbar_init(smem_u32(&sh->empty[s]), 1);
    }
    mbar_init(smem_u32(&sh->tmem_full), 1);
    mbar_init(smem_u32(&sh->tmem_empty), 16);  // 8 epilogue warps of each CTA; used in the leader only
    mbar_init(smem_u32(&sh->drained), 1);
    sh->abort = 0;
    fence_barrier_init();
    fence_proxy_async();
  }
  if (warp == 1) {
    tmem_alloc_pair(smem_u32(&sh->tmem_base), kTmemCols);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sh->tmem_base;
  if (warp >= 2) {
    const uint32_t quad = (uint32_t)(warp & 3), half = (uint32_t)((warp - 2) >> 2);
    const uint32_t lane_base = tmem + ((quad * 32u) << 16);
    if (half == 0) {  // constant UE8M0 scale bytes
      tmem_st_32x8_const(lane_base + kScaleCol, p.scale_word);
      tmem_st_32x8_const(lane_base + kScaleCol + 8, p.scale_word);
    }
    tmem_wait_st();
  }
  tc_fence_before();
  __syncthreads();
  cluster_arrive();  // the peer's barriers are initialised before anything is sent to them
  cluster_wait();
  tc_fence_after();

  if (warp == 0) {
    // ------------------------------ TMA producer (both CTAs) ------------------------------
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      const uint64_t pol_keep = l2_policy_evict_last(), pol_stream = l2_policy_evict_first();
      for (int item = pair; item < total_items && ok; item += npairs) {
        int l, tp, tq;
        decode_item(p, item, l, tp, tq);
        if (p.wave_counter) {  // both CTAs of every pair take part: 2 * npairs arrivals per wave
          const long long wave = item / npairs;
          const long long target = 2 * min((wave + 1) * (long long)npairs, (long long)total_items);
          if (!wave_barrier(p.wave_counter, (unsigned int)target, &sh->abort, p.status)) break;
        }
        const bool kara = kKara && karatsuba_modulus(l);
        for (int kb = 0; kb < p.kblocks; ++kb) {
          if (!wait_bounded(smem_u32(&sh->empty[stage]), phase ^ 1u, &sh->abort, p.status, 0x300 + stage)) {
            ok = false;
            break;
          }
          const uint32_t leader_full = map_to_cta(smem_u32(&sh->full[stage]), 0);
          const uint32_t dst = smem_u32(tiles + stage * kPairStageBytes);
          if (rank == 0) mbar_arrive_expect_tx(smem_u32(&sh->full[stage]), 2 * kPairStageBytes);
          const int x = kb * kTileKBytes;
          const int prow = (2 * tp + (int)rank) * kTileRows;
          // L2 priorities: the column-side tiles of the band are reused by every row tile of the band and
          // should stay; the row-side tiles are shared only within the current wave and may leave first
          tma_load_3d_pair_hint(dst + 0 * kPTileBytes, &map_p, leader_full, x, prow, 2 * l + 0, pol_keep);
          tma_load_3d_pair_hint(dst + 1 * kPTileBytes, &map_p, leader_full, x, prow, 2 * l + 1, pol_keep);
          if ((p.skip_top_first && l == 0) || kara) {
            // m = 169 needs p0 q0, p0 q1, p1 q0 only, a Karatsuba modulus p0 q0, p1 q1 here (and ps qs from the next
            // stage): 128-column instructions, for which this CTA supplies rows [64 rank, 64 rank + 64) of q0 and of
            // q1 instead of all of one of them
            tma_load_3d_pair(dst + 2 * kPTileBytes, &map_qh, leader_full, x, tq * W + 64 * (int)rank, 2 * l + 0);
            tma_load_3d_pair(dst + 2 * kPTileBytes + kPTileBytes / 2, &map_qh, leader_full, x, tq * W + 64 * (int)rank, 2 * l + 1);
          } else {
            tma_load_3d_pair_hint(dst + 2 * kPTileBytes, &map_q, leader_full, x, tq * W, 2 * l + (int)rank, pol_stream);
          }
          if (++stage == kPairStages) stage = 0, phase ^= 1u;
          if (kara) {
            // second stage of the k block: the sum-limb tiles ps (this CTA's 128 rows) and qs (its 64 rows)
            if (!wait_bounded(smem_u32(&sh->empty[stage]), phase ^ 1u, &sh->abort, p.status, 0x300 + stage)) {
              ok = false;
              break;
            }
            const uint32_t leader_full2 = map_to_cta(smem_u32(&sh->full[stage]), 0);
            const uint32_t dst2 = smem_u32(tiles + stage * kPairStageBytes);
            if (rank == 0) mbar_arrive_expect_tx(smem_u32(&sh->full[stage]), 2 * (kPTileBytes + kPTileBytes / 2));
            const int sp = p.sum_plane_base + karatsuba_rank(l);
            tma_load_3d_pair_hint(dst2, &map_p, leader_full2, x, prow, sp, pol_keep);
            tma_load_3d_pair(dst2 + 2 * kPTileBytes, &map_qh, leader_full2, x, tq * W + 64 * (int)rank, sp);
            if (++stage == kPairStages) stage = 0, phase ^= 1u;
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer (leader only) ------------------------------
    if (lane == 0 && rank == 0) {
      int stage = 0;
      uint32_t phase = 0, acc_phase = 0;
      const uint32_t sf = tmem + kScaleCol;
      constexpr uint32_t kIdesc = idesc_mxf4_pair(2 * W);
      bool ok = true;
      const bool count = p.count_cycles != 0;
      long long clk_start = count ? clock64() : 0, clk_empty = 0, clk_full = 0, clk_a = 0;
      for (int item = pair; item < total_items && ok; item += npairs) {
        int l, tp, tq;
        decode_item(p, item, l, tp, tq);
        const bool three = p.skip_top_first && l == 0;
        const bool kara = kKara && karatsuba_modulus(l);
        if (count) clk_a = clock64();
        if (!wait_bounded(smem_u32(&sh->tmem_empty), acc_phase ^ 1u, &sh->abort, p.status, 0x400)) break;
        if (count) clk_empty += clock64() - clk_a;
        tc_fence_after();
        for (int kb = 0; kb < p.kblocks; ++kb) {
          if (count) clk_a = clock64();
          if (!wait_bounded(smem_u32(&sh->full[stage]), phase, &sh->abort, p.status, 0x410 + stage)) {
            ok = false;
            break;
          }
          if (count) clk_full += clock64() - clk_a;
          tc_fence_after();
          const uint32_t base = smem_u32(tiles + stage * kPairStageBytes);
          if (kara) {
            // Karatsuba: a0 b0 and a1 b1 from this stage, (a0 + a1)(b0 + b1) from the next one
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
              const uint32_t first = (kb == 0 && ks == 0) ? 0u : 1u;
              mma_mxf4_pair(tmem + 0, smem_desc_sw128(base + 0 * kPTileBytes + ks * 32),
                            smem_desc_sw128(base + 2 * kPTileBytes + ks * 32), idesc_mxf4_pair(W), sf, sf, first);
              mma_mxf4_pair(tmem + 2 * W, smem_desc_sw128(base + 1 * kPTileBytes + ks * 32),
                            smem_desc_sw128(base + 2 * kPTileBytes + kPTileBytes / 2 + ks * 32), idesc_mxf4_pair(W), sf, sf, first);
            }
            mma_commit_pair(smem_u32(&sh->empty[stage]), (uint16_t)3);
            if (++stage == kPairStages) stage = 0, phase ^= 1u;
            if (count) clk_a = clock64();
            if (!wait_bounded(smem_u32(&sh->full[stage]), phase, &sh->abort, p.status, 0x410 + stage)) {
              ok = false;
              break;
            }
            if (count) clk_full += clock64() - clk_a;
            tc_fence_after();
            const uint32_t base2 = smem_u32(tiles + stage * kPairStageBytes);
#pragma unroll
            for (int ks = 0; ks < 4; ++ks)
              mma_mxf4_pair(tmem + W, smem_desc_sw128(base2 + ks * 32), smem_desc_sw128(base2 + 2 * kPTileBytes + ks * 32),
                            idesc_mxf4_pair(W), sf, sf, (kb == 0 && ks == 0) ? 0u : 1u);
          } else if (three) {
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
              const uint32_t first = (kb == 0 && ks == 0) ? 0u : 1u;
              const uint64_t p0 = smem_desc_sw128(base + 0 * kPTileBytes + ks * 32);
              const uint64_t p1 = smem_desc_sw128(base + 1 * kPTileBytes + ks * 32);
              const uint64_t q0 = smem_desc_sw128(base + 2 * kPTileBytes + ks * 32);
              const uint64_t q1 = smem_desc_sw128(base + 2 * kPTileBytes + kPTileBytes / 2 + ks * 32);
              mma_mxf4_pair(tmem + 0, p0, q0, idesc_mxf4_pair(W), sf, sf, first);
              mma_mxf4_pair(tmem + W, p0, q1, idesc_mxf4_pair(W), sf, sf, first);
              mma_mxf4_pair(tmem + W, p1, q0, idesc_mxf4_pair(W), sf, sf, 1u);
            }
          } else {
            if (kb == 0)  // p1 times an all-zero column-side tile, "overwrite": the 13^2 accumulator starts from 0
              mma_mxf4_pair(tmem + 2 * W, smem_desc_sw128(base + 1 * kPTileBytes), smem_desc_sw128(smem_u32(zero_tile)),
                            idesc_mxf4_pair(W), sf, sf, 0u);
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
              const uint64_t q = smem_desc_sw128(base + 2 * kPTileBytes + ks * 32);
              mma_mxf4_pair(tmem + 0, smem_desc_sw128(base + 0 * kPTileBytes + ks * 32), q, kIdesc, sf, sf,
                            (kb == 0 && ks == 0) ? 0u : 1u);
              mma_mxf4_pair(tmem + W, smem_desc_sw128(base + 1 * kPTileBytes + ks * 32), q, kIdesc, sf, sf, 1u);
            }
          }
          mma_commit_pair(smem_u32(&sh->empty[stage]), (uint16_t)3);
          if (++stage == kPairStages) stage = 0, phase ^= 1u;
        }
        if (!ok) break;
        mma_commit_pair(smem_u32(&sh->tmem_full), (uint16_t)3);
        acc_phase ^= 1u;
      }
      if (count && blockIdx.x == 0) {  // measurement aid: where the issuing thread of pair 0 spent its clocks
        p.status->mma_clk_total = clock64() - clk_start;
        p.status->mma_clk_wait_tmem = clk_empty;
        p.status->mma_clk_wait_operands = clk_full;
      }
      if (sh->abort) {
        mma_commit_pair(smem_u32(&sh->drained), (uint16_t)1);
        const uint64_t t0 = global_timer_ns();
        while (!mbar_try_wait(smem_u32(&sh->drained), 0u) && global_timer_ns() - t0 < kWaitLimitNs) {
        }
      }
    }
  } else {
    // ------------------------------ epilogue (both CTAs) ----------------------------------
    const uint32_t quad = (uint32_t)(warp & 3), half = (uint32_t)((warp - 2) >> 2);
    const uint32_t base = tmem + ((quad * 32u) << 16) + half * 64u;
    const uint32_t leader_empty = map_to_cta(smem_u32(&sh->tmem_empty), 0);
    uint32_t acc_phase = 0;
    for (int item = pair; item < total_items; item += npairs) {
      int l, tp, tq;
      decode_item(p, item, l, tp, tq);
      if (!__all_sync(0xFFFFFFFFu, wait_bounded(smem_u32(&sh->tmem_full), acc_phase, &sh->abort, p.status, 0x500 + warp))) break;
      tc_fence_after();
      const uint32_t m = (uint32_t)ep.m[l], recip = ep.recip[l], offset = ep.offset[l];
      uint32_t t[64];
      const int mode = (p.skip_top_first && l == 0) ? 0 : ((kKara && karatsuba_modulus(l)) ? 2 : 1);
      drain_and_release<kFast, false, kKara>(base, W, mode, offset, leader_empty, true, lane, t);
      const int64_t j = (int64_t)(2 * tp + (int)rank) * kTileRows + quad * 32 + lane;
      uint4* dst = reinterpret_cast<uint4*>(ep.res + (size_t)l * ep.res_stride + (size_t)j * (size_t)ep.res_ld +
                                            (size_t)tq * W + half * 64);
      reduce_and_store(t, m, recip, dst);
      acc_phase ^= 1u;
    }
  }

  tc_fence_before();
  __syncthreads();
  cluster_arrive();  // neither CTA leaves while the other may still signal its barriers
  cluster_wait();
  tc_fence_after();
  if (warp == 1) {
    __syncwarp();
    tmem_dealloc_pair(tmem, kTmemCols);
  }
}

// ------------------------------------------------------------------------------------
// DGEMM path for short K on CTA pairs: the two-accumulator form (see kGammaTileW in ozk_common.cuh).
//   ab = p0 beta + p1 gamma (mod m):  D_lo = p0 beta0 + p1 gamma0,  D_hi = p0 beta1 + p1 gamma1,  r = (D_lo + 13 D_hi) mod m
// p0, p1 are the B-matrix limbs (TMEM lanes), beta = the A-matrix residue and gamma = 13 * it, two limbs each, stacked
// along the TMEM columns: per K step two N = 240 instructions, p0 x [beta0 ; beta1] and p1 x [gamma0 ; gamma1], both
// into the same 240 columns.  A 256 x 120 tile needs 240 columns, so two accumulator sets fit tensor memory beside the
// scale-factor columns: the epilogue drains one set while the tensor core fills the other, which hides the turn-around
// of about 4 k clocks per tile that the three-accumulator kernel above pays (a third of a tile's time at K = 1024).
// Price: the A side carries four planes per modulus, and a stage holds 62 KiB (three stages).
// Each CTA loads its own p0, p1 rows, and of the stacked column-side operands the leader keeps beta0 and gamma0, its peer
// beta1 and gamma1 (120 rows each).
// ------------------------------------------------------------------------------------
constexpr int kGW = kGammaTileW;
static_assert(14 * 128 * kGammaMaxK < (1 << 22), "the epilogue holds D_lo + 13 D_hi plus an offset above 2^22 in 23 bits");
constexpr int kGQBytes = kGW * kTileKBytes;                      // one 120-row tile of a column-side plane
constexpr int kGStageBytes = 2 * kPTileBytes + 2 * kGQBytes;     // p0, p1, this CTA's halves of [beta0 ; beta1] and [gamma0 ; gamma1]
constexpr int kGStages = 3;
struct __align__(8) GammaShared {
  uint64_t full[kGStages];
  uint64_t empty[kGStages];
  uint64_t tmem_full[2];   // per accumulator set
  uint64_t tmem_empty[2];
  uint64_t staged[2];      // per output buffer: the 8 epilogue warps have written their residues
  uint64_t drained;
  uint32_t tmem_base;
  volatile int abort;
};
constexpr int kGOutBytes = kTileRows * kGW;  // residues of one CTA's 128 columns x 120 rows, one byte each
constexpr size_t kGammaSmemBytes = (size_t)kGStages * kGStageBytes + 2 * kGOutBytes + sizeof(GammaShared) + 1024;

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kPairThreads, 1)
residue_gemm_gamma_kernel(const __grid_constant__ CUtensorMap map_p, const __grid_constant__ CUtensorMap map_q,
                          const __grid_constant__ GemmCore p, const __grid_constant__ ResidueParams ep, int64_t rows_padded) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* out_stage = tiles + kGStages * kGStageBytes;  // two buffers of kGOutBytes
  GammaShared* sh = reinterpret_cast<GammaShared*>(out_stage + 2 * kGOutBytes);
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int pair = blockIdx.x >> 1, npairs = gridDim.x >> 1;
  const int total_items = p.L * p.tiles_p * p.tiles_q;  // tiles_p: 256-wide column tiles, tiles_q: 120-wide row tiles

  if (threadIdx.x == 0) {
    prefetch_tensormap(&map_p);
    prefetch_tensormap(&map_q);
    for (int s = 0; s < kGStages; ++s) {
      mbar_init(smem_u32(&sh->full[s]), 1);   // used in the leader only
      mbar_init(smem_u32(&sh->empty[s]), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(smem_u32(&sh->tmem_full[a]), 1);
      mbar_init(smem_u32(&sh->tmem_empty[a]), 16);  // 8 epilogue warps of each CTA; used in the leader only
      mbar_init(smem_u32(&sh->staged[a]), 8);
    }
    mbar_init(smem_u32(&sh->drained), 1);
    sh->abort = 0;
    fence_barrier_init();
    fence_proxy_async();
  }
  if (warp == 1) {
    tmem_alloc_pair(smem_u32(&sh->tmem_base), kTmemCols);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sh->tmem_base;
  if (warp >= 2) {
    const uint32_t quad = (uint32_t)(warp & 3), half = (uint32_t)((warp - 2) >> 2);
    if (half == 0) {  // constant UE8M0 scale bytes
      tmem_st_32x8_const(tmem + ((quad * 32u) << 16) + kScaleCol, p.scale_word);
      tmem_st_32x8_const(tmem + ((quad * 32u) << 16) + kScaleCol + 8, p.scale_word);
    }
    tmem_wait_st();
  }
  tc_fence_before();
  __syncthreads();
  cluster_arrive();  // the peer's barriers are initialised before anything is sent to them
  cluster_wait();
  tc_fence_after();

  if (warp == 0) {
    // ------------------------------ TMA producer (both CTAs) ------------------------------
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      const uint64_t pol_keep = l2_policy_evict_last(), pol_stream = l2_policy_evict_first();
      unsigned int seen = 0, probe = 0;  // the wave counter as last known, and as read during the previous item
      ItemCursor cur;
      cur.init(p, pair);
      int wave = 0;
      for (int item = pair; item < total_items && ok; item += npairs, ++wave, cur.advance(p, npairs)) {
        const int l = cur.l;
        int tp, tq;
        cur.tile(p, tp, tq);
        if (p.wave_counter) {
          // Both CTAs of every pair announce each item (2 * npairs arrivals per wave) and wait for the arrivals of the
          // wave before the previous one: the pairs stay within three tiles of each other (the planes of a modulus stay in L2
          // at these K), and no round trip to the counter is paid per tile.
          if (probe > seen) seen = probe;
          const long long target = wave >= 2 ? 2 * min((long long)(wave - 1) * npairs, (long long)total_items) : 0;
          if (!wave_barrier_lagged(p.wave_counter, (unsigned int)target, seen, &sh->abort, p.status)) break;
          probe = wave_counter_probe(p.wave_counter);
        }
        for (int kb = 0; kb < p.kblocks; ++kb) {
          if (!wait_bounded(smem_u32(&sh->empty[stage]), phase ^ 1u, &sh->abort, p.status, 0x600 + stage)) {
            ok = false;
            break;
          }
          const uint32_t leader_full = map_to_cta(smem_u32(&sh->full[stage]), 0);
          const uint32_t dst = smem_u32(tiles + stage * kGStageBytes);
          if (rank == 0) mbar_arrive_expect_tx(smem_u32(&sh->full[stage]), 2 * kGStageBytes);
          const int x = kb * kTileKBytes;
          const int prow = (2 * tp + (int)rank) * kTileRows;
          tma_load_3d_pair_hint(dst, &map_p, leader_full, x, prow, 2 * l, pol_keep);                           // p0, p1
          tma_load_4d_pair_hint(dst + 2 * kPTileBytes, &map_q, leader_full, x, tq * kGW, 2 * l + (int)rank, 0, pol_stream);  // beta, gamma
          if (++stage == kGStages) stage = 0, phase ^= 1u;
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer (leader only) ------------------------------
    if (lane == 0 && rank == 0) {
      int stage = 0;
      uint32_t phase = 0;
      const uint32_t sf = tmem + kScaleCol;
      constexpr uint32_t kIdesc = idesc_mxf4_pair(2 * kGW);

      bool ok = true;
      const bool count = p.count_cycles != 0;
      long long clk_start = count ? clock64() : 0, clk_empty = 0, clk_full = 0, clk_a = 0;
      int n = 0;
      for (int item = pair; item < total_items && ok; item += npairs, ++n) {
        const int set = n & 1;
        const uint32_t set_phase = (uint32_t)((n >> 1) & 1);
        const uint32_t acc = tmem + (uint32_t)(set * 2 * kGW);
        if (count) clk_a = clock64();
        if (!wait_bounded(smem_u32(&sh->tmem_empty[set]), set_phase ^ 1u, &sh->abort, p.status, 0x700 + set)) break;
        if (count) clk_empty += clock64() - clk_a;
        tc_fence_after();
        for (int kb = 0; kb < p.kblocks; ++kb) {
          if (count) clk_a = clock64();
          if (!wait_bounded(smem_u32(&sh->full[stage]), phase, &sh->abort, p.status, 0x710 + stage)) {
            ok = false;
            break;
          }
          if (count) clk_full += clock64() - clk_a;
          tc_fence_after();
          const uint32_t base = smem_u32(tiles + stage * kGStageBytes);
#pragma unroll
          for (int ks = 0; ks < 4; ++ks) {
            mma_mxf4_pair(acc, smem_desc_sw128(base + 0 * kPTileBytes + ks * 32), smem_desc_sw128(base + 2 * kPTileBytes + ks * 32), kIdesc,
                          sf, sf, (kb == 0 && ks == 0) ? 0u : 1u);
            mma_mxf4_pair(acc, smem_desc_sw128(base + 1 * kPTileBytes + ks * 32),
                          smem_desc_sw128(base + 2 * kPTileBytes + kGQBytes + ks * 32), kIdesc, sf, sf, 1u);
          }
          mma_commit_pair(smem_u32(&sh->empty[stage]), (uint16_t)3);
          if (++stage == kGStages) stage = 0, phase ^= 1u;
        }
        if (!ok) break;
        mma_commit_pair(smem_u32(&sh->tmem_full[set]), (uint16_t)3);
      }
      if (count && blockIdx.x == 0) {
        p.status->mma_clk_total = clock64() - clk_start;
        p.status->mma_clk_wait_tmem = clk_empty;
        p.status->mma_clk_wait_operands = clk_full;
      }
      if (sh->abort) {
        mma_commit_pair(smem_u32(&sh->drained), (uint16_t)1);
        const uint64_t t0 = global_timer_ns();
        while (!mbar_try_wait(smem_u32(&sh->drained), 0u) && global_timer_ns() - t0 < kWaitLimitNs) {
        }
      }
    }
  } else {
    // ------------------------------ epilogue (both CTAs) ----------------------------------
    // warp (quadrant q, half h): lanes 32 q .., columns [0, 64) or [64, 120) of both accumulators, 8 at a time.
    // The residues cross shared memory so that they leave as whole rows: a thread's 64 or 56 bytes (column j of C, rows
    // col0 ..) go into row quad * 32 + lane of an output buffer (120-byte pitch: the 8-byte writes of a warp fall on 16
    // distinct bank pairs), and each warp writes 16 of the 128 rows to memory, 30 lanes x 4 bytes = one 120-byte run of a
    // residue column per instruction (stored from the registers, a warp's store would touch 32 lines with 8 bytes each).
    // Two buffers: the rows of the previous tile are written out between the arithmetic of the current one, two rows
    // per chunk, so the store queue never holds the warp up.
    const uint32_t quad = (uint32_t)(warp & 3), half = (uint32_t)((warp - 2) >> 2);
    const int col0 = half ? 64 : 0, chunks = half ? 7 : 8;
    const uint32_t lane_base = tmem + ((quad * 32u) << 16) + (uint32_t)col0;
    const int row0 = (warp - 2) * 16;  // the rows of an output buffer this warp writes to memory
    const uint32_t out_base = smem_u32(out_stage);
    const uint32_t out_mine = (quad * 32u + (uint32_t)lane) * (uint32_t)kGW + (uint32_t)col0;
    const uint32_t out_rows = (uint32_t)(row0 * kGW + 4 * lane);
    constexpr uint32_t kInsert[4] = {0x3214u, 0x3240u, 0x3410u, 0x4210u};
    const float kOneTiny = __uint_as_float(1u), kThirteenTiny = __uint_as_float(13u);  // 2^-149 and 13 * 2^-149
    uint8_t* prev_dst = nullptr;  // where this warp's rows of the previous tile go; null: nothing pending (or beyond the rows)
    bool ok = true;
    int n = 0;
    ItemCursor cur;
    cur.init(p, pair);
    for (int item = pair; item < total_items; item += npairs, ++n, cur.advance(p, npairs)) {
      const int l = cur.l;
      int tp, tq;
      cur.tile(p, tp, tq);
      const int set = n & 1;
      const uint32_t set_phase = (uint32_t)((n >> 1) & 1);
      const uint32_t leader_empty = map_to_cta(smem_u32(&sh->tmem_empty[set]), 0);
      if (!__all_sync(0xFFFFFFFFu, wait_bounded(smem_u32(&sh->tmem_full[set]), set_phase, &sh->abort, p.status, 0x800 + warp))) {
        ok = false;
        break;
      }
      tc_fence_after();
      const uint32_t base = lane_base + (uint32_t)(set * 2 * kGW);
      uint32_t lo[8][8], hi[8][8];
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        if (c < chunks) {
          tmem_ld_32x8(base + 8 * c, lo[c]);
          tmem_ld_32x8(base + kGW + 8 * c, hi[c]);
        }
      }
      tmem_wait_ld();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(leader_empty);
      // every warp has put the previous tile into the other buffer, and has finished reading this one (the tile before that)
      if (n > 0 && !__all_sync(0xFFFFFFFFu, wait_bounded(smem_u32(&sh->staged[set ^ 1]), (uint32_t)(((n - 1) >> 1) & 1), &sh->abort,
                                                          p.status, 0x900 + warp))) {
        ok = false;
        break;
      }
      // |D_lo + 13 D_hi| <= 14 * 128 K < 2^22 for K <= kGammaMaxK; offset: the multiple of m just above 2^22
      const uint32_t m = (uint32_t)ep.m[l], recip1 = ep.recip[l] + 1u;
      const float offset_tiny = __uint_as_float(m * ((1u << 22) / m + 1u));  // as a subnormal: bit pattern = integer
      const uint32_t out_cur = out_base + (uint32_t)(set * kGOutBytes), out_prev = out_base + (uint32_t)((set ^ 1) * kGOutBytes);
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        if (c < chunks) {
          uint32_t w[2] = {0u, 0u};
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            // y = D_lo + 13 D_hi + offset < 2^23, formed as y * 2^-149: the bit pattern of that subnormal is the integer
            // y itself (both multiply-adds are exact), so no conversion is needed
            const uint32_t y = __float_as_uint(fmaf(__uint_as_float(hi[c][e]), kThirteenTiny, fmaf(__uint_as_float(lo[c][e]), kOneTiny, offset_tiny)));
            const uint32_t r = y - __umulhi(y, recip1) * m;  // exact for y < 2^24: recip1 = floor(2^32 / m) + 1
            w[e >> 2] = e & 3 ? __byte_perm(w[e >> 2], r, kInsert[e & 3]) : r;
          }
          asm volatile("st.shared.v2.u32 [%0], {%1, %2};" ::"r"(out_cur + out_mine + 8u * c), "r"(w[0]), "r"(w[1]) : "memory");
        }
        if (prev_dst) {  // rows 2 c and 2 c + 1 of the previous tile
          uint32_t v0, v1;
          asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v0) : "r"(out_prev + out_rows + (uint32_t)(2 * c * kGW)) : "memory");
          asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v1) : "r"(out_prev + out_rows + (uint32_t)((2 * c + 1) * kGW)) : "memory");
          *reinterpret_cast<uint32_t*>(prev_dst + (size_t)(2 * c) * (size_t)ep.res_ld) = v0;
          *reinterpret_cast<uint32_t*>(prev_dst + (size_t)(2 * c + 1) * (size_t)ep.res_ld) = v1;
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&sh->staged[set]));
      const int64_t i = (int64_t)tq * kGW + 4 * lane;  // the last row tile may reach past the padded rows
      prev_dst = (lane < kGW / 4 && i < rows_padded)
                     ? ep.res + (size_t)l * ep.res_stride + (size_t)((int64_t)(2 * tp + (int)rank) * kTileRows + row0) * (size_t)ep.res_ld + (size_t)i
                     : nullptr;
    }
    if (ok && n > 0) {  // the rows of the last tile
      const int set = (n - 1) & 1;
      if (__all_sync(0xFFFFFFFFu, wait_bounded(smem_u32(&sh->staged[set]), (uint32_t)(((n - 1) >> 1) & 1), &sh->abort, p.status, 0x900 + warp)) &&
          prev_dst) {
        const uint32_t src = out_base + (uint32_t)(set * kGOutBytes) + out_rows;
#pragma unroll
        for (int r = 0; r < 16; ++r) {
          uint32_t v;
          asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(src + (uint32_t)(r * kGW)) : "memory");
          *reinterpret_cast<uint32_t*>(prev_dst + (size_t)r * (size_t)ep.res_ld) = v;
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  cluster_arrive();  // neither CTA leaves while the other may still signal its barriers
  cluster_wait();
  tc_fence_after();
  if (warp == 1) {
    __syncwarp();
    tmem_dealloc_pair(tmem, kTmemCols);
  }
}

// ------------------------------------------------------------------------------------
// Probe: one 128 x 128 tile, serial load -> MMA -> read-back, FP32 accumulators written out.
// Pins the hardware formats (nibble order, E2M1 codes, UE8M0 byte, accumulator exactness).
// ------------------------------------------------------------------------------------
struct ProbeShared {
  uint64_t full;
  uint64_t done;
  uint32_t tmem_base;
  volatile int abort;
};

__global__ void __launch_bounds__(192, 1)
mma_probe_kernel(const __grid_constant__ CUtensorMap map_p, const __grid_constant__ CUtensorMap map_q, int kblocks,
                 uint32_t scale_word, float* __restrict__ D, StatusBlock* status, uint32_t extra_tx) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  ProbeShared* sh = reinterpret_cast<ProbeShared*>(tiles + 2 * kPTileBytes);
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&sh->full), 1);
    mbar_init(smem_u32(&sh->done), 1);
    sh->abort = 0;
    fence_barrier_init();
    fence_proxy_async();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&sh->tmem_base), 256);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sh->tmem_base;
  if (warp >= 2) {
    const uint32_t quad = (uint32_t)(warp & 3);
    tmem_st_32x8_const(tmem + ((quad * 32u) << 16) + 128, scale_word);
    tmem_wait_st();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 1 && lane == 0) {
    const uint32_t base = smem_u32(tiles);
    const uint32_t sf = tmem + 128;
    uint32_t phase = 0;
    for (int kb = 0; kb < kblocks; ++kb) {
      // extra_tx > 0 (test aid): the barrier expects bytes that nobody sends, so the bounded wait below runs out
      mbar_arrive_expect_tx(smem_u32(&sh->full), 2 * kPTileBytes + extra_tx);
      tma_load_2d(base, &map_p, smem_u32(&sh->full), kb * kTileKBytes, 0);
      tma_load_2d(base + kPTileBytes, &map_q, smem_u32(&sh->full), kb * kTileKBytes, 0);
      const uint64_t t0 = global_timer_ns();
      while (!mbar_try_wait(smem_u32(&sh->full), phase)) {
        if (global_timer_ns() - t0 > kWaitLimitNs) {
          sh->abort = 1;
          break;
        }
      }
      if (sh->abort) break;
      tc_fence_after();
      for (int ks = 0; ks < 4; ++ks)
        mma_mxf4(tmem, smem_desc_sw128(base + ks * 32), smem_desc_sw128(base + kPTileBytes + ks * 32),
                 idesc_mxf4(128), sf, sf, (kb | ks) ? 1u : 0u);
      mma_commit(smem_u32(&sh->done));
      const uint64_t t1 = global_timer_ns();
      while (!mbar_try_wait(smem_u32(&sh->done), phase)) {
        if (global_timer_ns() - t1 > kWaitLimitNs) {
          sh->abort = 1;
          break;
        }
      }
      if (sh->abort) break;
      phase ^= 1u;
    }
    if (sh->abort) atomicMin(&status->code, (int)OZK_ERR_DEVICE_TIMEOUT);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp >= 2 && !sh->abort) {
    const uint32_t quad = (uint32_t)(warp & 3);
    const int row = quad * 32 + lane;
    for (int c = 0; c < 4; ++c) {
      uint32_t d[32];
      tmem_ld_32x32(tmem + ((quad * 32u) << 16) + c * 32, d);
      tmem_wait_ld();
      for (int e = 0; e < 32; ++e) D[row * 128 + c * 32 + e] = __uint_as_float(d[e]);
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 1) {
    __syncwarp();
    tmem_dealloc(tmem, 256);
  }
}


// ------------------------------------------------------------------------------------
// Host side
// ------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(sym);
  }
  return fn;
}

// Planes of one operand as a (bytes along K, rows, plane) byte tensor; box = 128 bytes x box_rows.
// Rows of a box that fall outside the tensor are filled with zero bytes (E2M1 code 0 = value 0).
bool make_plane_map(CUtensorMap* map, const void* base, int64_t k_bytes, int64_t rows, int64_t planes, size_t plane_bytes,
                    int box_rows, size_t pitch = 0, int box_planes = 1) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  cuuint64_t dims[3] = {(cuuint64_t)k_bytes, (cuuint64_t)rows, (cuuint64_t)planes};
  cuuint64_t strides[2] = {(cuuint64_t)(pitch ? pitch : (size_t)k_bytes), (cuuint64_t)plane_bytes};
  cuuint32_t box[3] = {(cuuint32_t)kTileKBytes, (cuuint32_t)box_rows, (cuuint32_t)box_planes};
  cuuint32_t estr[3] = {1, 1, 1};
  const int rank = planes > 0 ? 3 : 2;
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, rank, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// A-side planes of the two-accumulator form as a (bytes along K, rows, plane, kind) tensor: kind 0 = the 2 L limb planes
// of beta, kind 1 = those of gamma, which follow them.  A box takes 120 rows of one plane of both kinds.
bool make_gamma_q_map(CUtensorMap* map, const void* base, int64_t k_bytes, int64_t rows, int L, size_t plane_bytes, size_t pitch) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  cuuint64_t dims[4] = {(cuuint64_t)k_bytes, (cuuint64_t)rows, (cuuint64_t)(2 * L), 2};
  cuuint64_t strides[3] = {(cuuint64_t)pitch, (cuuint64_t)plane_bytes, (cuuint64_t)plane_bytes * (cuuint64_t)(2 * L)};
  cuuint32_t box[4] = {(cuuint32_t)kTileKBytes, (cuuint32_t)kGammaTileW, 1, 2};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// cudaFuncSetAttribute acts on the current device only: remember per device ordinal where it has been done.
constexpr int kMaxDevices = 64;
int current_device_ordinal() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return -1;
  return dev;
}

// The CTA-pair (cta_group::2) kernel runs whenever the padded column count is a multiple of 256;
// OZK_GEMM_PAIR=0 in the environment forces the single-CTA kernel (measurement aid).
bool pair_kernel_enabled() {
  static int v = -1;
  if (v < 0) {
    const char* e = getenv("OZK_GEMM_PAIR");
    v = (e && e[0] == '0') ? 0 : 1;
  }
  return v == 1;
}

// OZK_GEMM_THREE=0 in the environment makes the CTA-pair kernel run modulus 169 like the others (four products in two
// instructions, the 13^2 term cancelling in the epilogue) instead of three narrower instructions: a measurement aid.
bool three_product_enabled() {
  static int v = -1;
  if (v < 0) {
    const char* e = getenv("OZK_GEMM_THREE");
    v = (e && e[0] == '0') ? 0 : 1;
  }
  return v == 1;
}

template <int NP, int NQ, int W, int STAGES, class Epi>
ozk_status launch_limb_gemm(const CUtensorMap& map_p, const CUtensorMap& map_q, const GemmCore& core,
                            const typename Epi::Params& ep, cudaStream_t st) {
  constexpr size_t kStageBytes = (size_t)NP * kPTileBytes + (size_t)NQ * W * kTileKBytes;
  const size_t smem = STAGES * kStageBytes + sizeof(GemmShared) + 1024;
  auto kernel = limb_gemm_kernel<NP, NQ, W, STAGES, Epi>;
  static std::atomic<bool> attr_set[kMaxDevices];
  const int dev = current_device_ordinal();
  if (dev < 0) return OZK_ERR_CUDA;
  if (!attr_set[dev].load(std::memory_order_acquire)) {
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return OZK_ERR_CUDA;
    attr_set[dev].store(true, std::memory_order_release);
  }
  const int sms = device_sm_count();
  if (sms < 1) return OZK_ERR_CUDA;
  const long long items = (long long)core.L * core.tiles_p * core.tiles_q;
  const int grid = (int)(items < sms ? items : sms);
  kernel<<<grid, 64 + 32 * Epi::kWarps, smem, st>>>(map_p, map_q, core, ep);
  return cudaGetLastError() == cudaSuccess ? OZK_OK : OZK_ERR_CUDA;
}

}  // namespace

// DGEMM path: residues r_l[j][i] for all moduli from the limb planes in the workspace, over the
// k range [k0, k0 + klen) (multiples of 256; klen = 0 means all of Kp), written to `res` (default:
// the workspace's residue matrices).
ozk_status gemm_residues(const Geometry& g, const ModulusTable& mt, uint8_t* ws, cudaStream_t st, int64_t k0, int64_t klen,
                         uint8_t* res) {
  if (klen <= 0) klen = g.Kp - k0;
  if (k0 < 0 || k0 % kTileKNibbles || klen % kTileKNibbles || k0 + klen > g.Kp || klen > (g.karatsuba ? kChunkKKaratsuba : kChunkK))
    return OZK_ERR_INVALID_ARG;
  const uint8_t* planes_b = ws + g.off_planes_b + k0 / 2;
  const uint8_t* planes_a = ws + g.off_planes_a + k0 / 2;
  CUtensorMap map_p, map_q;
  const int planes = planes_per_operand(g.L, g.karatsuba);
  if (!make_plane_map(&map_p, planes_b, klen / 2, g.Np, planes, g.plane_bytes_b, kTileRows, g.pitch)) return OZK_ERR_CUDA;
  if (!make_plane_map(&map_q, planes_a, klen / 2, g.Mp, planes, g.plane_bytes_a, 128, g.pitch)) return OZK_ERR_CUDA;
  GemmCore core;
  core.L = g.L;
  core.tiles_p = (int)(g.Np / kTileRows);
  core.tiles_q = (int)(g.Mp / 128);
  core.kblocks = (int)(klen / kTileKNibbles);
  core.group = 16;
  core.skip_top_first = (mt.m[0] == 169) ? 1 : 0;  // 13^2 a1 b1 vanishes mod 169 (Section 5.1)
  core.q_groups = 0;
  // one FP32 multiply-add before the release needs 128 K + 13 * 64 K = 960 K < 2^24 (Karatsuba: 976 K)
  core.fast_combine = (g.karatsuba ? klen <= 17152 : (g.K <= 17476 || klen <= 17408)) ? 1 : 0;
  core.count_cycles = 0;
  core.karatsuba = 0;  // the single-CTA kernel runs the four products on the same planes
  core.sum_plane_base = 0;
  core.wave_counter = nullptr;
  core.status = reinterpret_cast<StatusBlock*>(ws + g.off_status);
  core.scale_word = 0x80808080u;  // UE8M0 byte 0x80 = 2: both operands doubled, accumulators hold integers
  ResidueParams ep;
  for (int l = 0; l < kMaxModuli; ++l) {
    ep.m[l] = mt.m[l];
    ep.recip[l] = mt.recip[l];
    ep.offset[l] = (uint32_t)mt.m[l] * (uint32_t)(0x80000000u / (uint32_t)mt.m[l]);
  }
  ep.res = res ? res : ws + g.off_res;
  ep.res_ld = g.Mp;
  ep.res_stride = (size_t)g.Mp * (size_t)g.Np;
  if (g.gamma && g.Np % 256 == 0 && pair_kernel_enabled()) {
    // short K: the two-accumulator kernel on CTA pairs (the A side holds beta planes 0 .. 2L-1 and gamma planes 2L .. 4L-1).
    // Cooperative launch like the pair kernel below, which also serves as its fallback (on the beta planes).
    GemmCore gc = core;
    gc.tiles_p = (int)(g.Np / 256);
    gc.tiles_q = (int)((g.Mp + kGW - 1) / kGW);
    gc.group = 8;
    gc.skip_top_first = 0;
    gc.count_cycles = stage_timing_enabled() ? 1 : 0;
    gc.sum_plane_base = 2 * g.L;
    gc.wave_counter = reinterpret_cast<unsigned int*>(ws + g.off_status + 512);
    CUtensorMap map_p2, map_q120;  // one copy brings p0 and p1, another this CTA's limb of beta and of gamma
    if (!make_plane_map(&map_p2, planes_b, klen / 2, g.Np, planes, g.plane_bytes_b, kTileRows, g.pitch, 2)) return OZK_ERR_CUDA;
    if (!make_gamma_q_map(&map_q120, planes_a, klen / 2, g.Mp, g.L, g.plane_bytes_a, g.pitch)) return OZK_ERR_CUDA;
    static std::atomic<bool> attr_set[kMaxDevices];
    const int dev = current_device_ordinal();
    if (dev < 0) return OZK_ERR_CUDA;
    if (!attr_set[dev].load(std::memory_order_acquire)) {
      if (cudaFuncSetAttribute(residue_gemm_gamma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kGammaSmemBytes) != cudaSuccess)
        return OZK_ERR_CUDA;
      attr_set[dev].store(true, std::memory_order_release);
    }
    const int max_pairs = device_sm_count() / 2;
    if (max_pairs < 1) return OZK_ERR_CUDA;
    const long long items = (long long)gc.L * gc.tiles_p * gc.tiles_q;
    const int pairs = (int)(items < max_pairs ? items : max_pairs);
    if (gc.wave_counter && cudaMemsetAsync(gc.wave_counter, 0, 4, st) != cudaSuccess) return OZK_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(2 * pairs), 1, 1);
    cfg.blockDim = dim3(kPairThreads, 1, 1);
    cfg.dynamicSmemBytes = kGammaSmemBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, residue_gemm_gamma_kernel, map_p2, map_q120, gc, ep, (int64_t)g.Mp) == cudaSuccess) return OZK_OK;
    (void)cudaGetLastError();  // refused: the kernels below run on the beta planes
  }
  if (g.Np % 256 == 0 && pair_kernel_enabled()) {
    // CTA-pair kernel.  Its producers meet at a global counter before every wave of items, which needs
    // all CTAs resident: the launch is cooperative, and when that is refused the single-CTA kernel runs.
    GemmCore pc = core;
    pc.tiles_p = (int)(g.Np / 256);
    pc.group = 8;  // 8 column tiles of 256: the same 2048-column band as the single-CTA kernel
    pc.skip_top_first = (mt.m[0] == 169 && three_product_enabled()) ? 1 : 0;  // 13^2 a1 b1 vanishes mod 169 (Section 5.1)
    pc.count_cycles = stage_timing_enabled() ? 1 : 0;
    CUtensorMap map_qh;  // 64-row boxes of the A-side planes, for the three-product form of m = 169
    if (!make_plane_map(&map_qh, planes_a, klen / 2, g.Mp, planes, g.plane_bytes_a, 64, g.pitch)) return OZK_ERR_CUDA;
    pc.karatsuba = g.karatsuba;
    pc.sum_plane_base = 2 * g.L;
    pc.wave_counter = reinterpret_cast<unsigned int*>(ws + g.off_status + 512);
    const size_t smem = (size_t)kPairStages * kPairStageBytes + kPairZeroBytes + sizeof(GemmShared) + 1024;
    static std::atomic<bool> attr_set[kMaxDevices];
    const int dev = current_device_ordinal();
    if (dev < 0) return OZK_ERR_CUDA;
    if (!attr_set[dev].load(std::memory_order_acquire)) {
      if (cudaFuncSetAttribute(residue_gemm_pair_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess ||
          cudaFuncSetAttribute(residue_gemm_pair_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess ||
          cudaFuncSetAttribute(residue_gemm_pair_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess ||
          cudaFuncSetAttribute(residue_gemm_pair_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return OZK_ERR_CUDA;
      attr_set[dev].store(true, std::memory_order_release);
    }
    const int max_pairs = device_sm_count() / 2;
    if (max_pairs < 1) return OZK_ERR_CUDA;
    const long long items = (long long)pc.L * pc.tiles_p * pc.tiles_q;
    const int pairs = (int)(items < max_pairs ? items : max_pairs);
    if (cudaMemsetAsync(pc.wave_counter, 0, 4, st) != cudaSuccess) return OZK_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(2 * pairs), 1, 1);
    cfg.blockDim = dim3(kPairThreads, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e;
    if (pc.karatsuba)
      e = pc.fast_combine ? cudaLaunchKernelEx(&cfg, residue_gemm_pair_kernel<true, true>, map_p, map_q, map_qh, pc, ep)
                          : cudaLaunchKernelEx(&cfg, residue_gemm_pair_kernel<false, true>, map_p, map_q, map_qh, pc, ep);
    else
      e = pc.fast_combine ? cudaLaunchKernelEx(&cfg, residue_gemm_pair_kernel<true, false>, map_p, map_q, map_qh, pc, ep)
                          : cudaLaunchKernelEx(&cfg, residue_gemm_pair_kernel<false, false>, map_p, map_q, map_qh, pc, ep);
    if (e == cudaSuccess) return OZK_OK;
    (void)cudaGetLastError();  // the cooperative launch was refused: fall through to the single-CTA kernel
  }
  if (core.fast_combine) return launch_limb_gemm<2, 2, 128, 3, ResidueEpilogue<true>>(map_p, map_q, core, ep, st);
  return launch_limb_gemm<2, 2, 128, 3, ResidueEpilogue<false>>(map_p, map_q, core, ep, st);
}

// INT8 path: C (int32, column-major) from three limb planes per operand.
// INT8 path: C (int32, column-major) from three limb planes per operand.  128 x 64 tiles: five accumulators of
// 64 columns, three N = 192 instructions per K step, and three 72 KiB stages (an 80-wide tile leaves room for two
// stages only and measured 5 to 11 % slower).
ozk_status gemm_int8(const uint8_t* planes_a, const uint8_t* planes_b, int64_t M, int64_t N, int64_t Mp, int64_t Np, int64_t Kp,
                     int32_t* C, int64_t ldc, StatusBlock* status, cudaStream_t st) {
  constexpr int W = 64;
  CUtensorMap map_p, map_q;
  if (!make_plane_map(&map_p, planes_b, Kp / 2, Np, 3, (size_t)Np * (size_t)(Kp / 2), kTileRows)) return OZK_ERR_CUDA;
  if (!make_plane_map(&map_q, planes_a, Kp / 2, Mp, 3, (size_t)Mp * (size_t)(Kp / 2), W)) return OZK_ERR_CUDA;
  GemmCore core;
  core.L = 1;
  core.tiles_p = (int)(Np / kTileRows);
  core.tiles_q = (int)((M + W - 1) / W);
  core.kblocks = (int)(Kp / kTileKNibbles);
  core.group = 16;
  core.skip_top_first = 0;
  core.q_groups = 0;
  core.wave_counter = nullptr;
  core.fast_combine = 0;
  core.count_cycles = 0;
  core.karatsuba = 0;
  core.sum_plane_base = 0;
  core.status = status;
  core.scale_word = 0x80808080u;
  Int32Epilogue::Params ep;
  ep.C = C;
  ep.ldc = ldc;
  ep.M = M;
  ep.N = N;
  return launch_limb_gemm<3, 3, W, 3, Int32Epilogue>(map_p, map_q, core, ep, st);
}

// Scheme-I passes: 16 row-side limb planes (the 16th all zero) in 4 groups of 4, 15 column-side planes in
// 5 groups of 3; pass l = 5 * (row group) + (column group) writes its int64 block value to out[l].
ozk_status gemm_oz1_passes(const uint8_t* planes_a, const uint8_t* planes_b, int64_t Mp, int64_t Np, int64_t Kp, int64_t M,
                           long long* out, int64_t out_ld, StatusBlock* status, cudaStream_t st) {
  constexpr int W = 80;
  CUtensorMap map_p, map_q;
  if (!make_plane_map(&map_p, planes_b, Kp / 2, Np, 16, (size_t)Np * (size_t)(Kp / 2), kTileRows)) return OZK_ERR_CUDA;
  if (!make_plane_map(&map_q, planes_a, Kp / 2, Mp, 15, (size_t)Mp * (size_t)(Kp / 2), W)) return OZK_ERR_CUDA;
  GemmCore core;
  core.L = 20;
  core.tiles_p = (int)(Np / kTileRows);
  core.tiles_q = (int)((M + W - 1) / W);
  core.kblocks = (int)(Kp / kTileKNibbles);
  core.group = 16;
  core.skip_top_first = 0;
  core.q_groups = 5;
  core.wave_counter = nullptr;
  core.fast_combine = 0;
  core.count_cycles = 0;
  core.karatsuba = 0;
  core.sum_plane_base = 0;
  core.status = status;
  core.scale_word = 0x80808080u;
  Int64BlockEpilogue::Params ep;
  ep.out = out;
  ep.ld = out_ld;
  ep.pass_stride = (size_t)Np * (size_t)out_ld;
  return launch_limb_gemm<4, 3, W, 2, Int64BlockEpilogue>(map_p, map_q, core, ep, st);
}

ozk_status gemm_probe(const uint8_t* P, const uint8_t* Q, int64_t K, int scale_byte, float* D, uint8_t* ws, cudaStream_t st,
                      bool let_wait_expire) {
  CUtensorMap map_p, map_q;
  if (!make_plane_map(&map_p, P, K / 2, kTileRows, 0, 0, kTileRows)) return OZK_ERR_CUDA;
  if (!make_plane_map(&map_q, Q, K / 2, kTileRows, 0, 0, kTileRows)) return OZK_ERR_CUDA;
  const size_t smem = 2 * kPTileBytes + sizeof(ProbeShared) + 1024;
  if (cudaFuncSetAttribute(mma_probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return OZK_ERR_CUDA;
  const uint32_t b = (uint32_t)(scale_byte & 0xFF);
  mma_probe_kernel<<<1, 192, smem, st>>>(map_p, map_q, (int)(K / kTileKNibbles), b * 0x01010101u, D,
                                        reinterpret_cast<StatusBlock*>(ws), let_wait_expire ? 16u : 0u);
  return cudaGetLastError() == cudaSuccess ? OZK_OK : OZK_ERR_CUDA;
}

}  // namespace ozk
