// Limb GEMM with residue composition in the epilogue (Section 5.1: ab = a0 b0 + 13 (a0 b1 + a1 b0)
// + 13^2 a1 b1 (mod m); Section 6.4: all moduli in one launch, three accumulators per modulus,
// nothing but the residues written to memory; Lemma 3: every FP32 partial sum is an exact integer).
//
// One persistent CTA per SM walks a static list of work items (modulus l, tile of 128 columns
// of C, tile of 128 rows of C).  The tensor-core "row" side (TMEM lanes) holds the B-matrix
// limbs p0, p1 (plane rows = columns j of C) and the "column" side the A-matrix limbs q0, q1
// (plane rows = rows i of C), so a thread of the epilogue owns one j and consecutive i, which is
// the column-major order of the residue matrices and of C.
//
// Per 64-nibble K step two N = 256 instructions do the four limb products:
//     D[  0..255] += p0 * [q0 ; q1]    -> columns   0..127: p0 q0,  128..255: p0 q1
//     D[128..383] += p1 * [q0 ; q1]    -> columns 128..255: p1 q0,  256..383: p1 q1
// so columns 128..255 accumulate the two cross terms of weight 13 in one accumulator.
//
// Warp roles: 0 = TMA producer, 1 = MMA issuer (owns the TMEM allocation), 2..5 = epilogue.
// Every wait is bounded; on expiry the CTA records OZK_ERR_DEVICE_TIMEOUT, drains and returns.
#include "ozk_common.cuh"
#include "ozk_ptx.cuh"

namespace ozk {
namespace {

using namespace ptx;

constexpr int kStages = 3;
constexpr int kOperandTileBytes = kTileRows * kTileKBytes;  // 16 KiB: 128 rows x 128 bytes
constexpr int kStageBytes = 4 * kOperandTileBytes;          // p0, p1, q0, q1
constexpr int kGemmThreads = 192;
constexpr int kTmemCols = 512;
constexpr int kScaleCol = 384;  // scale-factor bytes live in TMEM columns 384..399
constexpr uint64_t kWaitLimitNs = 2000000000ull;

struct GemmParams {
  int L;
  int tiles_p;  // tiles along the columns of C (B-matrix plane rows)
  int tiles_q;  // tiles along the rows of C (A-matrix plane rows)
  int kblocks;  // Kp / 256
  int group;    // rasterisation: this many column tiles share one sweep over the row tiles
  int m[kMaxModuli];
  uint32_t recip[kMaxModuli];   // floor(2^32 / m)
  uint32_t offset[kMaxModuli];  // multiple of m close to 2^31: makes the composed value non-negative
  uint8_t* res;                 // [L][Np][Mp] bytes
  int64_t res_ld;               // Mp
  size_t res_stride;            // Mp * Np
  StatusBlock* status;
  uint32_t scale_word;          // four copies of the UE8M0 scale byte
};

struct __align__(8) GemmShared {
  uint64_t full[kStages];
  uint64_t empty[kStages];
  uint64_t tmem_full;
  uint64_t tmem_empty;
  uint64_t drained;
  uint32_t tmem_base;
  volatile int abort;
};

// Bounded wait on an mbarrier phase.  Returns false after the time limit or when another role
// of this CTA has already given up.
__device__ __forceinline__ bool wait_bounded(uint32_t bar, uint32_t parity, GemmShared* sh, StatusBlock* status, int where) {
  if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = global_timer_ns();
  for (uint32_t it = 1;; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 63u) == 0u) {
      if (sh->abort) return false;
      if (global_timer_ns() - t0 > kWaitLimitNs) {
        sh->abort = 1;
        atomicMin(&status->code, (int)OZK_ERR_DEVICE_TIMEOUT);
        atomicExch(&status->where, where);
        return false;
      }
    }
  }
}

__device__ __forceinline__ void decode_item(const GemmParams& p, int item, int& l, int& tp, int& tq) {
  const int per_mod = p.tiles_p * p.tiles_q;
  l = item / per_mod;
  const int t = item - l * per_mod;
  const int band = p.group * p.tiles_q;
  const int g = t / band;
  const int rem = t - g * band;
  const int gsize = min(p.group, p.tiles_p - g * p.group);
  tq = rem / gsize;
  tp = g * p.group + (rem - tq * gsize);
}

__global__ void __launch_bounds__(kGemmThreads, 1)
residue_gemm_kernel(const __grid_constant__ CUtensorMap map_p, const __grid_constant__ CUtensorMap map_q,
                    const __grid_constant__ GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  // operand stages need 1024-byte alignment (128-byte swizzle atoms)
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  GemmShared* sh = reinterpret_cast<GemmShared*>(tiles + kStages * kStageBytes);
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int total_items = p.L * p.tiles_p * p.tiles_q;

  if (threadIdx.x == 0) {
    prefetch_tensormap(&map_p);
    prefetch_tensormap(&map_q);
    for (int s = 0; s < kStages; ++s) {
      mbar_init(smem_u32(&sh->full[s]), 1);
      mbar_init(smem_u32(&sh->empty[s]), 1);
    }
    mbar_init(smem_u32(&sh->tmem_full), 1);
    mbar_init(smem_u32(&sh->tmem_empty), 4);
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
  if (warp >= 2) {  // constant UE8M0 scale bytes, identical for every row, column and K block
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
      uint32_t armed_parity[kStages];
      bool armed[kStages];
      for (int s = 0; s < kStages; ++s) armed[s] = false, armed_parity[s] = 0;
      bool ok = true;
      for (int item = blockIdx.x; item < total_items && ok; item += gridDim.x) {
        int l, tp, tq;
        decode_item(p, item, l, tp, tq);
        for (int kb = 0; kb < p.kblocks; ++kb) {
          if (!wait_bounded(smem_u32(&sh->empty[stage]), phase ^ 1u, sh, p.status, 0x000 + stage)) {
            ok = false;
            break;
          }
          const uint32_t bar = smem_u32(&sh->full[stage]);
          const uint32_t dst = smem_u32(tiles + stage * kStageBytes);
          mbar_arrive_expect_tx(bar, kStageBytes);
          armed[stage] = true;
          armed_parity[stage] = phase;
          const int x = kb * kTileKBytes;
          tma_load_3d(dst + 0 * kOperandTileBytes, &map_p, bar, x, tp * kTileRows, 2 * l + 0);
          tma_load_3d(dst + 1 * kOperandTileBytes, &map_p, bar, x, tp * kTileRows, 2 * l + 1);
          tma_load_3d(dst + 2 * kOperandTileBytes, &map_q, bar, x, tq * kTileRows, 2 * l + 0);
          tma_load_3d(dst + 3 * kOperandTileBytes, &map_q, bar, x, tq * kTileRows, 2 * l + 1);
          if (++stage == kStages) stage = 0, phase ^= 1u;
        }
      }
      if (sh->abort) {  // let copies already in flight land before the CTA leaves
        for (int s = 0; s < kStages; ++s)
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
      constexpr uint32_t kIdesc128 = idesc_mxf4(128);
      constexpr uint32_t kIdesc256 = idesc_mxf4(256);
      bool ok = true;
      for (int item = blockIdx.x; item < total_items && ok; item += gridDim.x) {
        if (!wait_bounded(smem_u32(&sh->tmem_empty), acc_phase ^ 1u, sh, p.status, 0x100)) break;
        tc_fence_after();
        for (int kb = 0; kb < p.kblocks; ++kb) {
          if (!wait_bounded(smem_u32(&sh->full[stage]), phase, sh, p.status, 0x110 + stage)) {
            ok = false;
            break;
          }
          tc_fence_after();
          const uint32_t base = smem_u32(tiles + stage * kStageBytes);
#pragma unroll
          for (int ks = 0; ks < 4; ++ks) {
            const uint64_t p0 = smem_desc_sw128(base + 0 * kOperandTileBytes + ks * 32);
            const uint64_t p1 = smem_desc_sw128(base + 1 * kOperandTileBytes + ks * 32);
            const uint64_t q0 = smem_desc_sw128(base + 2 * kOperandTileBytes + ks * 32);
            const uint64_t q1 = smem_desc_sw128(base + 3 * kOperandTileBytes + ks * 32);
            if (kb == 0 && ks == 0) {
              // first step of a tile: overwrite instead of accumulate, region by region
              mma_mxf4(tmem + 0, p0, q0, kIdesc128, sf, sf, 0u);
              mma_mxf4(tmem + 128, p0, q1, kIdesc128, sf, sf, 0u);
              mma_mxf4(tmem + 128, p1, q0, kIdesc128, sf, sf, 1u);
              mma_mxf4(tmem + 256, p1, q1, kIdesc128, sf, sf, 0u);
            } else {
              mma_mxf4(tmem + 0, p0, q0, kIdesc256, sf, sf, 1u);    // q0 and q1 are adjacent: 256 rows
              mma_mxf4(tmem + 128, p1, q0, kIdesc256, sf, sf, 1u);
            }
          }
          mma_commit(smem_u32(&sh->empty[stage]));
          if (++stage == kStages) stage = 0, phase ^= 1u;
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
    const uint32_t quad = (uint32_t)(warp & 3);
    const uint32_t lane_base = tmem + ((quad * 32u) << 16);
    uint32_t acc_phase = 0;
    for (int item = blockIdx.x; item < total_items; item += gridDim.x) {
      int l, tp, tq;
      decode_item(p, item, l, tp, tq);
      // the outcome must be warp-uniform: the TMEM loads below are warp-collective
      if (!__all_sync(0xFFFFFFFFu, wait_bounded(smem_u32(&sh->tmem_full), acc_phase, sh, p.status, 0x200 + warp))) break;
      tc_fence_after();
      const uint32_t m = (uint32_t)p.m[l], recip = p.recip[l], offset = p.offset[l];
      const int64_t j = (int64_t)tp * kTileRows + quad * 32 + lane;
      uint8_t* out = p.res + (size_t)l * p.res_stride + (size_t)j * (size_t)p.res_ld + (size_t)tq * kTileRows;
#pragma unroll 1
      for (int c = 0; c < 4; ++c) {
        uint32_t d0[32], d1[32], d2[32];
        tmem_ld_32x32(lane_base + 0 + c * 32, d0);
        tmem_ld_32x32(lane_base + 128 + c * 32, d1);
        tmem_ld_32x32(lane_base + 256 + c * 32, d2);
        tmem_wait_ld();
        uint32_t packed[8];
#pragma unroll
        for (int w = 0; w < 8; ++w) {
          uint32_t word = 0;
#pragma unroll
          for (int b = 0; b < 4; ++b) {
            const int e = 4 * w + b;
            const int v0 = __float2int_rn(__uint_as_float(d0[e]));
            const int v1 = __float2int_rn(__uint_as_float(d1[e]));
            const int v2 = __float2int_rn(__uint_as_float(d2[e]));
            const uint32_t t = (uint32_t)(v0 + 13 * v1 + 169 * v2) + offset;  // non-negative, < 2^32
            uint32_t r = t - __umulhi(t, recip) * m;                          // in [0, 2m)
            r = min(r, r - m);
            word |= r << (8 * b);
          }
          packed[w] = word;
        }
        uint4* dst = reinterpret_cast<uint4*>(out + c * 32);
        dst[0] = make_uint4(packed[0], packed[1], packed[2], packed[3]);
        dst[1] = make_uint4(packed[4], packed[5], packed[6], packed[7]);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&sh->tmem_empty));
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
// Probe: one 128 x 128 tile, serial load -> MMA -> read-back, FP32 accumulators written out.
// Pins the hardware formats (nibble order, E2M1 codes, UE8M0 byte, accumulator exactness).
// ------------------------------------------------------------------------------------
struct ProbeShared {
  uint64_t full;
  uint64_t done;
  uint32_t tmem_base;
  volatile int abort;
};

__global__ void __launch_bounds__(kGemmThreads, 1)
mma_probe_kernel(const __grid_constant__ CUtensorMap map_p, const __grid_constant__ CUtensorMap map_q, int kblocks,
                 uint32_t scale_word, float* __restrict__ D, StatusBlock* status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  ProbeShared* sh = reinterpret_cast<ProbeShared*>(tiles + 2 * kOperandTileBytes);
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
      mbar_arrive_expect_tx(smem_u32(&sh->full), 2 * kOperandTileBytes);
      tma_load_2d(base, &map_p, smem_u32(&sh->full), kb * kTileKBytes, 0);
      tma_load_2d(base + kOperandTileBytes, &map_q, smem_u32(&sh->full), kb * kTileKBytes, 0);
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
        mma_mxf4(tmem, smem_desc_sw128(base + ks * 32), smem_desc_sw128(base + kOperandTileBytes + ks * 32),
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

// Planes of one operand as a (bytes along K, rows, plane) byte tensor; box = 128 bytes x 128 rows.
bool make_plane_map(CUtensorMap* map, const void* base, int64_t k_bytes, int64_t rows, int64_t planes, size_t plane_bytes) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  cuuint64_t dims[3] = {(cuuint64_t)k_bytes, (cuuint64_t)rows, (cuuint64_t)planes};
  cuuint64_t strides[2] = {(cuuint64_t)k_bytes, (cuuint64_t)plane_bytes};
  cuuint32_t box[3] = {(cuuint32_t)kTileKBytes, (cuuint32_t)kTileRows, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  const int rank = planes > 0 ? 3 : 2;
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, rank, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int sm_count() {
  static int n = 0;
  if (!n) {
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
  }
  return n;
}

}  // namespace

ozk_status gemm_residues(const Geometry& g, const ModulusTable& mt, uint8_t* ws, cudaStream_t st) {
  CUtensorMap map_p, map_q;
  if (!make_plane_map(&map_p, ws + g.off_planes_b, g.Kp / 2, g.Np, 2 * g.L, g.plane_bytes_b)) return OZK_ERR_CUDA;
  if (!make_plane_map(&map_q, ws + g.off_planes_a, g.Kp / 2, g.Mp, 2 * g.L, g.plane_bytes_a)) return OZK_ERR_CUDA;
  GemmParams p;
  p.L = g.L;
  p.tiles_p = (int)(g.Np / kTileRows);
  p.tiles_q = (int)(g.Mp / kTileRows);
  p.kblocks = (int)(g.Kp / kTileKNibbles);
  p.group = 16;
  for (int l = 0; l < kMaxModuli; ++l) {
    p.m[l] = mt.m[l];
    p.recip[l] = mt.recip[l];
    p.offset[l] = (uint32_t)mt.m[l] * (uint32_t)(0x80000000u / (uint32_t)mt.m[l]);
  }
  p.res = ws + g.off_res;
  p.res_ld = g.Mp;
  p.res_stride = (size_t)g.Mp * (size_t)g.Np;
  p.status = reinterpret_cast<StatusBlock*>(ws + g.off_status);
  p.scale_word = 0x80808080u;  // UE8M0 byte 0x80 = 2: both operands doubled, accumulators hold integers
  const size_t smem = (size_t)kStages * kStageBytes + sizeof(GemmShared) + 1024;
  static bool attr_set = false;
  if (!attr_set) {
    if (cudaFuncSetAttribute(residue_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return OZK_ERR_CUDA;
    attr_set = true;
  }
  const long long items = (long long)p.L * p.tiles_p * p.tiles_q;
  const int grid = (int)(items < sm_count() ? items : sm_count());
  residue_gemm_kernel<<<grid, kGemmThreads, smem, st>>>(map_p, map_q, p);
  return cudaGetLastError() == cudaSuccess ? OZK_OK : OZK_ERR_CUDA;
}

ozk_status gemm_probe(const uint8_t* P, const uint8_t* Q, int64_t K, int scale_byte, float* D, uint8_t* ws, cudaStream_t st) {
  CUtensorMap map_p, map_q;
  if (!make_plane_map(&map_p, P, K / 2, kTileRows, 0, 0)) return OZK_ERR_CUDA;
  if (!make_plane_map(&map_q, Q, K / 2, kTileRows, 0, 0)) return OZK_ERR_CUDA;
  const size_t smem = 2 * kOperandTileBytes + sizeof(ProbeShared) + 1024;
  if (cudaFuncSetAttribute(mma_probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return OZK_ERR_CUDA;
  const uint32_t b = (uint32_t)(scale_byte & 0xFF);
  mma_probe_kernel<<<1, kGemmThreads, smem, st>>>(map_p, map_q, (int)(K / kTileKNibbles), b * 0x01010101u, D,
                                                 reinterpret_cast<StatusBlock*>(ws));
  return cudaGetLastError() == cudaSuccess ? OZK_OK : OZK_ERR_CUDA;
}

}  // namespace ozk
