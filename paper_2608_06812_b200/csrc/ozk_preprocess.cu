// Preprocessing kernels (Section 4.2 shared-exponent conversion; Section 5.1 residues and
// two-limb encoding; Section 6.2 fused decomposition with K-contiguous write-out).
//
//   build_lut         per modulus, for every centred residue one limb pair (c0, c1) as two E2M1 codes
//   scan_rows/cols    max |.| over the rows of A / the columns of B (exponent scan)
//   finalize_shifts   s_i = c - 1 - e_i, t_j likewise; flags NaN/Inf
//   encode_cols       B-side planes: source is already K-contiguous
//   encode_rows       A-side planes: source is M-contiguous, transposed through shared memory
//
// A limb plane is rows_p x Kp nibbles, K-contiguous, two nibbles per byte, the lower-k element
// in the low nibble.  Plane (l, limb) of an operand starts at (2*l + limb) * plane_bytes.
#include "ozk_common.cuh"
#include "ozk_convert.cuh"

namespace ozk {
namespace {

// Doubled E2M1 magnitudes in code order: code & 7 indexes this table, code & 8 is the sign.
__device__ __constant__ int8_t kDoubledE2M1[8] = {0, 1, 2, 3, 4, 6, 8, 12};

// ------------------------------------------------------------------------------------
// Limb-pair table: for modulus m and every centred residue r in [-96, 96) one 16-bit entry (index
// r + 96) holding the E2M1 codes of a limb pair (c0, c1) with c0 + 13 c1 = r (mod m): code(c0) in bits
// 0..3, code(c1) in bits 8..11.  Both limbs are in S with |c| <= 8; among the valid pairs the one with the
// fewest negative limbs, then the smallest max(|c0|,|c1|), then the smallest |c0|+|c1| is taken.  The encoder's residue is centred (|r| <= m/2 + 2 <= 87), so the sign of the converted
// integer needs no separate handling.
// ------------------------------------------------------------------------------------
__global__ void build_lut_kernel(ModulusTable mt, uint16_t* __restrict__ lut) {
  const int l = blockIdx.x;
  const int m = mt.m[l];
  for (int x = threadIdx.x; x < kLutStride; x += blockDim.x) {
    const int rho = ((x - kLutOffset) % m + m) % m;
    int best_key = 1 << 30, best = 0;
    for (int i1 = 0; i1 < 16; ++i1) {
      for (int i0 = 0; i0 < 16; ++i0) {
        if ((i0 == 8) || (i1 == 8)) continue;  // skip the negative-zero codes
        const int c0 = kDoubledE2M1[i0 & 7] * ((i0 & 8) ? -1 : 1);
        const int c1 = kDoubledE2M1[i1 & 7] * ((i1 & 8) ? -1 : 1);
        if ((c0 + 13 * c1 - rho) % m != 0) continue;
        const int a0 = abs(c0), a1 = abs(c1);
        if (max(a0, a1) > 8) continue;  // every class of every modulus has a pair with |c| <= 8 (keeps 128 K <= 2^24)
        // fewest negative limbs first (sign changes in the operand streams cost power on the tensor pipe:
        // a few per cent of the limb GEMM's time under the power cap), then smallest magnitudes
        const int key = 2000 * ((c0 < 0) + (c1 < 0)) + max(a0, a1) * 64 + (a0 + a1);
        if (key < best_key) {
          best_key = key;
          best = (i1 << 8) | i0;
        }
      }
    }
    lut[l * kLutStride + x] = (uint16_t)best;
  }
}

// ------------------------------------------------------------------------------------
// Exponent scan.  |x| compares like its IEEE bit pattern with the sign cleared.
// ------------------------------------------------------------------------------------
__device__ __forceinline__ unsigned long long abs_bits(double v) {
  return (unsigned long long)__double_as_longlong(v) & 0x7FFFFFFFFFFFFFFFull;
}

// A is M x K column-major: thread = row, loop over a slab of k; loads coalesce along rows.
__global__ void __launch_bounds__(256) scan_rows_kernel(const double* __restrict__ A, int64_t lda, int64_t M, int64_t K,
                                                        int kslab, unsigned long long* __restrict__ amax) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t k0 = (int64_t)blockIdx.y * kslab;
  const int64_t k1 = min(K, k0 + (int64_t)kslab);
  if (i >= M) return;
  unsigned long long best = 0;
  const double* p = A + i + k0 * lda;
  int64_t k = k0;
  for (; k + 8 <= k1; k += 8) {
    unsigned long long b[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) b[u] = abs_bits(__ldg(p + u * lda));
#pragma unroll
    for (int u = 0; u < 8; ++u) best = max(best, b[u]);
    p += 8 * lda;
  }
  for (; k < k1; ++k, p += lda) best = max(best, abs_bits(__ldg(p)));
  if (best) atomicMax(amax + i, best);
}

// B is K x N column-major: block = (column, k slab).  Each thread keeps four independent 16-byte loads in
// flight; the maxima meet by warp shuffles and one shared-memory step, one atomicMax per block.
__global__ void __launch_bounds__(256) scan_cols_kernel(const double* __restrict__ B, int64_t ldb, int64_t K, int kslab,
                                                        unsigned long long* __restrict__ amax) {
  __shared__ unsigned long long warp_best[8];
  const int64_t j = blockIdx.x;
  const int64_t k0 = (int64_t)blockIdx.y * kslab;
  const int64_t k1 = min(K, k0 + (int64_t)kslab);
  const double* col = B + j * ldb;
  unsigned long long best = 0;
  int64_t k = k0;
  if ((reinterpret_cast<uintptr_t>(col + k0) & 15) == 0) {  // kslab is even: every slab of an aligned column is aligned
    const int64_t span = 8 * (int64_t)blockDim.x;           // doubles per step: four double2 per thread
    for (; k + span <= k1; k += span) {
      const double2* p = reinterpret_cast<const double2*>(col + k) + threadIdx.x;
      double2 v[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) v[u] = __ldg(p + u * blockDim.x);
#pragma unroll
      for (int u = 0; u < 4; ++u) best = max(best, max(abs_bits(v[u].x), abs_bits(v[u].y)));
    }
  }
  for (int64_t kk = k + threadIdx.x; kk < k1; kk += blockDim.x) best = max(best, abs_bits(__ldg(col + kk)));
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) best = max(best, __shfl_xor_sync(0xFFFFFFFFu, best, off));
  if ((threadIdx.x & 31) == 0) warp_best[threadIdx.x >> 5] = best;
  __syncthreads();
  if (threadIdx.x == 0) {
#pragma unroll
    for (int w = 1; w < 8; ++w) best = max(best, warp_best[w]);
    if (best) atomicMax(amax + j, best);
  }
}

// e = floor(log2 |x|) from the bit pattern (subnormals included); shift = c - 1 - e; zero -> 0.
__global__ void finalize_shifts_kernel(const unsigned long long* __restrict__ amax, int64_t n, int64_t n_pad, int c_bits,
                                       int32_t* __restrict__ shifts, StatusBlock* __restrict__ status) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n_pad) return;
  int32_t s = 0;
  if (i < n) {
    const unsigned long long b = amax[i];
    if (b != 0) {
      const int E = (int)(b >> 52);
      if (E == 0x7FF) {
        atomicMin(&status->code, (int)OZK_ERR_NONFINITE);
      } else {
        const int e = E ? E - 1023 : (63 - __clzll((long long)b)) - 1074;
        s = c_bits - 1 - e;
      }
    }
  }
  shifts[i] = s;
}

// Eight consecutive-k integers of one plane row as signed 14-bit pieces, held in FP32
// (a = x3 2^42 + x2 2^28 + x1 2^14 + x0, every piece carrying the sign of a).  Integers of up to 56 bits
// need four pieces; kWide adds x4 2^56 for the extended-capacity mode (up to 62 bits).
template <bool kWide>
struct Piece8 {
  float x0[8], x1[8], x2[8], x3[8], x4[kWide ? 8 : 1];
};

template <bool kWide>
__device__ __forceinline__ void split8(const unsigned long long (&mag)[8], const bool (&neg)[8], Piece8<kWide>& p) {
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    const float sgn = neg[e] ? -1.0f : 1.0f;
    p.x0[e] = sgn * (float)(uint32_t)(mag[e] & 0x3FFFull);
    p.x1[e] = sgn * (float)(uint32_t)((mag[e] >> 14) & 0x3FFFull);
    p.x2[e] = sgn * (float)(uint32_t)((mag[e] >> 28) & 0x3FFFull);
    if (kWide) {
      p.x3[e] = sgn * (float)(uint32_t)((mag[e] >> 42) & 0x3FFFull);
      p.x4[e] = sgn * (float)(uint32_t)(mag[e] >> 56);  // <= 2^6
    } else {
      p.x3[e] = sgn * (float)(uint32_t)(mag[e] >> 42);  // < 2^14
    }
  }
}

// Residues of the eight values mod m_l and their limb codes packed as 8 nibbles per limb, on the FP32
// pipe (the integer pipes of this GPU run at half its rate).  All quantities are small exact integers:
//   t = x0 + x1 c14 + x2 c28 + x3 c42 (+ x4 c56)   |t| < 2^22   (c = centred residues of 2^14, 2^28, ...;
//                                                  |c| <= 84: 16383 (1 + 3 * 84) + 63 * 84 < 2^22)
//   q = round(t / m) by the add-2^23 trick,  r = t - q m   centred residue, |r| <= m/2 + 2
//   byte offset of the table entry = 2 (r + 96), read from the low bits of 2 r + 192 + 1.5 * 2^23
// Two neighbouring k share a byte: entry(even k) | entry(odd k) << 4 has the byte of limb 0 in bits
// 0..7 and the byte of limb 1 in bits 8..15.
template <bool kWide>
__device__ __forceinline__ void encode8(const Piece8<kWide>& p, float c14, float c28, float c42, float c56, float inv_m, float m_f,
                                        const uint16_t* __restrict__ lut_l, uint32_t& w0, uint32_t& w1) {
  constexpr float kMagic = 12582912.0f;  // 1.5 * 2^23 (bit pattern 0x4B400000): adding it rounds to an integer in the low mantissa bits
  // shared-memory address of the table minus the bit pattern of the magic constant: one integer add turns the
  // float below into the address of its entry
  const uint32_t delta = (uint32_t)__cvta_generic_to_shared(lut_l) - 0x4B400000u;
  uint32_t pair[4];
#pragma unroll
  for (int h = 0; h < 4; ++h) {
    uint32_t v[2];
#pragma unroll
    for (int o = 0; o < 2; ++o) {
      const int e = 2 * h + o;
      float t = fmaf(p.x3[e], c42, fmaf(p.x2[e], c28, fmaf(p.x1[e], c14, p.x0[e])));
      if (kWide) t = fmaf(p.x4[e], c56, t);
      const float q = fmaf(t, inv_m, kMagic) - kMagic;
      const float r = fmaf(-q, m_f, t);
      const uint32_t addr = __float_as_uint(fmaf(r, 2.0f, kMagic + 2.0f * kLutOffset)) + delta;  // table + 2 (r + 96)
      asm("ld.shared.u16 %0, [%1];" : "=r"(v[o]) : "r"(addr));
    }
    pair[h] = v[1] * 16u + v[0];  // the nibbles do not overlap: one multiply-add instead of shift and or
  }
  const uint32_t t0 = __byte_perm(pair[0], pair[1], 0x5410), t1 = __byte_perm(pair[2], pair[3], 0x5410);
  w0 = __byte_perm(t0, t1, 0x6420);
  w1 = __byte_perm(t0, t1, 0x7531);
}

// ------------------------------------------------------------------------------------
// B side: plane row = column j of B, source already K-contiguous.
// Block = 256 threads = 2048 consecutive k of one column; thread = 8 consecutive k.
// ------------------------------------------------------------------------------------
template <bool kWide>
__global__ void __launch_bounds__(256) encode_cols_kernel(const double* __restrict__ B, int64_t ldb, int64_t N, int64_t K,
                                                          int64_t Kp, ModulusTable mt, const uint16_t* __restrict__ lut,
                                                          const int32_t* __restrict__ shifts, uint8_t* __restrict__ planes,
                                                          size_t plane_bytes, size_t pitch, int64_t* __restrict__ int_out, int reps) {
  extern __shared__ __align__(16) uint16_t lut_s[];
  {  // the table is copied once per block and reused for `reps` chunks of 2048 k
    const uint4* src = reinterpret_cast<const uint4*>(lut);
    uint4* dst = reinterpret_cast<uint4*>(lut_s);
    for (int i = threadIdx.x; i < mt.L * kLutStride / 8; i += blockDim.x) dst[i] = src[i];
  }
  __syncthreads();
  const int64_t j = blockIdx.x;
  for (int rep = 0; rep < reps; ++rep) {
  const int64_t k = (((int64_t)blockIdx.y * reps + rep) * blockDim.x + threadIdx.x) * 8;
  if (k >= Kp) return;
  unsigned long long mag[8];
  bool neg[8];
#pragma unroll
  for (int e = 0; e < 8; ++e) mag[e] = 0, neg[e] = false;
  if (j < N && k < K) {
    const int s = shifts[j];
    const double* src = B + j * ldb + k;
    if (k + 8 <= K && ((reinterpret_cast<uintptr_t>(src) & 15) == 0)) {
      const double2* s2 = reinterpret_cast<const double2*>(src);
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const double2 v = __ldg(s2 + e);
        mag[2 * e] = to_integer_magnitude(v.x, s, &neg[2 * e]);
        mag[2 * e + 1] = to_integer_magnitude(v.y, s, &neg[2 * e + 1]);
      }
    } else {
#pragma unroll
      for (int e = 0; e < 8; ++e)
        if (k + e < K) mag[e] = to_integer_magnitude(__ldg(src + e), s, &neg[e]);
    }
    if (int_out) {
#pragma unroll
      for (int e = 0; e < 8; ++e)
        if (k + e < K) int_out[j * K + k + e] = neg[e] ? -(long long)mag[e] : (long long)mag[e];
    }
  }
  Piece8<kWide> p;
  split8<kWide>(mag, neg, p);
  uint8_t* dst = planes + (size_t)j * pitch + (size_t)(k / 2);
  for (int l = 0; l < mt.L; ++l) {
    uint32_t w0, w1;
    encode8<kWide>(p, mt.c14[l], mt.c28[l], mt.c42[l], mt.c56[l], mt.inv_m[l], mt.m_f[l], lut_s + l * kLutStride, w0, w1);
    *reinterpret_cast<uint32_t*>(dst + (size_t)(2 * l) * plane_bytes) = w0;
    *reinterpret_cast<uint32_t*>(dst + (size_t)(2 * l + 1) * plane_bytes) = w1;
  }
  }
}

// ------------------------------------------------------------------------------------
// A side: plane row = row i of A, source is M-contiguous.  Block = tile of 16 rows x 128 k.
//   load    coalesced along rows (16 rows = 128 contiguous bytes per k) into shared memory, stored
//           [row][group of 8 k][k in group] with odd strides, so that both the row-major writes
//           and the k-major reads below are free of bank conflicts
//   encode  thread = (row, group of 8 k); half a warp = the 16 groups of one row
//   store   straight to the planes: the 16 groups of a row are 64 contiguous bytes per plane
// ------------------------------------------------------------------------------------
constexpr int kRowTile = 16;
constexpr int kRowTileK = 128;
constexpr int kGroupStride = 9;                                         // doubles per group of 8 k (8 used)
constexpr int kRowStride = (kRowTileK / 8) * kGroupStride + 1;          // doubles per row: 145, odd

template <bool kWide>
__global__ void __launch_bounds__(256) encode_rows_kernel(const double* __restrict__ A, int64_t lda, int64_t M, int64_t K,
                                                          int64_t Kp, ModulusTable mt, const uint16_t* __restrict__ lut,
                                                          const int32_t* __restrict__ shifts, uint8_t* __restrict__ planes,
                                                          size_t plane_bytes, size_t pitch, int64_t* __restrict__ int_out, int reps) {
  extern __shared__ __align__(16) uint8_t smem[];
  uint16_t* lut_s = reinterpret_cast<uint16_t*>(smem);                          // L * kLutStride entries
  const int lut_bytes = (mt.L * kLutStride * (int)sizeof(uint16_t) + 15) & ~15;
  double* in_s = reinterpret_cast<double*>(smem + lut_bytes);                    // [16][145] doubles
  const int t = threadIdx.x;
  const int64_t i0 = (int64_t)blockIdx.x * kRowTile;
  {  // the table is copied once per block and reused for `reps` tiles along k
    const uint4* src = reinterpret_cast<const uint4*>(lut);
    uint4* dst = reinterpret_cast<uint4*>(lut_s);
    for (int i = t; i < mt.L * kLutStride / 8; i += blockDim.x) dst[i] = src[i];
  }
  const int r = t >> 4, g = t & 15;  // encode role: row r, k group g
  const int64_t i = i0 + r;
  const int s = shifts[i];           // shifts has Mp entries; padded rows hold 0
  for (int rep = 0; rep < reps; ++rep) {
    const int64_t k0 = ((int64_t)blockIdx.y * reps + rep) * kRowTileK;
    if (k0 >= Kp) break;        // uniform over the block
    if (rep) __syncthreads();   // the previous tile has been read
    {
      const int ti = t & 15, tk = t >> 4;  // load role: row ti, k = tk, tk + 16, ...
      const int64_t il = i0 + ti;
#pragma unroll
      for (int n = 0; n < 8; ++n) {
        const int kk = tk + 16 * n;
        const int64_t k = k0 + kk;
        in_s[ti * kRowStride + (kk >> 3) * kGroupStride + (kk & 7)] = (il < M && k < K) ? __ldg(A + il + k * lda) : 0.0;
      }
    }
    __syncthreads();
    unsigned long long mag[8];
    bool neg[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) mag[e] = to_integer_magnitude(in_s[r * kRowStride + g * kGroupStride + e], s, &neg[e]);
    if (int_out && i < M) {
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const int64_t k = k0 + 8 * g + e;
        if (k < K) int_out[i + k * M] = neg[e] ? -(long long)mag[e] : (long long)mag[e];
      }
    }
    Piece8<kWide> p;
    split8<kWide>(mag, neg, p);
    uint8_t* dst = planes + (size_t)i * pitch + (size_t)(k0 / 2) + 4 * g;
    for (int l = 0; l < mt.L; ++l) {
      uint32_t w0, w1;
      encode8<kWide>(p, mt.c14[l], mt.c28[l], mt.c42[l], mt.c56[l], mt.inv_m[l], mt.m_f[l], lut_s + l * kLutStride, w0, w1);
      *reinterpret_cast<uint32_t*>(dst + (size_t)(2 * l) * plane_bytes) = w0;
      *reinterpret_cast<uint32_t*>(dst + (size_t)(2 * l + 1) * plane_bytes) = w1;
    }
  }
}

// Decodes one limb plane into doubled-E2M1 integers, out[r + k*rows] (test support).
__global__ void decode_plane_kernel(const uint8_t* __restrict__ plane, int64_t rows, int64_t K, size_t pitch,
                                    int8_t* __restrict__ out) {
  const int64_t r = (int64_t)blockIdx.y * blockDim.x + threadIdx.x;
  const int64_t k = blockIdx.x;
  if (r >= rows || k >= K) return;
  const uint8_t byte = plane[(size_t)r * pitch + (size_t)(k / 2)];
  const int code = (k & 1) ? (byte >> 4) : (byte & 0xF);
  const int v = kDoubledE2M1[code & 7];
  out[r + k * rows] = (int8_t)((code & 8) ? -v : v);
}

}  // namespace

cudaError_t launch_build_lut(const ModulusTable& mt, uint8_t* lut, cudaStream_t st) {
  build_lut_kernel<<<mt.L, 192, 0, st>>>(mt, reinterpret_cast<uint16_t*>(lut));
  return cudaGetLastError();
}

// Row shifts s_i of A (which = 0) or column shifts t_j of B (which = 1): maxima, then c - 1 - e.
cudaError_t launch_scan_operand(const Geometry& g, int which, const double* X, int64_t ldx, uint8_t* ws, cudaStream_t st) {
  auto* status = reinterpret_cast<StatusBlock*>(ws + g.off_status);
  if (which == 0) {
    auto* amax = reinterpret_cast<unsigned long long*>(ws + g.off_amax_a);
    cudaError_t e = cudaMemsetAsync(amax, 0, (size_t)g.Mp * sizeof(unsigned long long), st);
    if (e != cudaSuccess) return e;
    if (g.K > 0) {
      const int kslab = 64;
      dim3 grid((unsigned)((g.M + 255) / 256), (unsigned)((g.K + kslab - 1) / kslab));
      scan_rows_kernel<<<grid, 256, 0, st>>>(X, ldx, g.M, g.K, kslab, amax);
    }
    finalize_shifts_kernel<<<(unsigned)((g.Mp + 255) / 256), 256, 0, st>>>(amax, g.M, g.Mp, g.c_bits,
                                                                          reinterpret_cast<int32_t*>(ws + g.off_s), status);
  } else {
    auto* amax = reinterpret_cast<unsigned long long*>(ws + g.off_amax_b);
    cudaError_t e = cudaMemsetAsync(amax, 0, (size_t)g.Np * sizeof(unsigned long long), st);
    if (e != cudaSuccess) return e;
    if (g.K > 0) {
      const int kslab = 8192;
      dim3 grid((unsigned)g.N, (unsigned)((g.K + kslab - 1) / kslab));
      scan_cols_kernel<<<grid, 256, 0, st>>>(X, ldx, g.K, kslab, amax);
    }
    finalize_shifts_kernel<<<(unsigned)((g.Np + 255) / 256), 256, 0, st>>>(amax, g.N, g.Np, g.c_bits,
                                                                          reinterpret_cast<int32_t*>(ws + g.off_t), status);
  }
  return cudaGetLastError();
}

cudaError_t launch_scan_and_shifts(const Geometry& g, const double* A, int64_t lda, const double* B, int64_t ldb,
                                   uint8_t* ws, cudaStream_t st) {
  cudaError_t e = launch_scan_operand(g, 0, A, lda, ws, st);
  if (e != cudaSuccess) return e;
  return launch_scan_operand(g, 1, B, ldb, ws, st);
}

// Limb planes of A (which = 0, rows of A) or of B (which = 1, columns of B).
cudaError_t launch_encode_operand(const Geometry& g, const ModulusTable& mt, int which, const double* X, int64_t ldx,
                                  uint8_t* ws, int64_t* int_out, cudaStream_t st) {
  const uint16_t* lut = reinterpret_cast<const uint16_t*>(ws + g.off_lut);
  const int lut_bytes = (mt.L * kLutStride * (int)sizeof(uint16_t) + 15) & ~15;
  const int reps = 4;
  const bool wide = g.c_bits > 56;  // integers beyond 56 bits take a fifth 14-bit piece
  if (which == 0) {
    const size_t smem = lut_bytes + (size_t)kRowTile * kRowStride * sizeof(double);
    auto* kernel = wide ? encode_rows_kernel<true> : encode_rows_kernel<false>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    dim3 grid((unsigned)(g.Mp / kRowTile), (unsigned)((g.Kp / kRowTileK + reps - 1) / reps));
    kernel<<<grid, 256, smem, st>>>(X, ldx, g.M, g.K, g.Kp, mt, lut, reinterpret_cast<const int32_t*>(ws + g.off_s),
                                    ws + g.off_planes_a, g.plane_bytes_a, g.pitch, int_out, reps);
  } else {
    dim3 grid((unsigned)g.Np, (unsigned)(((g.Kp + 2047) / 2048 + reps - 1) / reps));
    auto* kernel = wide ? encode_cols_kernel<true> : encode_cols_kernel<false>;
    kernel<<<grid, 256, lut_bytes, st>>>(X, ldx, g.N, g.K, g.Kp, mt, lut, reinterpret_cast<const int32_t*>(ws + g.off_t),
                                         ws + g.off_planes_b, g.plane_bytes_b, g.pitch, int_out, reps);
  }
  return cudaGetLastError();
}

cudaError_t launch_encode(const Geometry& g, const ModulusTable& mt, const double* A, int64_t lda, const double* B,
                          int64_t ldb, uint8_t* ws, int64_t* At_out, int64_t* Bt_out, cudaStream_t st) {
  cudaError_t e = launch_encode_operand(g, mt, 0, A, lda, ws, At_out, st);
  if (e != cudaSuccess) return e;
  return launch_encode_operand(g, mt, 1, B, ldb, ws, Bt_out, st);
}

cudaError_t launch_decode_plane(const uint8_t* plane, int64_t rows, int64_t K, size_t pitch, int8_t* out, cudaStream_t st) {
  if (rows == 0 || K == 0) return cudaSuccess;
  dim3 grid((unsigned)K, (unsigned)((rows + 127) / 128));
  decode_plane_kernel<<<grid, 128, 0, st>>>(plane, rows, K, pitch, out);
  return cudaGetLastError();
}

}  // namespace ozk
