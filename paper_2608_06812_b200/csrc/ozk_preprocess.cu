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
// Encoder tables (layout in ozk_common.cuh).  Limb pairs: for modulus m and every residue r in [0, m) the E2M1
// codes of a pair (c0, c1) with c0 + 13 c1 = r (mod m), both limbs in S with |c| <= 8; among the valid pairs the one
// with the fewest negative limbs, then the smallest max(|c0|, |c1|), then the smallest |c0| + |c1| is taken.
// The tables are indexed by t = (residue + 2^62) mod m, the value the encoder's contraction yields.
// Block l < L writes the two byte tables of modulus l; block L writes the B fragments of the encoder's MMA.
// ------------------------------------------------------------------------------------
__global__ void build_lut_kernel(ModulusTable mt, uint8_t* __restrict__ tables, int karatsuba) {
  const int l = blockIdx.x;
  if (l == mt.L) {
    // sum-limb tables of the Karatsuba variant: the limb-pair byte of an even-k element (code(c0) | code(c1) << 4)
    // gives the code of c0 + c1, in the low nibble (first table) and in the high nibble (second table)
    {
      uint8_t* sum_tab = tables + kLimbTabBytes + kEncFragBytes;
      const int x = threadIdx.x;  // 256 threads
      const int i0 = x & 15, i1 = x >> 4;
      const int c0 = kDoubledE2M1[i0 & 7] * ((i0 & 8) ? -1 : 1), c1 = kDoubledE2M1[i1 & 7] * ((i1 & 8) ? -1 : 1);
      const int sum = c0 + c1;
      int code = 0;  // pairs whose sum is not in S never occur in a Karatsuba table
      for (int i = 0; i < 16; ++i)
        if (i != 8 && kDoubledE2M1[i & 7] * ((i & 8) ? -1 : 1) == sum) code = i;
      sum_tab[x] = (uint8_t)code;
      sum_tab[256 + x] = (uint8_t)(code << 4);
    }
    // B fragments (m16n8k32, u8 x u8): tile T holds the moduli 2 T and 2 T + 1.  Column n of a tile belongs to
    // lane n / 2 of every quad and to modulus 2 T + n % 2: it is non-zero only in the k slots of that lane (bytes 0..3
    // of its element in slots 4 q .. 4 q + 3, bytes 4..7 in slots 16 + 4 q ..), where it holds 2^(8 p) mod m.
    // Lane (g, q) stores column g of the tile: register 0 = its slots 4 q .., register 1 = slots 16 + 4 q ...
    uint32_t* frag = reinterpret_cast<uint32_t*>(tables + kLimbTabBytes);
    for (int x = threadIdx.x; x < kEncTiles * 32; x += blockDim.x) {
      const int T = x >> 5, lane = x & 31, g = lane >> 2, q = lane & 3;
      const int mod = 2 * T + (g & 1);
      uint32_t r0 = 0, r1 = 0;
      if ((g >> 1) == q && mod < mt.L) {
        for (int p = 0; p < 4; ++p) {
          r0 |= (uint32_t)mt.c8[mod][p] << (8 * p);
          r1 |= (uint32_t)mt.c8[mod][4 + p] << (8 * p);
        }
      }
      frag[2 * x] = r0;
      frag[2 * x + 1] = r1;
    }
    return;
  }
  // one thread per candidate pair (c0, c1): the best pair of every residue class by an atomic minimum on
  // key * 256 + pair id (equal keys: the smaller id, i.e. the smaller code of c1, then of c0)
  __shared__ unsigned int best[kLimbTabStride];
  const int m = mt.m[l];
  for (int idx = threadIdx.x; idx < kLimbTabStride; idx += blockDim.x) best[idx] = 0xFFFFFFFFu;
  __syncthreads();
  {
    const int i1 = threadIdx.x >> 4, i0 = threadIdx.x & 15;
    if (i0 != 8 && i1 != 8) {  // skip the negative-zero codes
      const int c0 = kDoubledE2M1[i0 & 7] * ((i0 & 8) ? -1 : 1);
      const int c1 = kDoubledE2M1[i1 & 7] * ((i1 & 8) ? -1 : 1);
      const int a0 = abs(c0), a1 = abs(c1);
      bool admissible = max(a0, a1) <= 8;  // every class of every modulus has a pair with |c| <= 8 (keeps 128 K <= 2^24)
      if (karatsuba && karatsuba_modulus(l)) {  // the sum limb must be representable as well (Section 5.1, last paragraph)
        const int sa = abs(c0 + c1);
        admissible = admissible && (sa <= 4 || sa == 6 || sa == 8 || sa == 12);
      }
      if (admissible) {
        // fewest negative limbs first (sign changes in the operand streams cost power on the tensor pipe:
        // a few per cent of the limb GEMM's time under the power cap), then smallest magnitudes
        const int key = 2000 * ((c0 < 0) + (c1 < 0)) + max(a0, a1) * 64 + (a0 + a1);
        const int rho = ((c0 + 13 * c1) % m + m) % m;
        atomicMin(&best[rho], (unsigned int)key * 256u + (unsigned int)threadIdx.x);
      }
    }
  }
  __syncthreads();
  // the tables are indexed by the shifted residue idx = (rho + 2^62) mod m; the gamma tables hold the pair of 13 rho
  uint8_t* even = tables + (size_t)l * 2 * kLimbTabStride;
  uint8_t* odd = even + kLimbTabStride;
  uint8_t* even_g = tables + kLimbTabBytes + kEncFragBytes + kEncSumTabBytes + (size_t)l * 2 * kLimbTabStride;
  uint8_t* odd_g = even_g + kLimbTabStride;
  for (int idx = threadIdx.x; idx < kLimbTabStride; idx += blockDim.x) {
    const int rho = idx < m ? (idx - mt.off62[l] + m) % m : 0;
    const unsigned int pair = idx < m ? best[rho] & 0xFFu : 0u, pair_g = idx < m ? best[(13 * rho) % m] & 0xFFu : 0u;
    even[idx] = (uint8_t)((pair & 15u) | ((pair >> 4) << 4));
    odd[idx] = (uint8_t)((pair >> 4) | ((pair & 15u) << 4));
    even_g[idx] = (uint8_t)((pair_g & 15u) | ((pair_g >> 4) << 4));
    odd_g[idx] = (uint8_t)((pair_g >> 4) | ((pair_g & 15u) << 4));
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

// The same for both operands in one launch: the maxima of A's rows and of B's columns lie back to back (Mp, then Np
// entries).
__global__ void finalize_shifts_pair_kernel(const unsigned long long* __restrict__ amax, int64_t m, int64_t m_pad, int64_t n, int64_t n_pad,
                                            int c_bits, int32_t* __restrict__ shifts_a, int32_t* __restrict__ shifts_b,
                                            StatusBlock* __restrict__ status) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= m_pad + n_pad) return;
  const bool live = i < m_pad ? i < m : i - m_pad < n;
  int32_t s = 0;
  if (live) {
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
  if (i < m_pad) shifts_a[i] = s; else shifts_b[i - m_pad] = s;
}

// ------------------------------------------------------------------------------------
// Residues and limb codes of eight consecutive-k integers per thread, all moduli (Section 5.1), with the
// residue contraction on the tensor cores.
//
// The converted integer a (|a| <= 2^62) is shifted to v = a + 2^62 >= 0, whose eight bytes b_p give
//   t_l = sum_p b_p (2^(8 p) mod m_l)  =  a + 2^62  (mod m_l),   0 <= t_l < 2^19:
// an [elements x 8 bytes] by [8 bytes x moduli] product of bytes, run as mma.sync.m16n8k32 (u8 x u8 -> s32).
// The two 32-bit halves of v ARE the A fragments: a lane puts the halves of two of its elements into its own k
// slots of MMA rows g and g + 8, and the B fragments are block-sparse (a column answers only to the k slots of
// the lane that will read it, see build_lut_kernel), so the accumulators a lane gets back belong to its own
// elements: no data crosses lanes.  One MMA yields 2 elements x 2 moduli per lane; a tile of two moduli takes
// four MMAs for the thread's eight elements.  Then per element and modulus: t mod m = t - mulhi(t, recip1) m,
// one byte read from the limb-pair table, which is indexed by that shifted residue (byte tables keep a warp's 32
// reads within 32 to 43 words: almost no bank conflicts), and the nibbles of eight elements are merged into the
// two 32-bit plane words with byte permutes and three logic operations.
// ------------------------------------------------------------------------------------
__device__ __forceinline__ void mma_u8u8_16832(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                               uint32_t b1) {
  asm("mma.sync.aligned.m16n8k32.row.col.s32.u8.u8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
      : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "r"(0));
}

// v = (converted integer) + 2^62 of the thread's eight elements, as low and high words
struct Shifted8 {
  uint32_t lo[8], hi[8];
};
__device__ __forceinline__ void shift8(const long long (&a)[8], Shifted8& v) {
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    const unsigned long long x = (unsigned long long)a[e] + (1ull << 62);
    v.lo[e] = (uint32_t)x;
    v.hi[e] = (uint32_t)(x >> 32);
  }
}

// The moduli as compile-time constants: the loop over the moduli below is fully unrolled, so that the modulus, its
// reciprocal and the shared-memory address of its table are immediates of the three instructions per element and
// modulus.  This is the list the selection rule of Section 5.1 produces (169 first, then descending, pairwise
// coprime, two-limb representable); the launcher checks it against the host's own search before every launch.
__host__ __device__ constexpr int enc_modulus(int l) {
  constexpr int kList[kMaxModuli + 1] = {169, 115, 113, 112, 111, 109, 107, 103, 101, 97, 89, 83, 79, 73,
                                         71,  67,  61,  59,  53,  47,  43,  41,  31,  29, 19, 17, 11, 1};
  return kList[l < kMaxModuli ? l : kMaxModuli];
}
bool enc_moduli_match(const ModulusTable& mt) {
  for (int l = 0; l < mt.L; ++l)
    if (mt.m[l] != enc_modulus(l)) return false;
  return true;
}

// Shared-memory copy of the encoder tables (static arrays of the calling kernel: their addresses are compile-time
// constants): limb-pair byte tables of the first L moduli and the B fragments.
struct EncTables {
  uint8_t limb[kMaxModuli][2][kLimbTabStride];
  uint2 frag[kEncTiles][32];
  uint8_t sum[2][256];
  uint8_t limb_gamma[kMaxModuli][2][kLimbTabStride];   // copied only by the kernels that write gamma planes
};
static_assert(sizeof(EncTables) == kEncTableBytes, "shared copy mirrors the workspace layout");
template <bool kGamma>
__device__ __forceinline__ void load_tables(const uint8_t* __restrict__ tables, int L, EncTables* tab) {
  const int limb_vec = L * 2 * kLimbTabStride / 16, frag_vec = (int)((kEncFragBytes + kEncSumTabBytes) / 16);
  const uint4* src = reinterpret_cast<const uint4*>(tables);
  const uint4* src_frag = reinterpret_cast<const uint4*>(tables + kLimbTabBytes);
  uint4* dst = reinterpret_cast<uint4*>(tab->limb);
  uint4* dst_frag = reinterpret_cast<uint4*>(tab->frag);
  for (int i = threadIdx.x; i < limb_vec; i += blockDim.x) dst[i] = src[i];
  for (int i = threadIdx.x; i < frag_vec; i += blockDim.x) dst_frag[i] = src_frag[i];
  if constexpr (kGamma) {
    const uint4* src_g = reinterpret_cast<const uint4*>(tables + kLimbTabBytes + kEncFragBytes + kEncSumTabBytes);
    uint4* dst_g = reinterpret_cast<uint4*>(tab->limb_gamma);
    for (int i = threadIdx.x; i < limb_vec; i += blockDim.x) dst_g[i] = src_g[i];
  }
}

// Plane words of the thread's eight elements for every modulus, stored at dst + plane * plane_bytes.
// Warp-collective (all 32 lanes must call it).
// kGamma: also the two planes of 13 a mod m per modulus, at plane index 2 L + 2 l + limb (two-accumulator form, A side).
template <bool kKaratsuba, bool kGamma>
__device__ __forceinline__ void encode_planes(const Shifted8& v, int L, const EncTables& tab, uint8_t* dst, size_t plane_bytes) {
  const int lane = threadIdx.x & 31;
#pragma unroll
  for (int T = 0; T < kEncTiles; ++T) {
    if (2 * T >= L) break;
    const uint2 b = tab.frag[T][lane];
    int d[4][4];  // d[h]: elements 2 h (d[h][0], d[h][1]: moduli 2 T, 2 T + 1) and 2 h + 1 (d[h][2], d[h][3])
#pragma unroll
    for (int h = 0; h < 4; ++h) mma_u8u8_16832(d[h], v.lo[2 * h], v.lo[2 * h + 1], v.hi[2 * h], v.hi[2 * h + 1], b.x, b.y);
#pragma unroll
    for (int mm = 0; mm < 2; ++mm) {
      const int l = 2 * T + mm;
      if (l >= kMaxModuli || l >= L) break;  // odd modulus count: the last tile has one modulus only
      const uint32_t m = (uint32_t)enc_modulus(l), recip1 = (uint32_t)(0x100000000ull / (unsigned long long)enc_modulus(l)) + 1u;
      const uint8_t* even = tab.limb[l][0];
      const uint8_t* odd = tab.limb[l][1];
      uint32_t ea[4], eb[4];  // table bytes of the elements at even / odd k
      uint32_t ga[kGamma ? 4 : 1], gb[kGamma ? 4 : 1];
#pragma unroll
      for (int h = 0; h < 4; ++h) {
        const uint32_t t0 = (uint32_t)d[h][mm], t1 = (uint32_t)d[h][2 + mm];
        const uint32_t r0 = t0 - __umulhi(t0, recip1) * m, r1 = t1 - __umulhi(t1, recip1) * m;
        ea[h] = even[r0];
        eb[h] = odd[r1];
        if constexpr (kGamma) {
          ga[h] = tab.limb_gamma[l][0][r0];
          gb[h] = tab.limb_gamma[l][1][r1];
        }
      }
      if constexpr (kGamma) {
        const uint32_t ya = __byte_perm(__byte_perm(ga[0], ga[1], 0x0040), __byte_perm(ga[2], ga[3], 0x0040), 0x5410);
        const uint32_t yb = __byte_perm(__byte_perm(gb[0], gb[1], 0x0040), __byte_perm(gb[2], gb[3], 0x0040), 0x5410);
        *reinterpret_cast<uint32_t*>(dst + (size_t)(2 * L + 2 * l) * plane_bytes) = (ya & 0x0F0F0F0Fu) | (yb & 0xF0F0F0F0u);
        *reinterpret_cast<uint32_t*>(dst + (size_t)(2 * L + 2 * l + 1) * plane_bytes) = ((ya >> 4) & 0x0F0F0F0Fu) | ((yb << 4) & 0xF0F0F0F0u);
      }
      const uint32_t xa = __byte_perm(__byte_perm(ea[0], ea[1], 0x0040), __byte_perm(ea[2], ea[3], 0x0040), 0x5410);
      const uint32_t xb = __byte_perm(__byte_perm(eb[0], eb[1], 0x0040), __byte_perm(eb[2], eb[3], 0x0040), 0x5410);
      // even table: code(c0) | code(c1) << 4, odd table: code(c1) | code(c0) << 4
      *reinterpret_cast<uint32_t*>(dst + (size_t)(2 * l) * plane_bytes) = (xa & 0x0F0F0F0Fu) | (xb & 0xF0F0F0F0u);
      *reinterpret_cast<uint32_t*>(dst + (size_t)(2 * l + 1) * plane_bytes) = ((xa >> 4) & 0x0F0F0F0Fu) | ((xb << 4) & 0xF0F0F0F0u);
      if constexpr (kKaratsuba) {
        if (karatsuba_modulus(l)) {
          // sum-limb plane: code(c0 + c1) from the pair byte (odd-k bytes carry the nibbles swapped: swap them back)
          uint32_t sa[4], sb[4];
#pragma unroll
          for (int h = 0; h < 4; ++h) {
            sa[h] = tab.sum[0][ea[h]];
            sb[h] = tab.sum[1][((eb[h] << 4) | (eb[h] >> 4)) & 0xFFu];
          }
          const uint32_t ya = __byte_perm(__byte_perm(sa[0], sa[1], 0x0040), __byte_perm(sa[2], sa[3], 0x0040), 0x5410);
          const uint32_t yb = __byte_perm(__byte_perm(sb[0], sb[1], 0x0040), __byte_perm(sb[2], sb[3], 0x0040), 0x5410);
          *reinterpret_cast<uint32_t*>(dst + (size_t)(2 * L + karatsuba_rank(l)) * plane_bytes) = ya | yb;
        }
      }
    }
  }
}

// ------------------------------------------------------------------------------------
// B side: plane row = column j of B, source already K-contiguous.
// Block = 256 threads = 2048 consecutive k of one column; thread = 8 consecutive k (a warp = 256 k: whole warps
// lie inside or outside the padded K, which is a multiple of 256).
// ------------------------------------------------------------------------------------
template <bool kKaratsuba>
__global__ void __launch_bounds__(256) encode_cols_kernel(const double* __restrict__ B, int64_t ldb, int64_t N, int64_t K,
                                                          int64_t Kp, int L, const uint8_t* __restrict__ tables,
                                                          const int32_t* __restrict__ shifts, uint8_t* __restrict__ planes,
                                                          size_t plane_bytes, size_t pitch, int64_t* __restrict__ int_out, int reps) {
  __shared__ __align__(16) EncTables tab;
  load_tables<false>(tables, L, &tab);  // copied once per block and reused for `reps` chunks of 2048 k
  __syncthreads();
  const int64_t j = blockIdx.x;
  for (int rep = 0; rep < reps; ++rep) {
    const int64_t k = (((int64_t)blockIdx.y * reps + rep) * blockDim.x + threadIdx.x) * 8;
    if (k >= Kp) return;  // warp-uniform
    long long a[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) a[e] = 0;
    if (j < N && k < K) {
      const ScalePair sc = make_scale(shifts[j]);
      const double* src = B + j * ldb + k;
      if (k + 8 <= K && ((reinterpret_cast<uintptr_t>(src) & 15) == 0)) {
        const double2* s2 = reinterpret_cast<const double2*>(src);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const double2 x = __ldg(s2 + e);
          a[2 * e] = to_integer_rne(x.x, sc);
          a[2 * e + 1] = to_integer_rne(x.y, sc);
        }
      } else {
#pragma unroll
        for (int e = 0; e < 8; ++e)
          if (k + e < K) a[e] = to_integer_rne(__ldg(src + e), sc);
      }
      if (int_out) {
#pragma unroll
        for (int e = 0; e < 8; ++e)
          if (k + e < K) int_out[j * K + k + e] = a[e];
      }
    }
    Shifted8 v;
    shift8(a, v);
    encode_planes<kKaratsuba, false>(v, L, tab, planes + (size_t)j * pitch + (size_t)(k / 2), plane_bytes);
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

template <bool kKaratsuba, bool kGamma>
__global__ void __launch_bounds__(256) encode_rows_kernel(const double* __restrict__ A, int64_t lda, int64_t M, int64_t K,
                                                          int64_t Kp, int L, const uint8_t* __restrict__ tables,
                                                          const int32_t* __restrict__ shifts, uint8_t* __restrict__ planes,
                                                          size_t plane_bytes, size_t pitch, int64_t* __restrict__ int_out, int reps) {
  __shared__ __align__(16) EncTables tab;
  __shared__ double in_s[kRowTile * kRowStride];
  const int t = threadIdx.x;
  const int64_t i0 = (int64_t)blockIdx.x * kRowTile;
  load_tables<kGamma>(tables, L, &tab);  // copied once per block and reused for `reps` tiles along k
  const int r = t >> 4, g = t & 15;  // encode role: row r, k group g
  const int64_t i = i0 + r;
  const ScalePair sc = make_scale(shifts[i]);  // shifts has Mp entries; padded rows hold 0
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
    long long a[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) a[e] = to_integer_rne(in_s[r * kRowStride + g * kGroupStride + e], sc);
    if (int_out && i < M) {
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const int64_t k = k0 + 8 * g + e;
        if (k < K) int_out[i + k * M] = a[e];
      }
    }
    Shifted8 v;
    shift8(a, v);
    encode_planes<kKaratsuba, kGamma>(v, L, tab, planes + (size_t)i * pitch + (size_t)(k0 / 2) + 4 * g, plane_bytes);
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

cudaError_t launch_build_lut(const ModulusTable& mt, uint8_t* lut, int karatsuba, cudaStream_t st) {
  build_lut_kernel<<<mt.L + 1, 256, 0, st>>>(mt, lut, karatsuba);
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

// Both operands: one clearing of the two (adjacent) arrays of maxima, the two scans, one kernel for all shifts.
cudaError_t launch_scan_and_shifts(const Geometry& g, const double* A, int64_t lda, const double* B, int64_t ldb,
                                   uint8_t* ws, cudaStream_t st) {
  auto* status = reinterpret_cast<StatusBlock*>(ws + g.off_status);
  auto* amax_a = reinterpret_cast<unsigned long long*>(ws + g.off_amax_a);
  auto* amax_b = reinterpret_cast<unsigned long long*>(ws + g.off_amax_b);
  if (g.off_amax_b != g.off_amax_a + (size_t)g.Mp * sizeof(unsigned long long)) {  // not laid out back to back: one operand at a time
    cudaError_t e = launch_scan_operand(g, 0, A, lda, ws, st);
    if (e != cudaSuccess) return e;
    return launch_scan_operand(g, 1, B, ldb, ws, st);
  }
  cudaError_t e = cudaMemsetAsync(amax_a, 0, (size_t)(g.Mp + g.Np) * sizeof(unsigned long long), st);
  if (e != cudaSuccess) return e;
  if (g.K > 0) {
    const int kslab_a = 64, kslab_b = 8192;
    scan_rows_kernel<<<dim3((unsigned)((g.M + 255) / 256), (unsigned)((g.K + kslab_a - 1) / kslab_a)), 256, 0, st>>>(A, lda, g.M, g.K, kslab_a,
                                                                                                                  amax_a);
    scan_cols_kernel<<<dim3((unsigned)g.N, (unsigned)((g.K + kslab_b - 1) / kslab_b)), 256, 0, st>>>(B, ldb, g.K, kslab_b, amax_b);
  }
  finalize_shifts_pair_kernel<<<(unsigned)((g.Mp + g.Np + 255) / 256), 256, 0, st>>>(amax_a, g.M, g.Mp, g.N, g.Np, g.c_bits,
                                                                                     reinterpret_cast<int32_t*>(ws + g.off_s),
                                                                                     reinterpret_cast<int32_t*>(ws + g.off_t), status);
  return cudaGetLastError();
}

// Limb planes of A (which = 0, rows of A) or of B (which = 1, columns of B).
cudaError_t launch_encode_operand(const Geometry& g, const ModulusTable& mt, int which, const double* X, int64_t ldx,
                                  uint8_t* ws, int64_t* int_out, cudaStream_t st) {
  const uint8_t* tables = ws + g.off_lut;
  if (!enc_moduli_match(mt)) return cudaErrorInvalidValue;  // the kernels carry the modulus list as constants
  // tiles along k per block: four when there is enough work for several waves of blocks, fewer for small operands
  const int64_t k_units = which == 0 ? g.Kp / kRowTileK : (g.Kp + 2047) / 2048;
  const int64_t row_units = which == 0 ? g.Mp / kRowTile : g.Np;
  int reps = 4;
  while (reps > 1 && row_units * ((k_units + reps - 1) / reps) < 6 * (int64_t)device_sm_count()) reps >>= 1;
  if (which == 0) {
    dim3 grid((unsigned)(g.Mp / kRowTile), (unsigned)((g.Kp / kRowTileK + reps - 1) / reps));
    auto* kernel = g.karatsuba ? encode_rows_kernel<true, false> : (g.gamma ? encode_rows_kernel<false, true> : encode_rows_kernel<false, false>);
    kernel<<<grid, 256, 0, st>>>(X, ldx, g.M, g.K, g.Kp, mt.L, tables, reinterpret_cast<const int32_t*>(ws + g.off_s),
                                             ws + g.off_planes_a, g.plane_bytes_a, g.pitch, int_out, reps);
  } else {
    dim3 grid((unsigned)g.Np, (unsigned)(((g.Kp + 2047) / 2048 + reps - 1) / reps));
    auto* kernel = g.karatsuba ? encode_cols_kernel<true> : encode_cols_kernel<false>;
    kernel<<<grid, 256, 0, st>>>(X, ldx, g.N, g.K, g.Kp, mt.L, tables, reinterpret_cast<const int32_t*>(ws + g.off_t),
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
