// Shared declarations of the ozk library: layouts, parameter blocks, status word.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/ozk.h"

namespace ozk {

// ---- tiling constants ---------------------------------------------------------------
constexpr int kTileRows = 128;       // rows of a limb plane covered by one GEMM tile (either operand)
constexpr int kTileKNibbles = 256;   // k extent of one pipeline stage: 256 E2M1 nibbles = 128 bytes
constexpr int kTileKBytes = 128;
constexpr int kMaxModuli = OZK_MAX_MODULI;
constexpr int kCrtWords = 6;         // 192-bit integers cover sum r_l w_l for all 27 moduli
// Encoder tables in the workspace (rebuilt by a small kernel at every call):
//   limb-pair tables   per modulus two byte tables of kLimbTabStride entries indexed by (residue + 2^62) mod m: the
//                      E2M1 codes of a limb pair (c0, c1), c0 + 13 c1 = residue (mod m), as code(c0) | code(c1) << 4 for
//                      elements at even k and code(c1) | code(c0) << 4 for elements at odd k
//   B fragments        of the encoder's mma.sync (kEncTiles tiles of two moduli, 32 lanes, two registers)
//   sum-limb tables    indexed by an even-k limb-pair byte: the code of c0 + c1 in the low nibble / in the high nibble
//   gamma tables       like the limb-pair tables, for the residue class 13 * residue (two-accumulator form)
constexpr int kLimbTabStride = 176;  // >= 169, a multiple of 16
constexpr int kEncTiles = (kMaxModuli + 1) / 2;
constexpr size_t kLimbTabBytes = (size_t)kMaxModuli * 2 * kLimbTabStride;
constexpr size_t kEncFragBytes = (size_t)kEncTiles * 32 * 2 * sizeof(uint32_t);
constexpr size_t kEncSumTabBytes = 2 * 256;   // limb-pair byte -> E2M1 code of c0 + c1 (low nibble / high nibble): Karatsuba variant
constexpr size_t kEncTableBytes = kLimbTabBytes + kEncFragBytes + kEncSumTabBytes + kLimbTabBytes;   // last: gamma tables
constexpr int64_t kChunkK = OZK_CHUNK_K;  // longest k range of one limb-GEMM launch: 128 K <= 2^24 keeps FP32 sums exact (|limb| <= 8)
constexpr int64_t kMaxK = OZK_MAX_K;      // 16 ranges; the grid limits of the O(N^2) kernels lie beyond it

// ---- status word (first bytes of the workspace) -------------------------------------
struct StatusBlock {
  int code;          // 0, OZK_ERR_NONFINITE or OZK_ERR_DEVICE_TIMEOUT (first writer wins on severity)
  int where;         // which wait gave up (role * 256 + barrier id), for diagnostics
  // measurement aid (written only while stage timing is enabled): clocks of the limb GEMM's issuing thread in the
  // first CTA pair, in total and spent waiting for free tensor memory / for operand stages
  long long mma_clk_total, mma_clk_wait_tmem, mma_clk_wait_operands;
  int pad[56];
};
static_assert(sizeof(StatusBlock) == 256, "the wave counter of the limb GEMM sits at byte 512 of the same kibibyte");

// ---- problem geometry ---------------------------------------------------------------
struct Geometry {
  int64_t M, N, K;
  int64_t Mp, Np, Kp;      // padded to 128 / 128 / 256
  int L;
  int c_bits;
  int karatsuba;           // partial Karatsuba variant (Section 5.1, last paragraph): sum-limb planes after the 2 L regular ones
  int gamma;               // two-accumulator form for short K: the A side also carries the limb planes of 13 a mod m (after its 2 L planes)
  // byte offsets into the workspace
  size_t off_status, off_lut, off_amax_a, off_amax_b, off_s, off_t, off_planes_a, off_planes_b, off_res;
  size_t off_res_chunk;                  // second set of residue matrices, present when K > kChunkK (else 0)
  size_t pitch;                          // bytes from one plane row to the next: Kp / 2 plus padding
  size_t plane_bytes_a, plane_bytes_b;   // one limb plane: rows_p * pitch
  size_t total;
};

static inline int64_t round_up(int64_t x, int64_t m) { return (x + m - 1) / m * m; }

// Partial Karatsuba (Section 5.1, last paragraph): moduli all of whose residue classes have a limb pair (c0, c1)
// whose sum c0 + c1 is again in S, so that a0 b0, a1 b1 and (a0 + a1)(b0 + b1) replace the four products.  In the
// modulus list these are 83 (index 11) and everything from 73 (index 13) on: the paper's seven among the first 19.
// An exhaustive search (host side, at table build) checks this rule against the list in use.
__host__ __device__ constexpr bool karatsuba_modulus(int l) { return l == 11 || l >= 13; }
__host__ __device__ constexpr int karatsuba_rank(int l) { return l <= 11 ? 0 : l - 12; }   // Karatsuba moduli before index l
__host__ __device__ constexpr int karatsuba_count(int L) { return L <= 11 ? 0 : (L <= 13 ? 1 : L - 12); }
// Longest k range of one limb-GEMM launch with the variant on: sum limbs reach 12, 144 K <= 2^24 (Lemma 3)
constexpr int64_t kChunkKKaratsuba = 65536;
// Planes per operand: two per modulus, plus one sum-limb plane per Karatsuba modulus when the variant is on
static inline int planes_per_operand(int L, int karatsuba) { return 2 * L + (karatsuba ? karatsuba_count(L) : 0); }
// Two-accumulator form of the residue product (used for short K, where the turn-around between tiles weighs most):
//   a b = a0 beta + a1 gamma (mod m),  beta = b mod m,  gamma = 13 b mod m,  each in two limbs, so that
//   D_lo = a0 beta0 + a1 gamma0,  D_hi = a0 beta1 + a1 gamma1,  r = (D_lo + 13 D_hi) mod m
// needs two accumulators of W columns instead of three; with W = 120 two sets fit tensor memory and the read-back of one
// tile overlaps the products of the next.  The A-matrix side carries beta (its regular planes) and gamma (2 L more).
constexpr int kGammaTileW = 120;
constexpr int64_t kGammaMaxK = 1792;   // longest K that takes this form: measured faster up to here, level at 2048, slower beyond (more operand traffic)
static inline int planes_of_a(int L, int karatsuba, int gamma) { return planes_per_operand(L, karatsuba) + (gamma ? 2 * L : 0); }

// ---- per-modulus constants handed to kernels by value --------------------------------
struct ModulusTable {
  int L;
  int m[kMaxModuli];
  uint32_t recip[kMaxModuli];      // floor(2^32 / m)
  // encoder constants: the residue of a converted integer a is taken from the bytes b_p of a + 2^62 (non-negative) as
  //   t = sum_p b_p c8[p] < 2^19,  t = a + 2^62 (mod m);   t mod m = t - mulhi(t, floor(2^32 / m) + 1) m
  // (the limb-pair tables are indexed by t mod m, i.e. shifted by 2^62 mod m)
  uint8_t c8[kMaxModuli][8];       // 2^(8 p) mod m
  int off62[kMaxModuli];           // 2^62 mod m
};

struct CrtTable {
  int L;
  int words;                               // 32-bit words needed for S = sum r_l w_l
  int m[kMaxModuli];
  uint32_t w[kMaxModuli][kCrtWords];       // w_l little endian
  uint32_t P[kCrtWords];
  uint32_t halfP[kCrtWords];               // floor(P / 2)
  uint32_t negP[5];                        // 2^128 - P for P < 2^128 (four words), else 2^160 - P (five words)
  double inv_P;                            // 1 / P rounded to double
  int p_bits;                              // bit length of P
  // Integer quotient estimate of the carry-chain tails (P of at least 2^100, at most 2047 for floor(S / P)):
  // top = floor(S / 2^q_shift) < 2^32 with q_shift = p_bits - 21 = 32 q_word + q_bit, and
  // q_mul = floor(2^(52 + q_shift) / P * (1 - 2^-28)) < 2^32; (top * q_mul) >> 52 is floor(S / P) or one less.
  uint32_t q_mul;
  int q_word, q_bit;
  // B fragments of the reconstruction kernel's mma.sync.m16n8k32 (u8): tile, lane, register.  Lane (g, q) holds
  // column g of the tile; byte n of register 0 / 1 is the digit for modulus q + 4 n / q + 16 + 4 n.  Column c
  // of tile 0 carries digit (byte) 4 (c / 2) + c % 2 of the weights, of tile 1 digit 4 (c / 2) + 2 + c % 2, of
  // tile 2 digit 16 + c.
  uint32_t bfrag[3][32][2];
};

// per-device facts, cached per device ordinal (ozk_api.cu)
int device_sm_count();      // multiprocessors of the current device (0 on error)
bool device_is_sm100();     // compute capability 10.x
bool stage_timing_enabled();  // ozk_stage_timing_enable state (ozk_api.cu)

// registered workspace and layout (ozk_api.cu)
uint8_t* workspace_ptr();
size_t workspace_bytes();
bool make_geometry(int64_t M, int64_t N, int64_t K, int L, Geometry* g, int max_bits = 53);

// host-side constant builders (ozk_tables.cu)
int host_select_moduli(int count, int* out);
int host_capacity_bits(int64_t K, int L, int max_bits = 53);
bool host_build_modulus_table(int L, ModulusTable* t);
bool host_build_crt_table(int L, CrtTable* t);

// kernels' launchers (each returns cudaError_t of the launch)
cudaError_t launch_build_lut(const ModulusTable& mt, uint8_t* lut, int karatsuba, cudaStream_t st);
bool karatsuba_enabled();   // process-wide switch of the variant (ozk_api.cu)
bool gamma_form_enabled();  // two-accumulator form for short K (on unless OZK_GEMM_GAMMA=0: a measurement aid)
cudaError_t launch_scan_operand(const Geometry& g, int which, const double* X, int64_t ldx, uint8_t* ws, cudaStream_t st);
cudaError_t launch_encode_operand(const Geometry& g, const ModulusTable& mt, int which, const double* X, int64_t ldx,
                                  uint8_t* ws, int64_t* int_out, cudaStream_t st);
cudaError_t launch_scan_and_shifts(const Geometry& g, const double* A, int64_t lda, const double* B, int64_t ldb,
                                   uint8_t* ws, cudaStream_t st);
cudaError_t launch_encode(const Geometry& g, const ModulusTable& mt, const double* A, int64_t lda, const double* B,
                          int64_t ldb, uint8_t* ws, int64_t* At_out, int64_t* Bt_out, cudaStream_t st);
cudaError_t launch_decode_plane(const uint8_t* plane, int64_t rows, int64_t K, size_t pitch, int8_t* out, cudaStream_t st);
cudaError_t launch_crt(const Geometry& g, const CrtTable& ct, const uint8_t* res, int64_t res_ld, size_t res_stride,
                       const int32_t* s, const int32_t* t, double* C, int64_t ldc, uint32_t* x_out, cudaStream_t st);
cudaError_t launch_copy_residues(const Geometry& g, const uint8_t* res, uint8_t* out, cudaStream_t st);
cudaError_t launch_add_residues(const Geometry& g, const ModulusTable& mt, uint8_t* acc, const uint8_t* chunk, cudaStream_t st);

// limb GEMM (ozk_gemm.cu)
ozk_status gemm_residues(const Geometry& g, const ModulusTable& mt, uint8_t* ws, cudaStream_t st, int64_t k0 = 0,
                         int64_t klen = 0, uint8_t* res = nullptr);
ozk_status gemm_residues_chunked(const Geometry& g, const ModulusTable& mt, uint8_t* ws, cudaStream_t st);
ozk_status gemm_int8(const uint8_t* planes_a, const uint8_t* planes_b, int64_t M, int64_t N, int64_t Mp, int64_t Np, int64_t Kp,
                     int32_t* C, int64_t ldc, StatusBlock* status, cudaStream_t st);
ozk_status gemm_oz1_passes(const uint8_t* planes_a, const uint8_t* planes_b, int64_t Mp, int64_t Np, int64_t Kp, int64_t M,
                           long long* out, int64_t out_ld, StatusBlock* status, cudaStream_t st);
ozk_status gemm_probe(const uint8_t* P, const uint8_t* Q, int64_t K, int scale_byte, float* D, uint8_t* ws, cudaStream_t st,
                      bool let_wait_expire = false);

}  // namespace ozk
