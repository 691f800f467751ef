/*
 * ozk — FP64 GEMM emulated on NVIDIA B200 FP4 tensor cores by Ozaki scheme II on
 * base-13 E2M1 limbs, and bit-exact INT8 GEMM on the same limbs.
 *
 * C ABI.  Every matrix pointer is a DEVICE pointer owned by the caller; matrices are
 * column-major (element (r,c) at ptr[r + c*ld]).  `stream` is a cudaStream_t passed as
 * void* (NULL = the legacy default stream).  Compute calls enqueue work on `stream` and
 * return without synchronising; they allocate no memory.  All scratch lives in ONE
 * caller-owned device workspace registered with ozk_set_workspace(); calls that share
 * the workspace must be ordered by the caller (same stream, or events).
 *
 * Errors.  Argument errors are returned synchronously and enqueue nothing.
 * Data-dependent conditions (a NaN/Inf input, a bounded device wait that expired) are
 * recorded in a status word inside the workspace and reported by
 * ozk_get_async_status(), which synchronises the stream.  After OZK_ERR_NONFINITE or
 * OZK_ERR_DEVICE_TIMEOUT the output matrix is unspecified.
 */
#ifndef OZK_H_
#define OZK_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int ozk_status;
enum {
  OZK_OK = 0,
  OZK_ERR_INVALID_ARG = -1,    /* null pointer, negative size, ld too small, bad alignment */
  OZK_ERR_UNSUPPORTED = -2,    /* num_moduli out of range, K beyond an exactness bound, device is not sm_100 */
  OZK_ERR_WORKSPACE = -3,      /* no workspace registered, or it is too small for this call */
  OZK_ERR_CUDA = -4,           /* a CUDA runtime/driver call failed (launch, tensor-map encode) */
  OZK_ERR_NONFINITE = -5,      /* asynchronous: an input element is NaN or Inf */
  OZK_ERR_DEVICE_TIMEOUT = -6  /* asynchronous: a bounded wait inside a kernel gave up */
};

enum { OZK_MIN_MODULI = 2, OZK_MAX_MODULI = 27, OZK_DEFAULT_MODULI = 19 };
/* Longest k range of one limb-GEMM launch, and the largest K ozk_dgemm accepts (16 ranges). */
enum { OZK_CHUNK_K = 131072, OZK_MAX_K = 2097152 };

/* ---------------------------------------------------------------------------------------
 * Constants of the method (host-side, no GPU needed).
 * ------------------------------------------------------------------------------------- */

/* Section 5.1: the first `num_moduli` moduli chosen greedily in descending order from 169,
 * pairwise coprime, 169 the only multiple of 13, every residue class representable by two
 * limbs c0 + 13 c1 with c0, c1 in S = {0,+-1,+-2,+-3,+-4,+-6,+-8,+-12}.  The first 19 are the
 * list printed in the paper; 20..27 continue the same rule.  Writes num_moduli ints to
 * `out` (host memory); returns num_moduli, or OZK_ERR_INVALID_ARG. */
int ozk_get_moduli(int num_moduli, int* out);

/* Eq. 3 read for a general integer width: the largest c <= 53 with 2*K*2^(2c) < P, P the
 * product of the first num_moduli moduli.  Inputs are converted to integers of at most c
 * bits (Section 4.2).  Returns c >= 1, or OZK_ERR_UNSUPPORTED when no c >= 1 exists, or
 * OZK_ERR_INVALID_ARG. */
int ozk_capacity_bits(int64_t K, int num_moduli);

/* Section 5.2: the CRT constants for the first num_moduli moduli as little-endian 32-bit
 * words, 6 words each: P into P_words[6], w_l = (P/m_l) * ((P/m_l)^-1 mod m_l) into
 * weights[6*l .. 6*l+5] (host memory).  Returns OZK_OK or OZK_ERR_INVALID_ARG. */
ozk_status ozk_get_crt_constants(int num_moduli, uint32_t* P_words, uint32_t* weights);

const char* ozk_status_string(ozk_status status);
const char* ozk_version(void);

/* ---------------------------------------------------------------------------------------
 * Workspace.
 * ------------------------------------------------------------------------------------- */

/* Bytes of device workspace ozk_dgemm(M,N,K,...,num_moduli) needs: status block, limb-pair
 * tables, shifts s (rows of A) and t (columns of B), 2*num_moduli E2M1 limb planes per
 * operand padded to 128 rows x 256 k, and num_moduli residue matrices of one byte per
 * element of the padded C.  For 0 < K <= 1792 with N padding to a multiple of 256 the A side
 * holds two more planes per modulus (the limbs of 13 a mod m, see the two-accumulator form
 * under ozk_stage_residue_gemm); with the Karatsuba variant on, one sum-limb plane per Karatsuba
 * modulus and operand.  The size is therefore not monotonic in K (K = 1792 needs more than K = 2048): a caller that
 * reuses one workspace for several shapes registers the largest of their sizes.  Returns 0 on invalid arguments. */
size_t ozk_dgemm_workspace_bytes(int64_t M, int64_t N, int64_t K, int num_moduli);

/* Bytes of device workspace ozk_igemm_i8(M,N,K,...) needs (3 limb planes per operand). */
size_t ozk_igemm_i8_workspace_bytes(int64_t M, int64_t N, int64_t K);

/* Registers the caller-owned device buffer used by all later compute calls of this
 * process.  `dev_ptr` must be 256-byte aligned (any cudaMalloc / PyTorch allocation is).
 * The library never frees it.  Passing NULL unregisters. */
ozk_status ozk_set_workspace(void* dev_ptr, size_t bytes);

/* Synchronises `stream`, then reads and clears the status word in the workspace.
 * Returns OZK_OK, OZK_ERR_NONFINITE, OZK_ERR_DEVICE_TIMEOUT, OZK_ERR_WORKSPACE or OZK_ERR_CUDA. */
ozk_status ozk_get_async_status(void* stream);

/* ---------------------------------------------------------------------------------------
 * The hot path.
 * ------------------------------------------------------------------------------------- */

/* Emulated DGEMM, C = A*B with every C_ij the exact product of the integer-converted
 * inputs rounded once (Sections 4.2, 5; Fig. 3): shared-exponent conversion of the rows
 * of A and columns of B to integers of ozk_capacity_bits(K, num_moduli) bits, residues
 * mod each modulus as two base-13 E2M1 limbs, four FP4 limb products per modulus on the
 * tensor cores with the residue composed in the epilogue, single-pass integer CRT,
 * inverse scaling, one round-to-nearest-even.
 *   A: M x K, lda >= max(1,M).  B: K x N, ldb >= max(1,K).  C: M x N, ldc >= max(1,M), overwritten.
 *   num_moduli in [OZK_MIN_MODULI, OZK_MAX_MODULI]; 19 keeps all 53 bits for K <= 76549.
 *   One limb-GEMM launch covers at most 131072 values of k (FP32 accumulators stay exact
 *   integers: 128*K <= 2^24 with limbs |c| <= 8; Lemma 3 bounds K by 58254 for limbs up to 12).
 *   EXTENSION, not in the paper (which never splits K): a longer K is cut into such ranges, one
 *   limb-GEMM launch each, and the residues of the ranges are added modulo each modulus (the
 *   residue of a sum is the sum of the residues), up to OZK_MAX_K.  The capacity of
 *   ozk_capacity_bits(K, ...) always refers to the whole K.  M, N, K = 0 are allowed (K = 0
 *   gives C = 0).  M and N are otherwise limited only by the workspace.
 *   The library keeps per-device launch state keyed by the device ordinal, so one process may
 *   use several devices (each call acts on the current device, to which `stream` and all
 *   pointers must belong); the registered workspace and the stage timing are one per process,
 *   and calls from several host threads must be serialised by the caller.
 * Returns OZK_OK once the work is enqueued.  The call only enqueues kernels and memsets on
 * `stream` (no allocation, no synchronisation), so after one eager call, which sets the
 * kernels' attributes, it may be captured into a CUDA graph and replayed. */
ozk_status ozk_dgemm(int64_t M, int64_t N, int64_t K,
                     const double* A, int64_t lda,
                     const double* B, int64_t ldb,
                     double* C, int64_t ldc,
                     int num_moduli, void* stream);

/* EXTENSION, not in the paper: ozk_dgemm with the 53-bit cap on the converted integers
 * (Section 4.2) lifted to max_bits, 1 <= max_bits <= OZK_MAX_EXTENDED_BITS.  Every step is the
 * paper's; only the width is c = min(max_bits, largest c with 2 K 2^(2c) < P) (Eq. 3), so
 * with more than 19 moduli the row / column maximum converts without rounding and smaller
 * entries keep up to max_bits - 53 more bits below it (converted integers are held in 64-bit
 * words).  max_bits = 53 is ozk_dgemm itself.  Same arguments, workspace
 * (ozk_dgemm_workspace_bytes), layout, asynchrony and error behaviour as ozk_dgemm;
 * max_bits out of range -> OZK_ERR_INVALID_ARG.  ozk_capacity_bits_ext returns the width used. */
enum { OZK_MAX_EXTENDED_BITS = 62 };
int ozk_capacity_bits_ext(int64_t K, int num_moduli, int max_bits);
ozk_status ozk_dgemm_ext(int64_t M, int64_t N, int64_t K,
                         const double* A, int64_t lda,
                         const double* B, int64_t ldb,
                         double* C, int64_t ldc,
                         int num_moduli, int max_bits, void* stream);

/* Bit-exact INT8 x INT8 -> INT32 GEMM on FP4 tensor cores (Section 3, last paragraph;
 * Eq. 1 with p = q = 3): every int8 becomes three greedy base-13 limbs, nine limb
 * products are accumulated in five groups i+j = g and combined as sum_g 13^g G_g.
 *   A: M x K int8, B: K x N int8, C: M x N int32, column-major as above.
 *   K <= 87381 (three products of magnitude <= 64 share an FP32 accumulator:
 *   192*K <= 2^24); the int32 result is exact for K <= 131071 anyway. */
ozk_status ozk_igemm_i8(int64_t M, int64_t N, int64_t K,
                        const int8_t* A, int64_t lda,
                        const int8_t* B, int64_t ldb,
                        int32_t* C, int64_t ldc, void* stream);

/* ozk_dgemm for matrices in HOST memory (pinned memory for full speed): same result, same
 * arguments, but A, B and C are host pointers.  C is produced in blocks of 2048 x 2048 (larger
 * when a dimension exceeds 131072); the host-to-device copies of the column blocks of B and the
 * row blocks of A (sent alternately), the three stages, and the device-to-host copies of the
 * finished blocks of C run on three streams and overlap: a block of C is computed as soon as
 * its row block and its column block have arrived (the paper times device-resident data only,
 * Section 6.1).  The call returns once everything is enqueued; `stream` completes when C has
 * arrived in host memory.  The workspace holds the limb planes of A and B, one block of
 * residues, and two staging blocks each for A, B and C.  The first call creates two internal
 * streams and a pool of events.  K <= OZK_CHUNK_K here (OZK_ERR_UNSUPPORTED beyond). */
size_t ozk_dgemm_host_workspace_bytes(int64_t M, int64_t N, int64_t K, int num_moduli);
ozk_status ozk_dgemm_host(int64_t M, int64_t N, int64_t K,
                          const double* A, int64_t lda,
                          const double* B, int64_t ldb,
                          double* C, int64_t ldc,
                          int num_moduli, void* stream);

/* Emulated DGEMM by Ozaki scheme I on the same limbs (Section 4; Fig. 2; Eq. 1; Lemma 2): the
 * integer-converted inputs (c = 53 bits, Section 4.2) are decomposed into p = q = 15 greedy base-13
 * E2M1 limbs, the limb products are aggregated along the anti-diagonals i + j = g, weighted by 13^g
 * in multiword integers, scaled back and rounded once.  The result equals ozk_dgemm with 19 moduli
 * bit for bit (both are the exact product of the same converted integers rounded once, Section 7.1).
 * Arguments and layout as ozk_dgemm.  K <= 87381 (three products of magnitude <= 64 share an FP32
 * accumulator).  Workspace: 15 + 16 limb planes and 20 int64 block values per element of C. */
size_t ozk_dgemm_oz1_workspace_bytes(int64_t M, int64_t N, int64_t K);
ozk_status ozk_dgemm_oz1(int64_t M, int64_t N, int64_t K,
                         const double* A, int64_t lda,
                         const double* B, int64_t ldb,
                         double* C, int64_t ldc, void* stream);

/* ---------------------------------------------------------------------------------------
 * Staged entry points: the same kernels one stage at a time, used by the parity tests.
 * They use the registered workspace exactly as ozk_dgemm does.
 * ------------------------------------------------------------------------------------- */

/* Stage 1 (Section 4.2 + Section 5.1): exponent scan, integer conversion, residues,
 * limb planes.  Optional device outputs (NULL to skip):
 *   s_out[M], t_out[N]          the shifts s_i, t_j (int32)
 *   At_out[M*K], Bt_out[K*N]    the converted integers, column-major with ld = M and K (int64)
 * The limb planes stay in the workspace; ozk_stage_read_planes() copies them out. */
ozk_status ozk_stage_preprocess(int64_t M, int64_t N, int64_t K,
                                const double* A, int64_t lda, const double* B, int64_t ldb,
                                int num_moduli, int32_t* s_out, int32_t* t_out,
                                int64_t* At_out, int64_t* Bt_out, void* stream);

/* Decodes limb plane (modulus index l, limb 0|1) of operand 'A' or 'B' from the workspace
 * into doubled-E2M1 integers (int8, values in S): out[r + k*rows], r < rows (M for 'A',
 * N for 'B'), k < K.  Valid after ozk_stage_preprocess / ozk_dgemm on the same sizes.
 * limb = 2 reads the sum-limb plane of a Karatsuba modulus (variant on, see ozk_stage_set_karatsuba).
 * limb = 3 | 4 (operand 'A' only, sizes that take the two-accumulator form) reads limb 0 | 1 of
 * (13 a) mod m_l, the planes that form multiplies by the high limbs of B. */
ozk_status ozk_stage_read_planes(char operand, int64_t M, int64_t N, int64_t K, int num_moduli,
                                 int l, int limb, int8_t* out, void* stream);

/* Stage 2 (Section 5.1, Section 6.4): the limb GEMM with residue composition, on the
 * planes in the workspace.  residues_out (optional, device): num_moduli matrices of
 * M x N bytes, column-major with ld = M, r_l = (A~ B~) mod m_l in [0, m_l).
 * Two forms of the same residues (bit for bit).  Regular: b = b0 + 13 b1, a = a0 + 13 a1,
 * three accumulators a0 b0, a0 b1 + a1 b0, a1 b1 per tile of C.  Two-accumulator form, taken
 * for 0 < K <= 1792 when N pads to a multiple of 256: a b = b0 beta + b1 gamma (mod m) with
 * beta = a mod m and gamma = 13 a mod m, both as limb pairs, so that only the accumulators
 * b0 beta_0 + b1 gamma_0 and b0 beta_1 + b1 gamma_1 exist and two tiles of C fit tensor memory
 * at once: the read-back of one overlaps the products of the next (faster at short K, level
 * with the regular form at K = 2048 and slower beyond, because the A side moves twice the planes).  OZK_GEMM_GAMMA=0 in the
 * environment keeps the regular form at every K (measurement aid, read once per process). */
ozk_status ozk_stage_residue_gemm(int64_t M, int64_t N, int64_t K, int num_moduli,
                                  uint8_t* residues_out, void* stream);

/* Stage 3 (Section 5.2 + Section 4.2): direct CRT, symmetric representative, inverse
 * scaling, one rounding.  residues_in (optional, device; same layout as residues_out): if
 * given together with s_in[M], t_in[N], the stage runs on them instead of the workspace
 * contents.  x_out (optional, device): the reconstructed integer of every element as
 * 6 little-endian 32-bit words, two's complement, element (i,j) at x_out[6*(i + j*M)]. */
ozk_status ozk_stage_crt(int64_t M, int64_t N, int64_t K, int num_moduli,
                         const uint8_t* residues_in, const int32_t* s_in, const int32_t* t_in,
                         double* C, int64_t ldc, uint32_t* x_out, void* stream);

/* The paper has no counterpart to this entry point.  It is for callers that cannot allocate
 * device memory and so cannot provide the workspace the calls above need: code running under a
 * framework whose allocator owns all device memory and forbids raw cudaMalloc (which synchronises
 * the device), plug-ins inside latency-critical loops, processes that have no free memory left.
 * It computes what stage 1 computes first, the row shifts s_i = c - 1 - e_i of A
 * (c = ozk_capacity_bits(K, num_moduli), Section 4.2), and keeps its only scratch, one 64-bit
 * maximum per row, in a fixed array inside the library image: OZK_NOALLOC_MAX_ROWS rows,
 * 512 KiB, resident on every GPU that loads the library until the process exits.  This call and
 * everything it calls neither allocate nor free memory; the array itself is set up by the CUDA
 * driver when it loads the library's device code, which with lazy loading can be as late as the
 * first call on a device: make that call at start-up (a process with no free device memory gets
 * OZK_ERR_CUDA from it), as advised for stream capture below.  `stream` must belong to the
 * current device.
 *   A: M x K column-major FP64 (device), lda >= M.  s_out: M int32 (device).  An all-zero row
 *   gets 0; a row containing NaN or Inf gets INT32_MIN (there is no status word to report it).
 *   M > OZK_NOALLOC_MAX_ROWS, or K beyond the limits of ozk_dgemm -> OZK_ERR_UNSUPPORTED.
 * The first call on each device looks up the device address of the array (with that device
 * current); make that first call before starting any stream capture.  Every call uses the same
 * array and finds the previous call's contents in it: the rows it needs are cleared on `stream`
 * first, and two calls whose work overlaps on the GPU (different streams, no ordering) race. */
enum { OZK_NOALLOC_MAX_ROWS = 65536 };
ozk_status ozk_row_shifts_noalloc(int64_t M, int64_t K, const double* A, int64_t lda, int num_moduli,
                                  int32_t* s_out, void* stream);

/* Measurement aid (the paper times its stages with CUDA events, Section 6.1): when enabled,
 * ozk_dgemm records four CUDA events on its stream, before stage 1 and after each of the three
 * stages.  Enabling creates the events (a host-side allocation; do it outside timed regions).
 * ozk_stage_timing_read() synchronises on those events and writes the milliseconds of
 * preprocessing, limb GEMM and reconstruction to ms3[0..2] (host), averaged over the ozk_dgemm
 * calls made since enabling or since the previous read (the most recent 64 of them), so that a
 * timed loop need not synchronise between its calls.  No call since then -> OZK_ERR_INVALID_ARG. */
ozk_status ozk_stage_timing_enable(int enable);
ozk_status ozk_stage_timing_read(float* ms3);

/* Variant switch (process-wide, off by default): partial Karatsuba for the moduli whose residue classes all
 * have a limb pair (c0, c1) with c0 + c1 again a doubled E2M1 value: 83, 73, 71, 67, 61, 59, 53 among the
 * first 19 (Section 5.1, last paragraph; Section 6.4).  When on, the encoder writes a third plane of sum limbs
 * for those moduli and the CTA-pair limb GEMM forms a0 b0, a1 b1 and (a0 + a1)(b0 + b1) instead of the four
 * products (68 instead of 75 products at 19 moduli); the residues, hence C, are the same bit for bit.  Sum
 * limbs reach 12, so a limb-GEMM launch covers at most 65536 values of k (144 K <= 2^24, Lemma 3).  The
 * workspace grows by the sum-limb planes: query ozk_dgemm_workspace_bytes after switching.  The paper found
 * the variant slower under kernel fusion; so does this build (measurements in profiles/). */
ozk_status ozk_stage_set_karatsuba(int enable);

/* Measurement aid: while stage timing is enabled, the thread that issues the tensor-core
 * instructions of the limb GEMM's first CTA pair counts its clocks (clock64): clk3[0] the whole
 * kernel, clk3[1] waiting for tensor memory to be drained by the epilogue, clk3[2] waiting for
 * operand stages from the TMA producer; the rest it spent issuing.  Reads the counters the most
 * recent limb-GEMM launch left in the workspace (synchronise its stream first); host pointer. */
ozk_status ozk_stage_gemm_cycles(long long* clk3);

/* One tcgen05.mma.kind::mxf4.block_scale instruction sequence on caller-supplied packed
 * E2M1 operands, used to pin the hardware byte formats (nibble order, E2M1 codes, UE8M0
 * scale byte, FP32 accumulator exactness): D[128 x 128] (FP32, row-major, device) =
 * scale^2 * sum_k P[r,k] Q[c,k], P and Q being 128 x K nibbles, K-contiguous, two per byte,
 * K a multiple of 256.  scale_byte is the UE8M0 byte given to every block of both operands. */
ozk_status ozk_stage_mma_probe(const uint8_t* P, const uint8_t* Q, int64_t K, int scale_byte,
                               float* D, void* stream);

/* Test aid for the bounded waits (every wait on a barrier or counter inside the kernels gives up after two
 * seconds, records OZK_ERR_DEVICE_TIMEOUT in the status word and lets the kernel free its tensor memory
 * and return): launches the probe kernel above on zero operands held in the workspace with a barrier
 * that expects 16 bytes nobody sends, so that its wait runs out.  Afterwards ozk_get_async_status
 * returns OZK_ERR_DEVICE_TIMEOUT once and the context and the library remain usable.  Needs a
 * registered workspace of at least 192 KiB. */
ozk_status ozk_stage_wait_probe(void* stream);

#ifdef __cplusplus
}
#endif
#endif /* OZK_H_ */
