// C-ABI entry points of the ozk library: argument checks, workspace layout, stage sequencing.
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <atomic>

#include "ozk_common.cuh"

namespace ozk {
namespace {

struct Workspace {
  uint8_t* ptr = nullptr;
  size_t bytes = 0;
};
Workspace g_ws;

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Stage events of the most recent calls, in a ring: the reader averages over the calls since the
// last read without having synchronised between them.
constexpr int kTimingRing = 64;
struct StageTiming {
  bool enabled = false;
  bool created = false;
  int calls = 0;  // ozk_dgemm calls recorded since enable / the last read
  cudaEvent_t ev[kTimingRing][4];
};
StageTiming g_timing;
bool g_karatsuba = false;

void mark(int i, cudaStream_t st) {
  if (g_timing.enabled) cudaEventRecord(g_timing.ev[g_timing.calls % kTimingRing][i], st);
}

// Workspace layout for an (M, N, K, L) problem.  Returns false on invalid sizes.
bool make_geometry_impl(int64_t M, int64_t N, int64_t K, int L, Geometry* g, int max_bits) {
  if (M < 0 || N < 0 || K < 0 || L < OZK_MIN_MODULI || L > OZK_MAX_MODULI) return false;
  if (max_bits < 1 || max_bits > OZK_MAX_EXTENDED_BITS) return false;
  memset(g, 0, sizeof *g);
  g->M = M;
  g->N = N;
  g->K = K;
  g->L = L;
  g->Mp = round_up(M > 0 ? M : 1, kTileRows);
  g->Np = round_up(N > 0 ? N : 1, kTileRows);
  g->Kp = round_up(K > 0 ? K : 1, kTileKNibbles);
  g->c_bits = host_capacity_bits(K, L, max_bits);
  g->karatsuba = (g_karatsuba && karatsuba_count(L) > 0) ? 1 : 0;
  // short K on CTA pairs: two-accumulator form with gamma planes on the A side
  g->gamma = (!g->karatsuba && gamma_form_enabled() && K > 0 && K <= kGammaMaxK && g->Np % 256 == 0) ? 1 : 0;
  size_t off = 0;
  g->off_status = off;
  off += align_up(sizeof(StatusBlock), 1024);
  g->off_lut = off;
  off += align_up(kEncTableBytes, 1024);
  g->off_amax_a = off;
  off += (size_t)g->Mp * 8;
  g->off_amax_b = off;
  off += (size_t)g->Np * 8;
  off = align_up(off, 1024);
  g->off_s = off;
  off += align_up((size_t)g->Mp * 4, 1024);
  g->off_t = off;
  off += align_up((size_t)g->Np * 4, 1024);
  g->pitch = (size_t)(g->Kp / 2);
  g->plane_bytes_a = (size_t)g->Mp * g->pitch;
  g->plane_bytes_b = (size_t)g->Np * g->pitch;
  g->off_planes_a = off;
  off += (size_t)planes_of_a(L, g->karatsuba, g->gamma) * g->plane_bytes_a;
  g->off_planes_b = off;
  off += (size_t)planes_per_operand(L, g->karatsuba) * g->plane_bytes_b;
  g->off_res = off;
  off += (size_t)L * (size_t)g->Mp * (size_t)g->Np;
  g->off_res_chunk = 0;
  if (K > (g->karatsuba ? kChunkKKaratsuba : kChunkK)) {  // k ranges beyond the first leave their residues here before they are added in
    g->off_res_chunk = off;
    off += (size_t)L * (size_t)g->Mp * (size_t)g->Np;
  }
  g->total = align_up(off, 1024);
  return true;
}

ozk_status check_common(int64_t M, int64_t N, int64_t K, int L, Geometry* g, int max_bits = 53) {
  if (!make_geometry(M, N, K, L, g, max_bits)) return OZK_ERR_INVALID_ARG;
  if (K > kMaxK) return OZK_ERR_UNSUPPORTED;
  if (g->c_bits < 1) return OZK_ERR_UNSUPPORTED;
  if (!g_ws.ptr) return OZK_ERR_WORKSPACE;
  if (g_ws.bytes < g->total) return OZK_ERR_WORKSPACE;
  return OZK_OK;
}

ozk_status run_preprocess(const Geometry& g, const ModulusTable& mt, const double* A, int64_t lda, const double* B,
                          int64_t ldb, int64_t* At_out, int64_t* Bt_out, cudaStream_t st) {
  if (launch_build_lut(mt, g_ws.ptr + g.off_lut, g.karatsuba, st) != cudaSuccess) return OZK_ERR_CUDA;
  if (launch_scan_and_shifts(g, A, lda, B, ldb, g_ws.ptr, st) != cudaSuccess) return OZK_ERR_CUDA;
  if (launch_encode(g, mt, A, lda, B, ldb, g_ws.ptr, At_out, Bt_out, st) != cudaSuccess) return OZK_ERR_CUDA;
  return OZK_OK;
}

}  // namespace

bool make_geometry(int64_t M, int64_t N, int64_t K, int L, Geometry* g, int max_bits) {
  return make_geometry_impl(M, N, K, L, g, max_bits);
}

// Facts about the current device, looked up once per device ordinal (a process may use several devices).
namespace {
constexpr int kMaxDevices = 64;
struct DeviceFacts {
  std::atomic<int> sm_count{-1};
  std::atomic<int> major{-1};
};
DeviceFacts g_device_facts[kMaxDevices];
DeviceFacts* current_device_facts() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  DeviceFacts* f = &g_device_facts[dev];
  if (f->sm_count.load(std::memory_order_acquire) < 0) {
    int n = 0, major = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return nullptr;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return nullptr;
    f->major.store(major, std::memory_order_release);
    f->sm_count.store(n, std::memory_order_release);
  }
  return f;
}
}  // namespace
int device_sm_count() {
  DeviceFacts* f = current_device_facts();
  return f ? f->sm_count.load(std::memory_order_acquire) : 0;
}
bool device_is_sm100() {
  DeviceFacts* f = current_device_facts();
  return f && f->major.load(std::memory_order_acquire) == 10;
}

// Limb GEMM over all of K: one launch per k range of at most kChunkK (the FP32 accumulators stay exact
// integers inside a range, Lemma 3 with |limb| <= 8); the residues of later ranges are added modulo m.
ozk_status gemm_residues_chunked(const Geometry& g, const ModulusTable& mt, uint8_t* ws, cudaStream_t st) {
  const int64_t chunk = g.karatsuba ? kChunkKKaratsuba : kChunkK;
  if (g.Kp <= chunk) return gemm_residues(g, mt, ws, st);
  if (!g.off_res_chunk) return OZK_ERR_WORKSPACE;
  for (int64_t k0 = 0; k0 < g.Kp; k0 += chunk) {
    const int64_t klen = g.Kp - k0 < chunk ? g.Kp - k0 : chunk;
    const ozk_status rc = gemm_residues(g, mt, ws, st, k0, klen, k0 == 0 ? nullptr : ws + g.off_res_chunk);
    if (rc != OZK_OK) return rc;
    if (k0 > 0 && launch_add_residues(g, mt, ws + g.off_res, ws + g.off_res_chunk, st) != cudaSuccess) return OZK_ERR_CUDA;
  }
  return OZK_OK;
}
bool karatsuba_enabled() { return g_karatsuba; }
bool gamma_form_enabled() {
  static int v = -1;
  if (v < 0) {
    const char* e = getenv("OZK_GEMM_GAMMA");
    v = (e && e[0] == '0') ? 0 : 1;
  }
  return v == 1;
}
bool stage_timing_enabled() { return g_timing.enabled; }
uint8_t* workspace_ptr() { return g_ws.ptr; }
size_t workspace_bytes() { return g_ws.bytes; }

}  // namespace ozk

using namespace ozk;

extern "C" {

int ozk_get_moduli(int num_moduli, int* out) {
  if (!out || num_moduli < 1 || num_moduli > OZK_MAX_MODULI) return OZK_ERR_INVALID_ARG;
  return host_select_moduli(num_moduli, out) == num_moduli ? num_moduli : OZK_ERR_INVALID_ARG;
}

int ozk_capacity_bits_ext(int64_t K, int num_moduli, int max_bits) {
  if (K < 0 || num_moduli < 1 || num_moduli > OZK_MAX_MODULI || max_bits < 1 || max_bits > OZK_MAX_EXTENDED_BITS)
    return OZK_ERR_INVALID_ARG;
  const int c = host_capacity_bits(K, num_moduli, max_bits);
  return c >= 1 ? c : OZK_ERR_UNSUPPORTED;
}

int ozk_capacity_bits(int64_t K, int num_moduli) { return ozk_capacity_bits_ext(K, num_moduli, 53); }

ozk_status ozk_get_crt_constants(int num_moduli, uint32_t* P_words, uint32_t* weights) {
  CrtTable ct;
  if (!P_words || !weights || !host_build_crt_table(num_moduli, &ct)) return OZK_ERR_INVALID_ARG;
  memcpy(P_words, ct.P, sizeof ct.P);
  for (int l = 0; l < num_moduli; ++l) memcpy(weights + kCrtWords * l, ct.w[l], sizeof ct.w[l]);
  return OZK_OK;
}

const char* ozk_status_string(ozk_status s) {
  switch (s) {
    case OZK_OK: return "ok";
    case OZK_ERR_INVALID_ARG: return "invalid argument";
    case OZK_ERR_UNSUPPORTED: return "unsupported size, modulus count or device";
    case OZK_ERR_WORKSPACE: return "workspace missing or too small";
    case OZK_ERR_CUDA: return "CUDA call failed";
    case OZK_ERR_NONFINITE: return "non-finite input element";
    case OZK_ERR_DEVICE_TIMEOUT: return "bounded device wait expired";
    default: return "unknown status";
  }
}

const char* ozk_version(void) { return "ozk 0.1 (sm_100a)"; }

size_t ozk_dgemm_workspace_bytes(int64_t M, int64_t N, int64_t K, int num_moduli) {
  Geometry g;
  return make_geometry(M, N, K, num_moduli, &g) ? g.total : 0;
}

ozk_status ozk_set_workspace(void* dev_ptr, size_t bytes) {
  if (dev_ptr && (reinterpret_cast<uintptr_t>(dev_ptr) & 255)) return OZK_ERR_INVALID_ARG;
  g_ws.ptr = static_cast<uint8_t*>(dev_ptr);
  g_ws.bytes = dev_ptr ? bytes : 0;
  if (dev_ptr) {
    if (bytes < sizeof(StatusBlock)) return OZK_ERR_WORKSPACE;
    if (cudaMemset(dev_ptr, 0, sizeof(StatusBlock)) != cudaSuccess) return OZK_ERR_CUDA;
  }
  return OZK_OK;
}

ozk_status ozk_get_async_status(void* stream) {
  if (!g_ws.ptr) return OZK_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cudaStreamSynchronize(st) != cudaSuccess) return OZK_ERR_CUDA;
  StatusBlock sb;
  if (cudaMemcpy(&sb, g_ws.ptr, sizeof sb, cudaMemcpyDeviceToHost) != cudaSuccess) return OZK_ERR_CUDA;
  if (sb.code != 0) {
    if (sb.code == OZK_ERR_DEVICE_TIMEOUT) fprintf(stderr, "ozk: bounded wait expired at 0x%x\n", sb.where);
    cudaMemset(g_ws.ptr, 0, sizeof(StatusBlock));
  }
  return sb.code;
}

ozk_status ozk_stage_preprocess(int64_t M, int64_t N, int64_t K, const double* A, int64_t lda, const double* B,
                                int64_t ldb, int num_moduli, int32_t* s_out, int32_t* t_out, int64_t* At_out,
                                int64_t* Bt_out, void* stream) {
  Geometry g;
  ozk_status rc = check_common(M, N, K, num_moduli, &g);
  if (rc != OZK_OK) return rc;
  if (M == 0 || N == 0) return OZK_OK;
  if ((K > 0 && (!A || !B)) || lda < (M > 1 ? M : 1) || ldb < (K > 1 ? K : 1)) return OZK_ERR_INVALID_ARG;
  ModulusTable mt;
  if (!host_build_modulus_table(num_moduli, &mt)) return OZK_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  rc = run_preprocess(g, mt, A, lda, B, ldb, At_out, Bt_out, st);
  if (rc != OZK_OK) return rc;
  if (s_out && cudaMemcpyAsync(s_out, g_ws.ptr + g.off_s, (size_t)M * 4, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
    return OZK_ERR_CUDA;
  if (t_out && cudaMemcpyAsync(t_out, g_ws.ptr + g.off_t, (size_t)N * 4, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
    return OZK_ERR_CUDA;
  return OZK_OK;
}

ozk_status ozk_stage_read_planes(char operand, int64_t M, int64_t N, int64_t K, int num_moduli, int l, int limb,
                                 int8_t* out, void* stream) {
  Geometry g;
  ozk_status rc = check_common(M, N, K, num_moduli, &g);
  if (rc != OZK_OK) return rc;
  if (!out || l < 0 || l >= num_moduli || limb < 0 || limb > 4 || (operand != 'A' && operand != 'B')) return OZK_ERR_INVALID_ARG;
  if (limb == 2 && !(g.karatsuba && karatsuba_modulus(l))) return OZK_ERR_INVALID_ARG;  // sum-limb planes exist in the Karatsuba variant only
  const bool a = operand == 'A';
  if (limb >= 3 && !(a && g.gamma)) return OZK_ERR_INVALID_ARG;                          // gamma planes: A side, short K
  const int index = limb < 2 ? 2 * l + limb : (limb == 2 ? 2 * num_moduli + karatsuba_rank(l) : 2 * num_moduli + 2 * l + (limb - 3));
  const uint8_t* plane = g_ws.ptr + (a ? g.off_planes_a : g.off_planes_b) + (size_t)index * (a ? g.plane_bytes_a : g.plane_bytes_b);
  return launch_decode_plane(plane, a ? M : N, K, g.pitch, out, static_cast<cudaStream_t>(stream)) == cudaSuccess ? OZK_OK
                                                                                                                : OZK_ERR_CUDA;
}

ozk_status ozk_stage_residue_gemm(int64_t M, int64_t N, int64_t K, int num_moduli, uint8_t* residues_out, void* stream) {
  Geometry g;
  ozk_status rc = check_common(M, N, K, num_moduli, &g);
  if (rc != OZK_OK) return rc;
  if (M == 0 || N == 0) return OZK_OK;
  if (!device_is_sm100()) return OZK_ERR_UNSUPPORTED;
  ModulusTable mt;
  if (!host_build_modulus_table(num_moduli, &mt)) return OZK_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  rc = gemm_residues_chunked(g, mt, g_ws.ptr, st);
  if (rc != OZK_OK) return rc;
  if (residues_out && launch_copy_residues(g, g_ws.ptr + g.off_res, residues_out, st) != cudaSuccess) return OZK_ERR_CUDA;
  return OZK_OK;
}

ozk_status ozk_stage_crt(int64_t M, int64_t N, int64_t K, int num_moduli, const uint8_t* residues_in, const int32_t* s_in,
                         const int32_t* t_in, double* C, int64_t ldc, uint32_t* x_out, void* stream) {
  Geometry g;
  ozk_status rc = check_common(M, N, K, num_moduli, &g);
  if (rc != OZK_OK) return rc;
  if (M == 0 || N == 0) return OZK_OK;
  if (!C || ldc < M) return OZK_ERR_INVALID_ARG;
  if ((residues_in != nullptr) != (s_in != nullptr) || (s_in != nullptr) != (t_in != nullptr)) return OZK_ERR_INVALID_ARG;
  CrtTable ct;
  if (!host_build_crt_table(num_moduli, &ct)) return OZK_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  cudaError_t e;
  if (residues_in)
    e = launch_crt(g, ct, residues_in, M, (size_t)M * (size_t)N, s_in, t_in, C, ldc, x_out, st);
  else
    e = launch_crt(g, ct, g_ws.ptr + g.off_res, g.Mp, (size_t)g.Mp * (size_t)g.Np,
                   reinterpret_cast<const int32_t*>(g_ws.ptr + g.off_s), reinterpret_cast<const int32_t*>(g_ws.ptr + g.off_t), C,
                   ldc, x_out, st);
  return e == cudaSuccess ? OZK_OK : OZK_ERR_CUDA;
}

ozk_status ozk_dgemm(int64_t M, int64_t N, int64_t K, const double* A, int64_t lda, const double* B, int64_t ldb, double* C,
                     int64_t ldc, int num_moduli, void* stream) {
  return ozk_dgemm_ext(M, N, K, A, lda, B, ldb, C, ldc, num_moduli, 53, stream);
}

ozk_status ozk_dgemm_ext(int64_t M, int64_t N, int64_t K, const double* A, int64_t lda, const double* B, int64_t ldb,
                         double* C, int64_t ldc, int num_moduli, int max_bits, void* stream) {
  Geometry g;
  ozk_status rc = check_common(M, N, K, num_moduli, &g, max_bits);
  if (rc != OZK_OK) return rc;
  if (M == 0 || N == 0) return OZK_OK;
  if (!C || ldc < M || (K > 0 && (!A || !B)) || lda < (M > 1 ? M : 1) || ldb < (K > 1 ? K : 1)) return OZK_ERR_INVALID_ARG;
  if (!device_is_sm100()) return OZK_ERR_UNSUPPORTED;
  ModulusTable mt;
  CrtTable ct;
  if (!host_build_modulus_table(num_moduli, &mt) || !host_build_crt_table(num_moduli, &ct)) return OZK_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  mark(0, st);
  rc = run_preprocess(g, mt, A, lda, B, ldb, nullptr, nullptr, st);
  if (rc != OZK_OK) return rc;
  mark(1, st);
  rc = gemm_residues_chunked(g, mt, g_ws.ptr, st);
  if (rc != OZK_OK) return rc;
  mark(2, st);
  if (launch_crt(g, ct, g_ws.ptr + g.off_res, g.Mp, (size_t)g.Mp * (size_t)g.Np,
                 reinterpret_cast<const int32_t*>(g_ws.ptr + g.off_s), reinterpret_cast<const int32_t*>(g_ws.ptr + g.off_t), C, ldc,
                 nullptr, st) != cudaSuccess)
    return OZK_ERR_CUDA;
  mark(3, st);
  if (g_timing.enabled) ++g_timing.calls;
  return OZK_OK;
}

ozk_status ozk_stage_timing_enable(int enable) {
  if (enable && !g_timing.created) {
    for (int r = 0; r < kTimingRing; ++r)
      for (int i = 0; i < 4; ++i)
        if (cudaEventCreate(&g_timing.ev[r][i]) != cudaSuccess) return OZK_ERR_CUDA;
    g_timing.created = true;
  }
  g_timing.enabled = enable != 0;
  g_timing.calls = 0;
  return OZK_OK;
}

ozk_status ozk_stage_timing_read(float* ms3) {
  if (!ms3) return OZK_ERR_INVALID_ARG;
  if (g_timing.calls < 1) return OZK_ERR_INVALID_ARG;
  const int n = g_timing.calls < kTimingRing ? g_timing.calls : kTimingRing;
  double sum[3] = {0.0, 0.0, 0.0};
  for (int back = 0; back < n; ++back) {
    cudaEvent_t* ev = g_timing.ev[(g_timing.calls - 1 - back) % kTimingRing];
    if (cudaEventSynchronize(ev[3]) != cudaSuccess) return OZK_ERR_CUDA;
    for (int i = 0; i < 3; ++i) {
      float ms = 0.0f;
      if (cudaEventElapsedTime(&ms, ev[i], ev[i + 1]) != cudaSuccess) return OZK_ERR_CUDA;
      sum[i] += ms;
    }
  }
  for (int i = 0; i < 3; ++i) ms3[i] = (float)(sum[i] / n);
  g_timing.calls = 0;
  return OZK_OK;
}

ozk_status ozk_stage_set_karatsuba(int enable) {
  g_karatsuba = enable != 0;
  return OZK_OK;
}

ozk_status ozk_stage_gemm_cycles(long long* clk3) {
  if (!clk3) return OZK_ERR_INVALID_ARG;
  if (!g_ws.ptr) return OZK_ERR_WORKSPACE;
  StatusBlock sb;
  if (cudaMemcpy(&sb, g_ws.ptr, sizeof sb, cudaMemcpyDeviceToHost) != cudaSuccess) return OZK_ERR_CUDA;
  clk3[0] = sb.mma_clk_total;
  clk3[1] = sb.mma_clk_wait_tmem;
  clk3[2] = sb.mma_clk_wait_operands;
  return OZK_OK;
}

ozk_status ozk_stage_mma_probe(const uint8_t* P, const uint8_t* Q, int64_t K, int scale_byte, float* D, void* stream) {
  if (!P || !Q || !D || K <= 0 || K % kTileKNibbles != 0) return OZK_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(P) & 15) || (reinterpret_cast<uintptr_t>(Q) & 15)) return OZK_ERR_INVALID_ARG;
  if (!g_ws.ptr) return OZK_ERR_WORKSPACE;
  if (!device_is_sm100()) return OZK_ERR_UNSUPPORTED;
  return gemm_probe(P, Q, K, scale_byte, D, g_ws.ptr, static_cast<cudaStream_t>(stream));
}

ozk_status ozk_stage_wait_probe(void* stream) {
  // operands and result of one 128 x 128 x 256 probe live in the workspace, past the status block and the tables
  const size_t off_p = 64 << 10, off_q = 96 << 10, off_d = 128 << 10, need = (128 << 10) + 128 * 128 * sizeof(float);
  if (!g_ws.ptr || g_ws.bytes < need) return OZK_ERR_WORKSPACE;
  if (!device_is_sm100()) return OZK_ERR_UNSUPPORTED;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cudaMemsetAsync(g_ws.ptr + off_p, 0, 64 << 10, st) != cudaSuccess) return OZK_ERR_CUDA;
  return gemm_probe(g_ws.ptr + off_p, g_ws.ptr + off_q, kTileKNibbles, 0x7F, reinterpret_cast<float*>(g_ws.ptr + off_d), g_ws.ptr, st,
                    true);
}

}  // extern "C"
