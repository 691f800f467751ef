// ozk_dgemm_host: the same computation as ozk_dgemm for matrices that live in HOST memory, with the
// PCIe copies overlapped with the stages (the paper times device-resident data only, Section 6.1;
// this entry point serves callers whose operands start and end on the host).
//
// C is produced in blocks of columns.  Three streams run concurrently:
//   copy-in   A once, then the column blocks of B into two alternating device buffers
//   compute   (the caller's stream) stage 1 for A once; per block: stage 1 for the block of B, limb GEMM,
//             CRT into one of two alternating device buffers
//   copy-out  the finished column blocks of C
// so that after the first block the transfers hide behind the limb GEMM.
#include <mutex>

#include "ozk_common.cuh"

namespace ozk {
namespace {

constexpr int kMaxBlocks = 64;
constexpr int64_t kBlockCols = 4096;

struct HostPipe {
  bool ready = false;
  cudaStream_t s_in = nullptr, s_out = nullptr;
  cudaEvent_t start = nullptr, a_in = nullptr;
  cudaEvent_t b_in[kMaxBlocks], enc[kMaxBlocks], c_done[kMaxBlocks], c_out[kMaxBlocks];
};
HostPipe g_pipe;
std::mutex g_pipe_mutex;

bool ensure_pipe() {
  std::lock_guard<std::mutex> lock(g_pipe_mutex);
  if (g_pipe.ready) return true;
  if (cudaStreamCreateWithFlags(&g_pipe.s_in, cudaStreamNonBlocking) != cudaSuccess) return false;
  if (cudaStreamCreateWithFlags(&g_pipe.s_out, cudaStreamNonBlocking) != cudaSuccess) return false;
  auto mk = [](cudaEvent_t* e) { return cudaEventCreateWithFlags(e, cudaEventDisableTiming) == cudaSuccess; };
  if (!mk(&g_pipe.start) || !mk(&g_pipe.a_in)) return false;
  for (int b = 0; b < kMaxBlocks; ++b)
    if (!mk(&g_pipe.b_in[b]) || !mk(&g_pipe.enc[b]) || !mk(&g_pipe.c_done[b]) || !mk(&g_pipe.c_out[b])) return false;
  g_pipe.ready = true;
  return true;
}

struct HostLayout {
  Geometry g;  // geometry of one column block (N = block width)
  int64_t block_cols;
  int blocks;
  size_t off_a, off_b[2], off_c[2], total;
};

bool make_host_layout(int64_t M, int64_t N, int64_t K, int L, HostLayout* h) {
  if (M < 0 || N < 0 || K < 0) return false;
  h->block_cols = N < kBlockCols ? round_up(N > 0 ? N : 1, 256) : kBlockCols;
  h->blocks = (int)((N + h->block_cols - 1) / h->block_cols);
  if (h->blocks < 1) h->blocks = 1;
  if (h->blocks > kMaxBlocks) return false;
  if (!make_geometry(M, h->block_cols, K, L, &h->g)) return false;
  auto up = [](size_t x) { return (x + 1023) / 1024 * 1024; };
  size_t off = h->g.total;
  h->off_a = off;
  off += up((size_t)(M > 0 ? M : 1) * (size_t)(K > 0 ? K : 1) * 8);
  for (int i = 0; i < 2; ++i) {
    h->off_b[i] = off;
    off += up((size_t)(K > 0 ? K : 1) * (size_t)h->block_cols * 8);
  }
  for (int i = 0; i < 2; ++i) {
    h->off_c[i] = off;
    off += up((size_t)(M > 0 ? M : 1) * (size_t)h->block_cols * 8);
  }
  h->total = off;
  return true;
}

}  // namespace
}  // namespace ozk

using namespace ozk;

extern "C" {

size_t ozk_dgemm_host_workspace_bytes(int64_t M, int64_t N, int64_t K, int num_moduli) {
  HostLayout h;
  return make_host_layout(M, N, K, num_moduli, &h) ? h.total : 0;
}

ozk_status ozk_dgemm_host(int64_t M, int64_t N, int64_t K, const double* A, int64_t lda, const double* B, int64_t ldb,
                          double* C, int64_t ldc, int num_moduli, void* stream) {
  HostLayout h;
  if (!make_host_layout(M, N, K, num_moduli, &h)) return OZK_ERR_INVALID_ARG;
  if (K > 131072 || h.g.c_bits < 1 || h.g.Mp / 32 > 65535) return OZK_ERR_UNSUPPORTED;
  uint8_t* ws = workspace_ptr();
  if (!ws || workspace_bytes() < h.total) return OZK_ERR_WORKSPACE;
  if (M == 0 || N == 0) return OZK_OK;
  if (!C || ldc < M || (K > 0 && (!A || !B)) || lda < (M > 1 ? M : 1) || ldb < (K > 1 ? K : 1)) return OZK_ERR_INVALID_ARG;
  ModulusTable mt;
  CrtTable ct;
  if (!host_build_modulus_table(num_moduli, &mt) || !host_build_crt_table(num_moduli, &ct)) return OZK_ERR_INVALID_ARG;
  if (!ensure_pipe()) return OZK_ERR_CUDA;
  HostPipe& p = g_pipe;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  double* dA = reinterpret_cast<double*>(ws + h.off_a);
  double* dB[2] = {reinterpret_cast<double*>(ws + h.off_b[0]), reinterpret_cast<double*>(ws + h.off_b[1])};
  double* dC[2] = {reinterpret_cast<double*>(ws + h.off_c[0]), reinterpret_cast<double*>(ws + h.off_c[1])};
  const Geometry& g = h.g;
#define OZK_TRY(call) do { if ((call) != cudaSuccess) return OZK_ERR_CUDA; } while (0)
  // the side streams start after whatever the caller has already enqueued on `stream`
  OZK_TRY(cudaEventRecord(p.start, st));
  OZK_TRY(cudaStreamWaitEvent(p.s_in, p.start, 0));
  OZK_TRY(cudaStreamWaitEvent(p.s_out, p.start, 0));
  if (K > 0)
    OZK_TRY(cudaMemcpy2DAsync(dA, (size_t)M * 8, A, (size_t)lda * 8, (size_t)M * 8, (size_t)K, cudaMemcpyHostToDevice, p.s_in));
  OZK_TRY(cudaEventRecord(p.a_in, p.s_in));
  // stage 1 for A (row shifts, limb planes), once
  OZK_TRY(launch_build_lut(mt, ws + g.off_lut, st));
  OZK_TRY(cudaStreamWaitEvent(st, p.a_in, 0));
  OZK_TRY(launch_scan_operand(g, 0, dA, M, ws, st));
  OZK_TRY(launch_encode_operand(g, mt, 0, dA, M, ws, nullptr, st));
  for (int b = 0; b < h.blocks; ++b) {
    const int64_t j0 = (int64_t)b * h.block_cols;
    const int64_t nb = N - j0 < h.block_cols ? N - j0 : h.block_cols;
    Geometry gb = g;  // same layout and padded width; only the number of valid columns changes
    gb.N = nb;
    if (b >= 2) OZK_TRY(cudaStreamWaitEvent(p.s_in, p.enc[b - 2], 0));  // the buffer's previous block has been encoded
    if (K > 0)
      OZK_TRY(cudaMemcpy2DAsync(dB[b & 1], (size_t)K * 8, B + j0 * ldb, (size_t)ldb * 8, (size_t)K * 8, (size_t)nb,
                                cudaMemcpyHostToDevice, p.s_in));
    OZK_TRY(cudaEventRecord(p.b_in[b], p.s_in));
    OZK_TRY(cudaStreamWaitEvent(st, p.b_in[b], 0));
    OZK_TRY(launch_scan_operand(gb, 1, dB[b & 1], K > 0 ? K : 1, ws, st));
    OZK_TRY(launch_encode_operand(gb, mt, 1, dB[b & 1], K > 0 ? K : 1, ws, nullptr, st));
    OZK_TRY(cudaEventRecord(p.enc[b], st));
    const ozk_status rc = gemm_residues(gb, mt, ws, st);
    if (rc != OZK_OK) return rc;
    if (b >= 2) OZK_TRY(cudaStreamWaitEvent(st, p.c_out[b - 2], 0));  // the buffer's previous block has left the device
    OZK_TRY(launch_crt(gb, ct, ws + g.off_res, g.Mp, (size_t)g.Mp * (size_t)g.Np, reinterpret_cast<const int32_t*>(ws + g.off_s),
                       reinterpret_cast<const int32_t*>(ws + g.off_t), dC[b & 1], M, nullptr, st));
    OZK_TRY(cudaEventRecord(p.c_done[b], st));
    OZK_TRY(cudaStreamWaitEvent(p.s_out, p.c_done[b], 0));
    OZK_TRY(cudaMemcpy2DAsync(C + j0 * ldc, (size_t)ldc * 8, dC[b & 1], (size_t)M * 8, (size_t)M * 8, (size_t)nb,
                              cudaMemcpyDeviceToHost, p.s_out));
    OZK_TRY(cudaEventRecord(p.c_out[b], p.s_out));
  }
  OZK_TRY(cudaStreamWaitEvent(st, p.c_out[h.blocks - 1], 0));  // `stream` completes when C has arrived
#undef OZK_TRY
  return OZK_OK;
}

}  // extern "C"
