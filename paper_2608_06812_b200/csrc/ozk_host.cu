// ozk_dgemm_host: the same computation as ozk_dgemm for matrices that live in HOST memory, with the
// PCIe copies overlapped with the stages (the paper times device-resident data only, Section 6.1;
// this entry point serves callers whose operands start and end on the host).
//
// C is produced in blocks of 4096 x 4096.  Three streams run concurrently:
//   copy-in   row block 0 of A, the column blocks of B, then the remaining row blocks of A
//   compute   (the caller's stream) stage 1 for a row block of A as it arrives, stage 1 for each column
//             block of B once (its planes stay on the device), then per block limb GEMM and CRT
//   copy-out  the finished blocks of C
// A row block only needs its own rows for its shifts and planes (one exponent per row, Section 4.2), so
// the first limb GEMM starts after one block of A and one block of B have arrived, and from then on
// the transfers hide behind the limb GEMM.  Staging buffers and events are used in rings of two.
#include <mutex>

#include "ozk_common.cuh"

namespace ozk {
namespace {

constexpr int kMaxBlocks = 64;
constexpr int64_t kBlock = 4096;

struct HostPipe {
  bool ready = false;
  cudaStream_t s_in = nullptr, s_out = nullptr;
  cudaEvent_t start = nullptr;
  cudaEvent_t a_in[2], a_done[2], b_in[2], b_enc[2], c_done[2], c_out[2];
};
HostPipe g_pipe;
std::mutex g_pipe_mutex;

bool ensure_pipe() {
  std::lock_guard<std::mutex> lock(g_pipe_mutex);
  if (g_pipe.ready) return true;
  if (cudaStreamCreateWithFlags(&g_pipe.s_in, cudaStreamNonBlocking) != cudaSuccess) return false;
  if (cudaStreamCreateWithFlags(&g_pipe.s_out, cudaStreamNonBlocking) != cudaSuccess) return false;
  auto mk = [](cudaEvent_t* e) { return cudaEventCreateWithFlags(e, cudaEventDisableTiming) == cudaSuccess; };
  if (!mk(&g_pipe.start)) return false;
  for (int i = 0; i < 2; ++i)
    if (!mk(&g_pipe.a_in[i]) || !mk(&g_pipe.a_done[i]) || !mk(&g_pipe.b_in[i]) || !mk(&g_pipe.b_enc[i]) ||
        !mk(&g_pipe.c_done[i]) || !mk(&g_pipe.c_out[i]))
      return false;
  g_pipe.ready = true;
  return true;
}

struct HostLayout {
  Geometry g;  // geometry of one block: sizes, pitch, plane sizes (offsets are set per block)
  int64_t mb, nb;  // block rows / columns
  int rblocks, cblocks;
  size_t off_status, off_lut;
  size_t off_amax_a[2], off_s[2], off_planes_a[2], off_stage_a[2];
  size_t off_amax_b, off_t, off_planes_b;  // per column block: + b * stride
  size_t stride_amax_b, stride_t, stride_planes_b;
  size_t off_res, off_stage_b[2], off_stage_c[2];
  size_t total;
};

bool make_host_layout(int64_t M, int64_t N, int64_t K, int L, HostLayout* h) {
  if (M < 0 || N < 0 || K < 0) return false;
  h->mb = M < kBlock ? (M > 0 ? M : 1) : kBlock;
  h->nb = N < kBlock ? round_up(N > 0 ? N : 1, 256) : kBlock;
  h->rblocks = (int)((M + h->mb - 1) / h->mb);
  h->cblocks = (int)((N + h->nb - 1) / h->nb);
  if (h->rblocks < 1) h->rblocks = 1;
  if (h->cblocks < 1) h->cblocks = 1;
  if (h->rblocks > kMaxBlocks || h->cblocks > kMaxBlocks) return false;
  if (!make_geometry(h->mb, h->nb, K, L, &h->g)) return false;
  const Geometry& g = h->g;
  auto up = [](size_t x) { return (x + 1023) / 1024 * 1024; };
  const size_t kk = (size_t)(K > 0 ? K : 1);
  size_t off = 0;
  h->off_status = off;
  off += 1024;
  h->off_lut = off;
  off += up((size_t)kMaxModuli * kLutStride * sizeof(uint16_t));
  for (int i = 0; i < 2; ++i) {
    h->off_amax_a[i] = off;
    off += up((size_t)g.Mp * 8);
    h->off_s[i] = off;
    off += up((size_t)g.Mp * 4);
  }
  h->stride_amax_b = up((size_t)g.Np * 8);
  h->stride_t = up((size_t)g.Np * 4);
  h->stride_planes_b = 2 * (size_t)L * g.plane_bytes_b;
  h->off_amax_b = off;
  off += h->stride_amax_b * h->cblocks;
  h->off_t = off;
  off += h->stride_t * h->cblocks;
  for (int i = 0; i < 2; ++i) {
    h->off_planes_a[i] = off;
    off += 2 * (size_t)L * g.plane_bytes_a;
  }
  h->off_planes_b = off;
  off += h->stride_planes_b * h->cblocks;
  h->off_res = off;
  off += up((size_t)L * (size_t)g.Mp * (size_t)g.Np);
  for (int i = 0; i < 2; ++i) {
    h->off_stage_a[i] = off;
    off += up((size_t)h->mb * kk * 8);
  }
  for (int i = 0; i < 2; ++i) {
    h->off_stage_b[i] = off;
    off += up(kk * (size_t)h->nb * 8);
  }
  for (int i = 0; i < 2; ++i) {
    h->off_stage_c[i] = off;
    off += up((size_t)h->mb * (size_t)h->nb * 8);
  }
  h->total = off;
  return true;
}

// Geometry of block (row buffer ra, column block b) with `rows` x `cols` valid elements.
Geometry block_geometry(const HostLayout& h, int ra, int b, int64_t rows, int64_t cols) {
  Geometry g = h.g;
  g.M = rows;
  g.N = cols;
  g.off_status = h.off_status;
  g.off_lut = h.off_lut;
  g.off_amax_a = h.off_amax_a[ra];
  g.off_s = h.off_s[ra];
  g.off_planes_a = h.off_planes_a[ra];
  g.off_amax_b = h.off_amax_b + (size_t)b * h.stride_amax_b;
  g.off_t = h.off_t + (size_t)b * h.stride_t;
  g.off_planes_b = h.off_planes_b + (size_t)b * h.stride_planes_b;
  g.off_res = h.off_res;
  return g;
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
  if (K > kChunkK || h.g.c_bits < 1 || h.g.Mp / 32 > 65535) return OZK_ERR_UNSUPPORTED;
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
  const int64_t kk = K > 0 ? K : 1;
#define OZK_TRY(call) do { if ((call) != cudaSuccess) return OZK_ERR_CUDA; } while (0)
  // the side streams start after whatever the caller has already enqueued on `stream`
  OZK_TRY(cudaEventRecord(p.start, st));
  OZK_TRY(cudaStreamWaitEvent(p.s_in, p.start, 0));
  OZK_TRY(cudaStreamWaitEvent(p.s_out, p.start, 0));
  OZK_TRY(launch_build_lut(mt, ws + h.off_lut, st));
  int out_index = 0;
  for (int r = 0; r < h.rblocks; ++r) {
    const int ra = r & 1;
    const int64_t i0 = (int64_t)r * h.mb;
    const int64_t rows = M - i0 < h.mb ? M - i0 : h.mb;
    double* dA = reinterpret_cast<double*>(ws + h.off_stage_a[ra]);
    // row block r of A: copy in (once the buffers of row block r-2 are free), then stage 1 for these rows
    if (r >= 2) OZK_TRY(cudaStreamWaitEvent(p.s_in, p.a_done[ra], 0));
    if (K > 0)
      OZK_TRY(cudaMemcpy2DAsync(dA, (size_t)h.mb * 8, A + i0, (size_t)lda * 8, (size_t)rows * 8, (size_t)K,
                                cudaMemcpyHostToDevice, p.s_in));
    OZK_TRY(cudaEventRecord(p.a_in[ra], p.s_in));
    OZK_TRY(cudaStreamWaitEvent(st, p.a_in[ra], 0));
    {
      const Geometry ga = block_geometry(h, ra, 0, rows, h.nb);
      OZK_TRY(launch_scan_operand(ga, 0, dA, h.mb, ws, st));
      OZK_TRY(launch_encode_operand(ga, mt, 0, dA, h.mb, ws, nullptr, st));
    }
    for (int b = 0; b < h.cblocks; ++b) {
      const int64_t j0 = (int64_t)b * h.nb;
      const int64_t cols = N - j0 < h.nb ? N - j0 : h.nb;
      const Geometry g = block_geometry(h, ra, b, rows, cols);
      if (r == 0) {  // column block b of B: copy in and encode once; its planes and shifts stay resident
        const int bb = b & 1;
        double* dB = reinterpret_cast<double*>(ws + h.off_stage_b[bb]);
        if (b >= 2) OZK_TRY(cudaStreamWaitEvent(p.s_in, p.b_enc[bb], 0));
        if (K > 0)
          OZK_TRY(cudaMemcpy2DAsync(dB, (size_t)kk * 8, B + j0 * ldb, (size_t)ldb * 8, (size_t)K * 8, (size_t)cols,
                                    cudaMemcpyHostToDevice, p.s_in));
        OZK_TRY(cudaEventRecord(p.b_in[bb], p.s_in));
        OZK_TRY(cudaStreamWaitEvent(st, p.b_in[bb], 0));
        OZK_TRY(launch_scan_operand(g, 1, dB, kk, ws, st));
        OZK_TRY(launch_encode_operand(g, mt, 1, dB, kk, ws, nullptr, st));
        OZK_TRY(cudaEventRecord(p.b_enc[bb], st));
      }
      const ozk_status rc = gemm_residues(g, mt, ws, st);
      if (rc != OZK_OK) return rc;
      const int oc = out_index & 1;
      double* dC = reinterpret_cast<double*>(ws + h.off_stage_c[oc]);
      if (out_index >= 2) OZK_TRY(cudaStreamWaitEvent(st, p.c_out[oc], 0));  // this buffer's previous block has left
      OZK_TRY(launch_crt(g, ct, ws + g.off_res, g.Mp, (size_t)g.Mp * (size_t)g.Np, reinterpret_cast<const int32_t*>(ws + g.off_s),
                         reinterpret_cast<const int32_t*>(ws + g.off_t), dC, h.mb, nullptr, st));
      OZK_TRY(cudaEventRecord(p.c_done[oc], st));
      OZK_TRY(cudaStreamWaitEvent(p.s_out, p.c_done[oc], 0));
      OZK_TRY(cudaMemcpy2DAsync(C + i0 + j0 * ldc, (size_t)ldc * 8, dC, (size_t)h.mb * 8, (size_t)rows * 8, (size_t)cols,
                                cudaMemcpyDeviceToHost, p.s_out));
      OZK_TRY(cudaEventRecord(p.c_out[oc], p.s_out));
      ++out_index;
    }
    OZK_TRY(cudaEventRecord(p.a_done[ra], st));
  }
  // `stream` completes when the last block of C has arrived (the copy-out stream is in order)
  OZK_TRY(cudaStreamWaitEvent(st, p.c_out[(out_index - 1) & 1], 0));
#undef OZK_TRY
  return OZK_OK;
}

}  // extern "C"
