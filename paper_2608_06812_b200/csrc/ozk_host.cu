// ozk_dgemm_host: the same computation as ozk_dgemm for matrices that live in HOST memory, with the
// PCIe copies overlapped with the stages (the paper times device-resident data only, Section 6.1;
// this entry point serves callers whose operands start and end on the host).
//
// C is produced in blocks (2048 x 2048 by default).  Three streams run concurrently:
//   copy-in   column block 0 of B, row block 0 of A, column block 1 of B, row block 1 of A, ...
//   compute   (the caller's stream) stage 1 for each block of A or B as it arrives (its planes and
//             shifts stay on the device), then limb GEMM and CRT for every block of C whose row block
//             and column block have both arrived
//   copy-out  the finished blocks of C
// A row block only needs its own rows for its shifts and planes (one exponent per row, Section 4.2),
// likewise a column block of B, so the first limb GEMM starts after one small block of each has
// arrived; the number of blocks of C that can be computed grows quadratically with the data that
// has arrived, and after a short start-up the transfers hide behind the limb GEMM.  Staging buffers
// and their events are used in rings of two.
#include <stdlib.h>

#include <mutex>

#include "ozk_common.cuh"

namespace ozk {
namespace {

constexpr int kMaxBlocks = 64;
constexpr int64_t kBlock = 2048;

struct HostPipe {
  bool ready = false;
  cudaStream_t s_in = nullptr, s_out = nullptr;
  cudaEvent_t start = nullptr;
  cudaEvent_t a_in[2], a_enc[2], b_in[2], b_enc[2], c_done[2], c_out[2];
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
    if (!mk(&g_pipe.a_in[i]) || !mk(&g_pipe.a_enc[i]) || !mk(&g_pipe.b_in[i]) || !mk(&g_pipe.b_enc[i]) ||
        !mk(&g_pipe.c_done[i]) || !mk(&g_pipe.c_out[i]))
      return false;
  g_pipe.ready = true;
  return true;
}

// Block edge: 2048, grown in steps of 256 until neither direction needs more than kMaxBlocks blocks.
// OZK_HOST_BLOCK (a multiple of 256) overrides the 2048 (measurement aid).
int64_t block_edge(int64_t M, int64_t N) {
  int64_t edge = kBlock;
  if (const char* e = getenv("OZK_HOST_BLOCK")) {
    const long long v = atoll(e);
    if (v >= 256 && v % 256 == 0) edge = v;
  }
  const int64_t longest = M > N ? M : N;
  const int64_t needed = round_up((longest + kMaxBlocks - 1) / kMaxBlocks, 256);
  return edge > needed ? edge : needed;
}

struct HostLayout {
  Geometry g;  // geometry of a full block: sizes, pitch, plane sizes (offsets and ragged sizes are set per block)
  int64_t mb, nb;  // block rows / columns
  int rblocks, cblocks;
  size_t off_status, off_lut;
  size_t off_amax_a, off_s, off_planes_a;  // per row block: + r * stride
  size_t stride_amax_a, stride_s, stride_planes_a;
  size_t off_amax_b, off_t, off_planes_b;  // per column block: + b * stride
  size_t stride_amax_b, stride_t, stride_planes_b;
  size_t off_res, off_stage_a[2], off_stage_b[2], off_stage_c[2];
  size_t total;
};

bool make_host_layout(int64_t M, int64_t N, int64_t K, int L, HostLayout* h) {
  if (M < 0 || N < 0 || K < 0) return false;
  const int64_t edge = block_edge(M, N);
  h->mb = M < edge ? (M > 0 ? M : 1) : edge;
  h->nb = N < edge ? round_up(N > 0 ? N : 1, 256) : edge;
  h->rblocks = (int)((M + h->mb - 1) / h->mb);
  h->cblocks = (int)((N + h->nb - 1) / h->nb);
  if (h->rblocks < 1) h->rblocks = 1;
  if (h->cblocks < 1) h->cblocks = 1;
  if (h->rblocks > kMaxBlocks || h->cblocks > kMaxBlocks) return false;
  if (!make_geometry(h->mb, h->nb, K, L, &h->g)) return false;
  h->g.karatsuba = 0;  // the host-buffer path keeps the two planes per modulus
  h->g.gamma = 0;
  const Geometry& g = h->g;
  auto up = [](size_t x) { return (x + 1023) / 1024 * 1024; };
  const size_t kk = (size_t)(K > 0 ? K : 1);
  size_t off = 0;
  h->off_status = off;
  off += 1024;
  h->off_lut = off;
  off += up(kEncTableBytes);
  h->stride_amax_a = up((size_t)g.Mp * 8);
  h->stride_s = up((size_t)g.Mp * 4);
  h->off_amax_a = off;
  off += h->stride_amax_a * h->rblocks;
  h->off_s = off;
  off += h->stride_s * h->rblocks;
  h->stride_amax_b = up((size_t)g.Np * 8);
  h->stride_t = up((size_t)g.Np * 4);
  h->off_amax_b = off;
  off += h->stride_amax_b * h->cblocks;
  h->off_t = off;
  off += h->stride_t * h->cblocks;
  h->stride_planes_a = 2 * (size_t)L * g.plane_bytes_a;
  h->off_planes_a = off;
  off += h->stride_planes_a * h->rblocks;
  h->stride_planes_b = 2 * (size_t)L * g.plane_bytes_b;
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

// Geometry of block (row block r, column block b) with `rows` x `cols` valid elements.  A ragged last
// block is padded to the tile size only, not to the full block, so its planes lie more densely in
// their region and its limb GEMM does no more work than its size asks for.
Geometry block_geometry(const HostLayout& h, int r, int b, int64_t rows, int64_t cols) {
  Geometry g = h.g;
  g.M = rows;
  g.N = cols;
  g.Mp = round_up(rows, kTileRows);
  g.Np = round_up(cols, 256);
  if (g.Np > h.g.Np) g.Np = h.g.Np;
  g.plane_bytes_a = (size_t)g.Mp * g.pitch;
  g.plane_bytes_b = (size_t)g.Np * g.pitch;
  g.off_status = h.off_status;
  g.off_lut = h.off_lut;
  g.off_amax_a = h.off_amax_a + (size_t)r * h.stride_amax_a;
  g.off_s = h.off_s + (size_t)r * h.stride_s;
  g.off_planes_a = h.off_planes_a + (size_t)r * h.stride_planes_a;
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
  OZK_TRY(launch_build_lut(mt, ws + h.off_lut, 0, st));
  auto rows_of = [&](int r) { const int64_t i0 = (int64_t)r * h.mb; return M - i0 < h.mb ? M - i0 : h.mb; };
  auto cols_of = [&](int b) { const int64_t j0 = (int64_t)b * h.nb; return N - j0 < h.nb ? N - j0 : h.nb; };
  int out_index = 0;
  // limb GEMM, CRT and copy-out of block (r, b) of C; both operands' planes are on the device
  auto compute_block = [&](int r, int b) -> ozk_status {
    const int64_t i0 = (int64_t)r * h.mb, j0 = (int64_t)b * h.nb;
    const int64_t rows = rows_of(r), cols = cols_of(b);
    const Geometry g = block_geometry(h, r, b, rows, cols);
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
    return OZK_OK;
  };
  // arrivals alternate between the two operands while both have blocks left: B0 A0 B1 A1 ...
  int next_r = 0, next_b = 0;
  while (next_r < h.rblocks || next_b < h.cblocks) {
    const bool take_b = next_b < h.cblocks && (next_b <= next_r || next_r >= h.rblocks);
    if (take_b) {
      const int b = next_b++, ring = b & 1;
      const int64_t j0 = (int64_t)b * h.nb, cols = cols_of(b);
      double* dB = reinterpret_cast<double*>(ws + h.off_stage_b[ring]);
      if (b >= 2) OZK_TRY(cudaStreamWaitEvent(p.s_in, p.b_enc[ring], 0));  // the staging buffer has been encoded
      if (K > 0)
        OZK_TRY(cudaMemcpy2DAsync(dB, (size_t)kk * 8, B + j0 * ldb, (size_t)ldb * 8, (size_t)K * 8, (size_t)cols,
                                  cudaMemcpyHostToDevice, p.s_in));
      OZK_TRY(cudaEventRecord(p.b_in[ring], p.s_in));
      OZK_TRY(cudaStreamWaitEvent(st, p.b_in[ring], 0));
      const Geometry g = block_geometry(h, 0, b, rows_of(0), cols);
      OZK_TRY(launch_scan_operand(g, 1, dB, kk, ws, st));
      OZK_TRY(launch_encode_operand(g, mt, 1, dB, kk, ws, nullptr, st));
      OZK_TRY(cudaEventRecord(p.b_enc[ring], st));
      for (int r = 0; r < next_r; ++r) {
        const ozk_status rc = compute_block(r, b);
        if (rc != OZK_OK) return rc;
      }
    } else {
      const int r = next_r++, ring = r & 1;
      const int64_t i0 = (int64_t)r * h.mb, rows = rows_of(r);
      double* dA = reinterpret_cast<double*>(ws + h.off_stage_a[ring]);
      if (r >= 2) OZK_TRY(cudaStreamWaitEvent(p.s_in, p.a_enc[ring], 0));
      if (K > 0)
        OZK_TRY(cudaMemcpy2DAsync(dA, (size_t)h.mb * 8, A + i0, (size_t)lda * 8, (size_t)rows * 8, (size_t)K,
                                  cudaMemcpyHostToDevice, p.s_in));
      OZK_TRY(cudaEventRecord(p.a_in[ring], p.s_in));
      OZK_TRY(cudaStreamWaitEvent(st, p.a_in[ring], 0));
      const Geometry g = block_geometry(h, r, 0, rows, cols_of(0));
      OZK_TRY(launch_scan_operand(g, 0, dA, h.mb, ws, st));
      OZK_TRY(launch_encode_operand(g, mt, 0, dA, h.mb, ws, nullptr, st));
      OZK_TRY(cudaEventRecord(p.a_enc[ring], st));
      for (int b = 0; b < next_b; ++b) {
        const ozk_status rc = compute_block(r, b);
        if (rc != OZK_OK) return rc;
      }
    }
  }
  // `stream` completes when the last block of C has arrived (the copy-out stream is in order)
  OZK_TRY(cudaStreamWaitEvent(st, p.c_out[(out_index - 1) & 1], 0));
#undef OZK_TRY
  return OZK_OK;
}

}  // extern "C"
