// Register-row compaction (Section 3.2, X -> X' = [X_prefix; X_suffix]) and beam lineage bookkeeping.
//
// compact_kernel: one CTA per (register slot m, sequence b).  The source row is position
// idx_b[m] = m (m < r_h) or L_b - r_t + (m - r_h) of the sequence; its K and V rows (Hkv*D elements
// each, contiguous) are copied as 16-byte vectors into row m of the sequence's pages, and the Q row
// (Hq*D elements) into q_reg[b, m].  Pure byte moves: results are bit-identical to the source.
#include "earn_common.cuh"

namespace earn {
namespace {

__global__ void __launch_bounds__(128) compact_kernel(CompactArgs a) {
  pdl_launch_dependents();
  pdl_wait();   // everything below reads or writes global memory
  const int m = blockIdx.x, b = blockIdx.y;
  const int R = a.r_head + a.r_tail;
  const int lo = a.cu_seqlens[b], len = a.cu_seqlens[b + 1] - lo;
  const int pos = (m < a.r_head) ? m : len - a.r_tail + (m - a.r_head);
  const int64_t src_row = (int64_t)lo + pos;
  const int page = m / EARN_PAGE_TOKENS;
  int phys = a.block_table ? a.block_table[b * a.pages_per_seq + page] : b * a.pages_per_seq + page;
  phys = min(max(phys, 0), a.n_pages - 1);   // a corrupt table writes a wrong page, never outside the cache
  const int64_t dst_row = (int64_t)phys * EARN_PAGE_TOKENS + (m % EARN_PAGE_TOKENS);

  const int kv_vec = a.kv_row_bytes / 16;
  const uint4* ks = reinterpret_cast<const uint4*>(reinterpret_cast<const char*>(a.k) + src_row * a.kv_row_bytes);
  const uint4* vs = reinterpret_cast<const uint4*>(reinterpret_cast<const char*>(a.v) + src_row * a.kv_row_bytes);
  uint4* kd = reinterpret_cast<uint4*>(reinterpret_cast<char*>(a.k_shared) + dst_row * a.kv_row_bytes);
  uint4* vd = reinterpret_cast<uint4*>(reinterpret_cast<char*>(a.v_shared) + dst_row * a.kv_row_bytes);
  for (int i = threadIdx.x; i < kv_vec; i += blockDim.x) {
    uint4 x = __ldg(ks + i), y = __ldg(vs + i);
    kd[i] = x;
    vd[i] = y;
  }
  if (a.q != nullptr) {
    const int q_vec = a.q_row_bytes / 16;
    const uint4* qs = reinterpret_cast<const uint4*>(reinterpret_cast<const char*>(a.q) + src_row * a.q_row_bytes);
    uint4* qd = reinterpret_cast<uint4*>(reinterpret_cast<char*>(a.q_reg) + ((int64_t)b * R + m) * a.q_row_bytes);
    for (int i = threadIdx.x; i < q_vec; i += blockDim.x) qd[i] = __ldg(qs + i);
  }
  if (a.reg_idx != nullptr && threadIdx.x == 0) a.reg_idx[b * R + m] = pos;
}

__global__ void beam_reparent_kernel(int beams, int max_new, int step, const int32_t* parent,
                                     const int32_t* lineage_in, int32_t* lineage_out, int n_beams) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n_beams * max_new) return;
  int j = i / max_new, t = i % max_new;
  int src = (j / beams) * beams + min(max(parent[j], 0), beams - 1);
  int val;
  if (t < step - 1) val = lineage_in ? lineage_in[(int64_t)src * max_new + t] : src;
  else val = j;   // row step-1 is written by beam j itself at this step; later rows are not read yet
  lineage_out[i] = val;
}

}  // namespace

cudaError_t launch_compact(const CompactArgs& a, cudaStream_t st) {
  dim3 grid(a.r_head + a.r_tail, a.batch);
  cudaError_t e = launch_pdl(compact_kernel, grid, dim3(128), 0, st, a);
  note_launch();
  return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t launch_beam_reparent(int batch, int beams, int max_new, int step, const int32_t* parent,
                                 const int32_t* lineage_in, int32_t* lineage_out, cudaStream_t st) {
  int n = batch * beams * max_new;
  note_launch();
  beam_reparent_kernel<<<(n + 255) / 256, 256, 0, st>>>(beams, max_new, step, parent, lineage_in, lineage_out,
                                                        batch * beams);
  return cudaGetLastError();
}

}  // namespace earn
