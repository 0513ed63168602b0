// Decode attention (Eq. 4) over a SHORT key list: the compact register cache of a layer l >= k plus the few generated
// tokens (Section 3.2, decoding rule), one tile of at most 16 query rows per (sequence, kv head).
//
// With 30 to 130 cache positions per (sequence, kv head) a launch moves a few MB: it is not the HBM stream that sets
// its time but the chain of dependent steps inside a CTA (fetch, a few tiles of arithmetic, store) and the hand-over
// from one launch to the next.  A per-CTA timeline of the one-warp streaming kernel on this case showed 5.8 us of
// chain for 1.9 us of transfer: one warp walking four tiles in turn, index arithmetic for the generated tokens between
// the stream-order wait and the first fetch, then the store.  This kernel is shaped for the chain instead:
//   * one CTA = (sequence, kv head), NW warps, the WHOLE list (at most NW tiles of 16 positions) in shared memory;
//   * before the stream-order wait (when the host allows it, see DecodeArgs::prefetch_shared): all index arithmetic
//     and the fetch of the shared segment; after it only what the step brought: q, k_new / v_new, the generated tokens;
//   * S = Q K^T split over the KEYS -- warp w takes tile w (one round of MMAs) -- and the scores meet in shared memory;
//   * every warp then holds the whole score row: one plain softmax (no running maximum, nothing to rescale or merge);
//   * O = P V split over the COLUMNS of V -- warp w takes D / NW of them -- so no partial outputs are combined;
//   * Eq. 4's append is served from the tile already in shared memory (no second fetch of k_new / v_new).
// Two block-wide barriers per launch.  Everything else (which rows a lane holds, P rounded to bf16 before P V, fp32
// accumulation, log2-domain exponentials) is as in the streaming kernels.
#include <type_traits>

#include "decode_tile.cuh"
#include "sm100_ptx.cuh"

namespace earn {
namespace {
using namespace dec;

// Pins a value computed ahead of the stream-order wait: the compiler otherwise sinks pure arithmetic to its first use,
// which is behind the wait, on the critical path.
__device__ __forceinline__ void pin(int& x) { asm volatile("" : "+r"(x)); }
__device__ __forceinline__ void pin(int64_t& x) { asm volatile("" : "+l"(x)); }
template <typename T>
__device__ __forceinline__ void pin(T*& x) { asm volatile("" : "+l"(x)); }

template <int D, int NW>
struct ShortSmem {
  using G = Geo<D>;
  static constexpr int KV_B = NW * G::STAGE_B;            // NW (K tile, V tile) pairs
  static constexpr int Q_B = 16 * G::PITCH;               // the 16 query rows
  static constexpr int SC_PITCH = NW * 16 + 8;            // floats per score row (padded)
  static constexpr int SC_B = 16 * SC_PITCH * 4;
  static constexpr int BYTES = KV_B + Q_B + SC_B;
};

template <int D, int NW>
__global__ void __launch_bounds__(NW * 32) decode_short_kernel(DecodeArgs a) {
  using G = Geo<D>;
  using S = ShortSmem<D, NW>;
  constexpr int NT = NW * 32, CH = G::CH, RPP = NT / CH;   // RPP: list positions (rows) one pass of all threads covers
  constexpr int PASSES = NW * 16 / RPP, QPASSES = 16 / RPP;
  constexpr int KSTEPS = D / 16;
  constexpr int NPW = D / 8 / NW;                          // 8-column blocks of V (and O) per warp
  static_assert(NPW >= 2 && NPW % 2 == 0 && 16 % RPP == 0, "column split");
  extern __shared__ __align__(128) uint8_t smem[];
  const uint32_t kv = ptx::smem_u32(smem), qs = kv + S::KV_B;
  float* sc = reinterpret_cast<float*>(smem + S::KV_B + S::Q_B);

  const bool early_fetch = a.prefetch_shared != 0;
  if (!early_fetch) {
    pdl_wait();
    if (a.trigger_early) pdl_launch_dependents();   // never ahead of the wait (see decode_mma.cu)
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int b = blockIdx.z, kvh = blockIdx.x;
  RowMap rm;
  rm.b = b; rm.kvh = kvh; rm.row0 = 0; rm.g = a.Hq / a.Hkv; rm.W = a.beams; rm.n_rows = rm.W * rm.g; rm.Hq = a.Hq;
  const int g = rm.g, W = rm.W, step = a.step;
  const int seq_lo = a.src.paged ? 0 : a.cu_seqlens[b];
  const int n_shared = a.src.paged ? a.src.n_regs : (a.cu_seqlens[b + 1] - seq_lo);
  const int n_total = n_shared + W * step;                 // every beam of the sequence has rows in this one tile
  const float scale_log2 = a.scale * kLog2e;
  const bf16* kg = reinterpret_cast<const bf16*>(a.src.k);
  const bf16* vg = reinterpret_cast<const bf16*>(a.src.v);

  // ---- where every row lives, worked out ONCE per row (thread p for list position p, the next 16 threads for the
  // query rows) and passed through a table in shared memory: the divisions and 64-bit products of this arithmetic,
  // done by every thread for each of its pieces, were 2 us of a CTA's life.  The table sits in the score area, which
  // nothing else uses before the first barrier behind the wait.
  const bool affine = !a.src.paged || a.src.block_table == nullptr;
  const int64_t row_base = a.src.paged ? (int64_t)b * a.src.pages_per_seq * EARN_PAGE_TOKENS : (int64_t)seq_lo;
  int64_t* tab_off = reinterpret_cast<int64_t*>(sc);          // [NW*16] element offset of the row (this kv head) in its tensor
  int64_t* tab_q = tab_off + NW * 16;                          // [16] element offset of the query / output row, -1: none
  int* tab_key = reinterpret_cast<int*>(tab_q + 16);           // [NW*16] -1: shared or zero row; -3: newest token; else j * max_new + t
  int* tab_beam = tab_key + NW * 16;                           // [16] beam of the query row
  static_assert((NW * 16 + 16) * 12 <= S::SC_B, "table fits the score area");
  if ((int)threadIdx.x < NW * 16) {
    const int p = threadIdx.x;
    int64_t off = 0;
    int key = -1;
    if (p < n_shared) {
      off = ((affine ? row_base + p : key_row(a.src, b, p)) * a.Hkv + kvh) * D;
    } else if (p < n_total) {
      const int pk = p - n_shared, w = pk / step, t = pk - w * step;
      const int64_t j = (int64_t)b * W + w;
      if (t == step - 1) {
        key = -3;
        off = (j * a.Hkv + kvh) * D;
      } else {
        key = (int)(j * a.max_new + t);
        off = ((j * a.max_new + t) * a.Hkv + kvh) * D;   // flat slabs, identity lineage; corrected behind the wait otherwise
      }
    }
    tab_off[p] = off;
    tab_key[p] = key;
  } else if ((int)threadIdx.x < NW * 16 + 16) {
    const int r = threadIdx.x - NW * 16;
    tab_q[r] = rm.offset(r, D);
    tab_beam[r] = r / g;
  }
  __syncthreads();

  // ---- copies: thread -> (list position r_t + i * RPP, 16-byte chunk c_t), K and V alike; position p sits in row
  // p % 16 of tile p / 16.  Shared rows are fetched now; rows past the list, and query rows past W*g, are zeroed with
  // plain stores; the rest waits.
  const int c_t = threadIdx.x % CH, r_t = threadIdx.x / CH;
  auto dst_of = [&](int p) { return kv + (uint32_t)(p >> 4) * G::STAGE_B + (uint32_t)(p & 15) * G::PITCH + (uint32_t)c_t * 16; };
  int64_t p_off[PASSES];
  int p_key[PASSES];
#pragma unroll
  for (int i = 0; i < PASSES; ++i) {   // (all table reads first, in one block of code: they overlap)
    p_off[i] = tab_off[r_t + i * RPP] + c_t * 8;
    p_key[i] = tab_key[r_t + i * RPP];
  }
#pragma unroll
  for (int i = 0; i < PASSES; ++i) {
    const int p = r_t + i * RPP;
    if (p < n_shared) {
      cp_async16(dst_of(p), kg + p_off[i]);
      cp_async16(dst_of(p) + G::TILE_B, vg + p_off[i]);
    } else if (p >= n_total) {
      uint8_t* z = smem + (p >> 4) * G::STAGE_B + (p & 15) * G::PITCH + c_t * 16;
      *reinterpret_cast<uint4*>(z) = make_uint4(0u, 0u, 0u, 0u);
      *reinterpret_cast<uint4*>(z + G::TILE_B) = make_uint4(0u, 0u, 0u, 0u);
    }
  }
  int64_t q_off[QPASSES];
#pragma unroll
  for (int i = 0; i < QPASSES; ++i) {
    q_off[i] = tab_q[r_t + i * RPP];
    if (q_off[i] < 0)
      *reinterpret_cast<uint4*>(smem + S::KV_B + (r_t + i * RPP) * G::PITCH + c_t * 16) = make_uint4(0u, 0u, 0u, 0u);
  }
  const int r0 = lane >> 2, r1 = r0 + 8, c2 = (lane & 3) * 2;
  int64_t o_off0 = tab_q[r0], o_off1 = tab_q[r1];
  int seen_bits = 0;   // bit n * 4 + e: element e of 8-column block n of this warp's score tile is visible to its row
  {
    // generated tokens a row may see: its own beam's, at list positions vis .. vis + step - 1
    const int vis0 = n_shared + tab_beam[r0] * step, vis1 = n_shared + tab_beam[r1] * step;
#pragma unroll
    for (int n = 0; n < 2; ++n)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int p = warp * KT + n * 8 + c2 + (e & 1), v0 = e >= 2 ? vis1 : vis0;
        if (p < n_shared || (p >= v0 && p < v0 + step)) seen_bits |= 1 << (n * 4 + e);
      }
  }
  // Eq. 4, append: the newest token of beam w sits at list position n_shared + w * step + step - 1; piece i of the
  // W * 2 * CH 16-byte pieces goes from the tile in shared memory to the private segment.  The first piece of each
  // thread (all of them up to four beams) is addressed here, ahead of the wait.
  auto app_piece = [&](int i, const uint8_t*& src, bf16*& dst) {
    const int w = i / (2 * CH), c = i % (2 * CH), p = n_shared + w * step + step - 1;
    src = smem + (p >> 4) * G::STAGE_B + (c >= CH ? G::TILE_B : 0) + (p & 15) * G::PITCH + (c % CH) * 16;
    dst = reinterpret_cast<bf16*>(c >= CH ? a.v_priv : a.k_priv) +
          (priv_row(a, (int64_t)b * W + w, step - 1) * a.Hkv + kvh) * D + (c % CH) * 8;
  };
  const uint8_t* app_src = nullptr;
  bf16* app_dst = nullptr;
  // (a page table of the private segment may have been written just ahead of this launch: it is read behind the wait)
  if ((int)threadIdx.x < W * 2 * CH && a.priv_table == nullptr) app_piece(threadIdx.x, app_src, app_dst);
  {
    pin(app_src); pin(app_dst);
    pin(o_off0); pin(o_off1); pin(seen_bits);
#pragma unroll
    for (int i = 0; i < PASSES; ++i) { pin(p_off[i]); pin(p_key[i]); }
#pragma unroll
    for (int i = 0; i < QPASSES; ++i) pin(q_off[i]);
  }

  if (early_fetch) {
    pdl_wait();   // q, k_new, v_new, the private segment and the lineage table are read from here on
    if (a.trigger_early) pdl_launch_dependents();
  }
  {
    const bf16* qg = reinterpret_cast<const bf16*>(a.q);
#pragma unroll
    for (int i = 0; i < QPASSES; ++i)   // (a pass without query rows is skipped by every thread alike)
      if (i * RPP < rm.n_rows && q_off[i] >= 0)
        cp_async16(qs + (uint32_t)(r_t + i * RPP) * G::PITCH + (uint32_t)c_t * 16, qg + q_off[i] + c_t * 8);
    const bf16 *kpriv = reinterpret_cast<const bf16*>(a.k_priv), *vpriv = reinterpret_cast<const bf16*>(a.v_priv);
    const bf16 *knew = reinterpret_cast<const bf16*>(a.k_new), *vnew = reinterpret_cast<const bf16*>(a.v_new);
#pragma unroll
    for (int i = 0; i < PASSES; ++i) {
      // a pass that holds no generated token is skipped by every thread alike: a compare and a branch, no more
      if ((i + 1) * RPP <= n_shared || i * RPP >= n_total) continue;
      const int p = r_t + i * RPP;
      if (p_key[i] == -1) continue;
      int64_t off = p_off[i];
      if ((a.lineage != nullptr || a.priv_table != nullptr) && p_key[i] >= 0) {
        // the token lives in the slab of the beam that generated it, and possibly behind a page table
        const int t = p_key[i] % a.max_new;
        const int64_t slab = a.lineage != nullptr ? min(max(a.lineage[p_key[i]], 0), a.batch * W - 1) : p_key[i] / a.max_new;
        off = (priv_row(a, slab, t) * a.Hkv + kvh) * D + c_t * 8;
      }
      const bool fresh = p_key[i] == -3;
      cp_async16(dst_of(p), (fresh ? knew : kpriv) + off);
      cp_async16(dst_of(p) + G::TILE_B, (fresh ? vnew : vpriv) + off);
    }
  }
  cp_async_commit();
  cp_async_wait<0>();
  __syncthreads();

  // ---- Eq. 4, append, from the tile in shared memory
  if (app_src != nullptr) *reinterpret_cast<uint4*>(app_dst) = *reinterpret_cast<const uint4*>(app_src);
  for (int i = threadIdx.x + (a.priv_table == nullptr ? NT : 0); i < W * 2 * CH; i += NT) {
    app_piece(i, app_src, app_dst);
    *reinterpret_cast<uint4*>(app_dst) = *reinterpret_cast<const uint4*>(app_src);
  }

  // ---- S = Q K^T for tile `warp`; scaled scores (log2 domain) into shared memory, invisible positions as -inf
  const int mat = lane >> 3;
  if (warp * KT < n_total) {
    const uint32_t q_lane = qs + (uint32_t)((lane & 7) + ((lane >> 3) & 1) * 8) * G::PITCH + (uint32_t)(lane >> 4) * 16;
    const uint32_t k_lane = kv + warp * G::STAGE_B + (uint32_t)(((mat >> 1) << 3) + (lane & 7)) * G::PITCH + (uint32_t)(mat & 1) * 16;
    float s[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}}, s2[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
    for (int kk = 0; kk < KSTEPS; kk += 2) {
      uint32_t qa[4], qb[4], b0, b1, b2, b3, d0, d1, d2, d3;
      ldsm_x4(q_lane + kk * 32, qa[0], qa[1], qa[2], qa[3]);
      ldsm_x4(q_lane + (kk + 1) * 32, qb[0], qb[1], qb[2], qb[3]);
      ldsm_x4(k_lane + kk * 32, b0, b1, b2, b3);
      ldsm_x4(k_lane + (kk + 1) * 32, d0, d1, d2, d3);
      mma_bf16(s[0], qa, b0, b1);
      mma_bf16(s[1], qa, b2, b3);
      mma_bf16(s2[0], qb, d0, d1);
      mma_bf16(s2[1], qb, d2, d3);
    }
#pragma unroll
    for (int n = 0; n < 2; ++n) {
      float x[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) x[e] = (seen_bits >> (n * 4 + e)) & 1 ? (s[n][e] + s2[n][e]) * scale_log2 : -INFINITY;
      *reinterpret_cast<float2*>(sc + r0 * S::SC_PITCH + warp * KT + n * 8 + c2) = make_float2(x[0], x[1]);
      *reinterpret_cast<float2*>(sc + r1 * S::SC_PITCH + warp * KT + n * 8 + c2) = make_float2(x[2], x[3]);
    }
  }
  __syncthreads();

  // ---- softmax and P V, compiled once per number of key tiles in the list: with the tile count a run-time test inside
  // the unrolled loops, every tile became a basic block of its own and its shared-memory load, exponentials and MMAs
  // ran at their full latency one tile after another.
  const int n_tiles = (n_total + KT - 1) / KT;   // 1 .. NW
  float l0, l1, o[NPW][4];
  auto tail = [&](auto n_tiles_tag) {
    constexpr int N_TILES = decltype(n_tiles_tag)::value;
    // ---- softmax of the lane's two rows over the whole list (every warp the same), P as bf16 A-fragments
    float x0[NW][4], m0 = -INFINITY, m1 = -INFINITY;   // [tile][(r0, c2..) (r1, c2..) (r0, 8 + c2..) (r1, 8 + c2..)] pairs
    float y0[NW][4];
#pragma unroll
    for (int kk = 0; kk < NW; ++kk) {
      if (kk < N_TILES) {
        const float2 a0 = *reinterpret_cast<const float2*>(sc + r0 * S::SC_PITCH + kk * KT + c2);
        const float2 a1 = *reinterpret_cast<const float2*>(sc + r1 * S::SC_PITCH + kk * KT + c2);
        const float2 a2 = *reinterpret_cast<const float2*>(sc + r0 * S::SC_PITCH + kk * KT + 8 + c2);
        const float2 a3 = *reinterpret_cast<const float2*>(sc + r1 * S::SC_PITCH + kk * KT + 8 + c2);
        x0[kk][0] = a0.x; x0[kk][1] = a0.y; x0[kk][2] = a2.x; x0[kk][3] = a2.y;
        y0[kk][0] = a1.x; y0[kk][1] = a1.y; y0[kk][2] = a3.x; y0[kk][3] = a3.y;
        m0 = fmaxf(m0, fmaxf(fmaxf(a0.x, a0.y), fmaxf(a2.x, a2.y)));
        m1 = fmaxf(m1, fmaxf(fmaxf(a1.x, a1.y), fmaxf(a3.x, a3.y)));
      }
    }
    m0 = fmaxf(m0, __shfl_xor_sync(0xffffffffu, m0, 1));
    m0 = fmaxf(m0, __shfl_xor_sync(0xffffffffu, m0, 2));
    m1 = fmaxf(m1, __shfl_xor_sync(0xffffffffu, m1, 1));
    m1 = fmaxf(m1, __shfl_xor_sync(0xffffffffu, m1, 2));
    if (m0 == -INFINITY) m0 = 0.f;   // a row past W*g of a list without shared rows: never stored
    if (m1 == -INFINITY) m1 = 0.f;
    uint32_t pf[NW][4];
    l0 = 0.f, l1 = 0.f;
#pragma unroll
    for (int kk = 0; kk < NW; ++kk) {
      if (kk < N_TILES) {
        const float p0 = ex2(x0[kk][0] - m0), p1 = ex2(x0[kk][1] - m0), p2 = ex2(x0[kk][2] - m0), p3 = ex2(x0[kk][3] - m0);
        const float q0 = ex2(y0[kk][0] - m1), q1 = ex2(y0[kk][1] - m1), q2 = ex2(y0[kk][2] - m1), q3 = ex2(y0[kk][3] - m1);
        l0 += (p0 + p1) + (p2 + p3);
        l1 += (q0 + q1) + (q2 + q3);
        pf[kk][0] = pack2(p0, p1); pf[kk][1] = pack2(q0, q1); pf[kk][2] = pack2(p2, p3); pf[kk][3] = pack2(q2, q3);
      }
    }
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
    l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 2);

    // ---- O = P V for this warp's columns [warp * D / NW, (warp + 1) * D / NW)
#pragma unroll
    for (int n = 0; n < NPW; ++n) o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f;
    const uint32_t v_lane = kv + G::TILE_B + (uint32_t)(((mat & 1) << 3) + (lane & 7)) * G::PITCH + (uint32_t)(mat >> 1) * 16 +
                            (uint32_t)warp * (NPW * 16);
#pragma unroll
    for (int kk = 0; kk < NW; ++kk) {
      if (kk < N_TILES) {
#pragma unroll
        for (int nn = 0; nn < NPW / 2; ++nn) {
          uint32_t b0, b1, b2, b3;
          ldsm_x4_t(v_lane + kk * G::STAGE_B + nn * 32, b0, b1, b2, b3);
          mma_bf16(o[2 * nn], pf[kk], b0, b1);
          mma_bf16(o[2 * nn + 1], pf[kk], b2, b3);
        }
      }
    }
  };
  if (n_tiles <= 1) tail(std::integral_constant<int, 1>{});
  else if (n_tiles == 2) tail(std::integral_constant<int, 2>{});
  else if (n_tiles == 3) tail(std::integral_constant<int, 3>{});
  else if (NW == 4 || n_tiles == 4) tail(std::integral_constant<int, 4>{});
  else if constexpr (NW > 4) {
    if (n_tiles == 5) tail(std::integral_constant<int, 5>{});
    else if (n_tiles == 6) tail(std::integral_constant<int, 6>{});
    else if (n_tiles == 7) tail(std::integral_constant<int, 7>{});
    else tail(std::integral_constant<int, 8>{});
  }
  if (!a.trigger_early) pdl_launch_dependents();
  const float i0 = 1.f / l0, i1 = 1.f / l1;
  bf16* og = reinterpret_cast<bf16*>(a.o);
#pragma unroll
  for (int n = 0; n < NPW; ++n) {
    const int col = warp * (NPW * 8) + n * 8 + c2;
    if (o_off0 >= 0) *reinterpret_cast<uint32_t*>(og + o_off0 + col) = pack2(o[n][0] * i0, o[n][1] * i0);
    if (o_off1 >= 0) *reinterpret_cast<uint32_t*>(og + o_off1 + col) = pack2(o[n][2] * i1, o[n][3] * i1);
  }
}

template <int D, int NW>
cudaError_t launch_short(const DecodeArgs& a, cudaStream_t st) {
  constexpr int smem = ShortSmem<D, NW>::BYTES;
  cudaError_t e = ensure_dynamic_smem<decode_short_kernel<D, NW>>(smem);
  if (e != cudaSuccess) return e;
  e = launch_pdl(decode_short_kernel<D, NW>, dim3(a.Hkv, 1, a.batch), dim3(NW * 32), smem, st, a);
  note_launch();
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace

// One row tile, no split, no order table, and the longest list (shared segment + every beam's generated tokens) fits
// NW tiles.
bool decode_short_supported(const DecodeArgs& a, int max_shared_len) {
  return a.dtype == EARN_BF16 && a.plan.row_tiles == 1 && a.plan.n_splits <= 1 && a.order == nullptr &&
         max_shared_len + a.beams * a.step <= (a.D == 64 ? 4 : 8) * KT;
}

cudaError_t launch_decode_short(const DecodeArgs& a, int max_shared_len, cudaStream_t st) {
  const bool four = max_shared_len + a.beams * a.step <= 4 * KT;
  if (a.D == 64) return launch_short<64, 4>(a, st);
  return four ? launch_short<128, 4>(a, st) : launch_short<128, 8>(a, st);
}

}  // namespace earn
