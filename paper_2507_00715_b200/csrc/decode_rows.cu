// Decode attention (Eq. 4) when the query rows of a (sequence, kv head) fill several 16-row tiles: beam search,
// where W beams x g heads of the group share one kv head (the paper generates with beam 20, Appendix A.3).
//
// Every row tile needs the whole shared segment (the prompt K/V of a layer l < k, or the compact register pages
// of a layer l >= k).  One CTA per row tile would fetch it once per tile (three times at 10 beams x 4 heads,
// which left the prompt-cache layers L2-bound at 2.7 TB/s on B200).  Here one CTA = (sequence, kv head, split of
// the shared segment, group of RT row tiles), one warp per row tile:
//   phase 1  all warps copy the shared segment tile by tile into ONE ring of shared memory (16-byte cp.async,
//            a block-wide barrier per tile) and each warp attends its own 16 rows to every tile;
//   phase 2  (split 0) each warp walks the generated tokens of its own beams alone, through its slice of the ring;
//   finish   per warp, exactly as in the one-row-tile kernel: write the rows, or publish a partial and fold.
// DRAM traffic of a prompt-cache layer of the ragged 10-beam workload fell to 737 MB (710 MB algorithmic) and the
// layer from 260 us to 232 us; what bounds it now is latency at three CTAs per SM (166 registers per thread):
// 40 query rows per kv head are 10 times the mma.sync work per byte of the one-beam case.  Forcing four CTAs per
// SM (128 registers, a shallower ring) measured 271 us, two CTAs 271 us.
#include "decode_tile.cuh"
#include "sm100_ptx.cuh"

namespace earn {
namespace {
using namespace dec;

// RT warps = row tiles per CTA; ST ring stages, a multiple of RT; MINB = CTAs per SM the register budget allows for
template <int D, int RT, int ST, int MINB>
__global__ void __launch_bounds__(RT * 32, MINB) decode_rows_kernel(DecodeArgs a) {
  using G = Geo<D>;
  constexpr int NT = RT * 32, CH = G::CH, SPW = ST / RT;   // SPW: ring stages a warp owns in phase 2
  static_assert(ST % RT == 0 && SPW >= 1 && NT % CH == 0 && ST >= 4, "ring slices");
  extern __shared__ __align__(128) uint8_t smem[];
  // As in the one-row-tile kernel: with prefetch_shared the first tiles of the shared segment are fetched before the
  // wait for the kernel ahead on the stream (which cannot have written them); the order table is written just ahead.
  const bool early_fetch = a.prefetch_shared && a.order == nullptr;
  if (!early_fetch) {
    pdl_wait();
    if (a.trigger_early) pdl_launch_dependents();   // never ahead of the wait (see decode_mma.cu)
  }

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // CTAs are handed out in grid order: with an order table the longest sequences start first and the launch does
  // not end on a long sequence that started late
  const int b = a.order ? a.order[blockIdx.z] : (int)blockIdx.z, kvh = blockIdx.x;
  const int row_groups = (a.plan.row_tiles + RT - 1) / RT;
  const int split = blockIdx.y / row_groups, row_tile = (blockIdx.y % row_groups) * RT + warp;
  const bool active = row_tile < a.plan.row_tiles;   // a warp without a row tile still helps with the copies
  RowMap rm;
  rm.b = b; rm.kvh = kvh; rm.row0 = row_tile * 16; rm.g = a.Hq / a.Hkv; rm.W = a.beams; rm.n_rows = rm.W * rm.g; rm.Hq = a.Hq;
  const int g = rm.g, W = rm.W, step = a.step;
  const int seq_lo = a.src.paged ? 0 : a.cu_seqlens[b];
  const int shared_len = a.src.paged ? a.src.n_regs : (a.cu_seqlens[b + 1] - seq_lo);
  const int key_begin = split * a.plan.chunk;
  const int n_shared = max(min(key_begin + a.plan.chunk, shared_len) - key_begin, 0);
  if (n_shared == 0 && split != 0) {   // a split past the end of this sequence
    if (early_fetch) pdl_wait();
    return;
  }
  const int n_sh_tiles = (n_shared + KT - 1) / KT;
  const float scale_log2 = a.scale * kLog2e;

  Sources src;
  src.k[0] = reinterpret_cast<const bf16*>(a.src.k); src.v[0] = reinterpret_cast<const bf16*>(a.src.v);
  src.k[1] = reinterpret_cast<const bf16*>(a.k_priv); src.v[1] = reinterpret_cast<const bf16*>(a.v_priv);
  src.k[2] = reinterpret_cast<const bf16*>(a.k_new); src.v[2] = reinterpret_cast<const bf16*>(a.v_new);

  // ---- phase 1 copies: thread -> (row r_t + i * NT/CH of the tile, 16-byte chunk c_t), K and V alike
  const uint32_t ring = ptx::smem_u32(smem);
  const int c_t = threadIdx.x % CH, r_t = threadIdx.x / CH;
  const bool affine = !a.src.paged || a.src.block_table == nullptr;
  const int64_t row_base = a.src.paged ? (int64_t)b * a.src.pages_per_seq * EARN_PAGE_TOKENS : (int64_t)seq_lo;
  auto issue_shared = [&](int tile, int stage) {
    const uint32_t kdst = ring + stage * G::STAGE_B + (uint32_t)c_t * 16, vdst = kdst + G::TILE_B;
#pragma unroll
    for (int i = 0; i < (KT + NT / CH - 1) / (NT / CH); ++i) {   // NT / CH rows per pass; the last pass may be partial
      const int r = r_t + i * (NT / CH), p = tile * KT + r;
      if (KT % (NT / CH) != 0 && r >= KT) break;
      const bool ok = p < n_shared;
      const int64_t row = !ok ? 0 : affine ? row_base + key_begin + p : key_row(a.src, b, key_begin + p);
      const int64_t off = (row * a.Hkv + kvh) * D + c_t * 8;
      cp_async16(kdst + r * G::PITCH, src.k[0] + off, ok ? 16 : 0);
      cp_async16(vdst + r * G::PITCH, src.v[0] + off, ok ? 16 : 0);
    }
  };
#pragma unroll
  for (int s = 0; s < ST - 2; ++s) {
    if (s < n_sh_tiles) issue_shared(s, s);
    cp_async_commit();
  }
  if (early_fetch) {
    pdl_wait();   // the lineage table, q, k_new, v_new and the private segment are read from here on
    if (a.trigger_early) pdl_launch_dependents();
  }

  // ---- where the generated tokens of this row tile's beams live: resolved now (lane -> positions lane, lane + 32,
  // ... of the tile's list), so that the lineage look-ups are in flight together and under phase 1
  const int w_lo = rm.row0 / g, w_hi = min((rm.row0 + 15) / g, W - 1);
  const int n_priv = (active && split == 0) ? (w_hi - w_lo + 1) * step : 0, n_pt = (n_priv + KT - 1) / KT;
  constexpr int NPRE = 4;   // rounds of 32 positions resolved ahead (8 tiles); later tiles are resolved as they come
  int64_t pre[NPRE];        // element offset * 4 + tensor, -1: no such position
#pragma unroll
  for (int j = 0; j < NPRE; ++j) {
    const int pk = j * 32 + lane;
    int which = 1;
    pre[j] = -1;
    if (pk < n_priv) pre[j] = private_row<D>(a, b, kvh, w_lo, pk, which) * 4 + which;
  }

  // ---- the Q fragments, while the first tiles are in flight
  RowTile<D> t;
  if (active) t.init(reinterpret_cast<const bf16*>(a.q), rm, lane);

  // two tiles per round: one block-wide barrier and one softmax step per 32 positions
  for (int it = 0; it < n_sh_tiles; it += 2) {
    cp_async_wait<ST - 4>();   // this thread's copies of tiles it and it+1 have landed ...
    __syncthreads();           // ... and everyone's; every warp is also done with tiles it-2 and it-1, whose stages are refilled next
#pragma unroll
    for (int u = 0; u < 2; ++u) {
      const int nxt = it + ST - 2 + u;
      if (nxt < n_sh_tiles) issue_shared(nxt, nxt % ST);
      cp_async_commit();
    }
    if (active) {
      const uint32_t ks = ring + (it % ST) * G::STAGE_B, vs = ks + G::TILE_B;
      const uint32_t ks2 = ring + ((it + 1) % ST) * G::STAGE_B, vs2 = ks2 + G::TILE_B;
      if ((it + 2) * KT <= n_shared) {
        t.attend2(ks, vs, ks2, vs2, scale_log2, lane);
      } else {
        t.attend(ks, vs, scale_log2, lane, (it + 1) * KT > n_shared, [&](int c, bool) { return it * KT + c < n_shared; });
        if (it + 1 < n_sh_tiles)
          t.attend(ks2, vs2, scale_log2, lane, true, [&](int c, bool) { return (it + 1) * KT + c < n_shared; });
      }
    }
  }
  cp_async_wait<0>();
  if (!a.trigger_early) pdl_launch_dependents();   // from here on the next kernel on the stream may be scheduled
  __syncthreads();           // the ring is idle: each warp takes its slice
  if (!active) return;
  // ---- Eq. 4: append (split 0).  Nothing in this launch reads the rows it writes (the newest token comes straight
  // from k_new / v_new), so the copy stays out of the way of the loads above.
  if (split == 0) append_new_rows<D>(a, rm, lane, 32);

  // ---- phase 2 (split 0): the generated tokens of this row tile's beams, newest from k_new / v_new
  if (split == 0) {
    // positions of its list each of the lane's two rows may see: its own beam's `step` tokens
    const int vis0 = ((rm.row0 + (lane >> 2)) / g - w_lo) * step, vis1 = ((rm.row0 + (lane >> 2) + 8) / g - w_lo) * step;
    const uint32_t mine = ring + warp * SPW * G::STAGE_B;
    auto issue_private = [&](int tile, int stage) {
      if (tile < 2 * NPRE) {   // tiles 2j and 2j + 1 were resolved by lanes 0..15 and 16..31 of round j
        const int j = tile >> 1;
        const int64_t e = j == 0 ? pre[0] : j == 1 ? pre[1] : j == 2 ? pre[2] : pre[3];
        copy_resolved_tile<D>(mine + stage * G::STAGE_B, e < 0 ? -1 : e >> 2, (int)(e & 3), src, lane, (tile & 1) * 16);
      } else {
        const int pk = tile * KT + lane;
        int64_t off = -1;
        int which = 1;
        if (lane < KT && pk < n_priv) off = private_row<D>(a, b, kvh, w_lo, pk, which);
        copy_resolved_tile<D>(mine + stage * G::STAGE_B, off, which, src, lane);
      }
    };
#pragma unroll
    for (int s = 0; s < SPW - 1; ++s) {
      if (s < n_pt) issue_private(s, s);
      cp_async_commit();
    }
    for (int it = 0; it < n_pt; ++it) {
      {
        const int nxt = it + SPW - 1;
        if (nxt < n_pt) issue_private(nxt, nxt % SPW);
        cp_async_commit();
        cp_async_wait<SPW - 1>();
        __syncwarp();
      }
      const uint32_t ks = mine + (it % SPW) * G::STAGE_B, vs = ks + G::TILE_B;
      t.attend(ks, vs, scale_log2, lane, true, [&](int c, bool second) {   // only the row's own beam is visible
        const int pk = it * KT + c, v0 = second ? vis1 : vis0;
        return pk >= v0 && pk < v0 + step && pk < n_priv;
      });
      __syncwarp();
    }
    cp_async_wait<0>();
    __syncwarp();
  }

  t.reduce_sums();
  if (a.plan.n_splits <= 1) {
    t.store_rows(smem + warp * SPW * G::STAGE_B, reinterpret_cast<bf16*>(a.o), rm, lane);
  } else {
    const int live_splits = max(1, min(a.plan.n_splits, (shared_len + a.plan.chunk - 1) / a.plan.chunk));
    publish_and_fold<D>(t, a, rm, split, live_splits, row_tile, lane);
  }
}

template <int D, int RT, int ST, int MINB>
cudaError_t launch_rows(const DecodeArgs& a, cudaStream_t st) {
  constexpr int smem = ST * Geo<D>::STAGE_B;
  cudaError_t e = ensure_dynamic_smem<decode_rows_kernel<D, RT, ST, MINB>>(smem);
  if (e != cudaSuccess) return e;
  const int splits = a.plan.n_splits > 0 ? a.plan.n_splits : 1;
  dim3 grid(a.Hkv, splits * ((a.plan.row_tiles + RT - 1) / RT), a.batch);
  e = launch_pdl(decode_rows_kernel<D, RT, ST, MINB>, grid, dim3(RT * 32), smem, st, a);
  note_launch();
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace

cudaError_t launch_decode_rows(const DecodeArgs& a, cudaStream_t st) {
  // four warps, eight stages: 68 KB of shared memory allow three CTAs per SM; hold the registers to that too
  if (a.plan.row_tiles > 2) {
    // Three row tiles per CTA (96 threads, six stages, four CTAs per SM) when that leaves fewer warps without a row
    // tile than four would (3, 5, 6 and 9 row tiles) and the shared segment is short, so that the launch is bound by
    // the latency chain of a CTA and by how many CTAs are resident, not by streaming.  Measured on B200: 48
    // sequences x 4 kv heads x 140 rows (20 beams, group of 7), 50-200 token prompts: 16.3 -> 10.3 us per
    // compact-cache layer, 27.0 -> 20.2 us per prompt-cache layer; 128 sequences x 8 kv heads x 40 rows: 42.7 -> 34.7
    // us per compact-cache layer, but 201 -> 208 us per prompt-cache layer of up to 2048 tokens, which therefore
    // keeps four warps and the eight-stage ring.
    const int rt = a.plan.row_tiles, idle3 = (rt + 2) / 3 * 3 - rt, idle4 = (rt + 3) / 4 * 4 - rt;
    const bool three = idle3 < idle4 && a.plan.chunk <= 512;
    if (three) return a.D == 64 ? launch_rows<64, 3, 6, 4>(a, st) : launch_rows<128, 3, 6, 4>(a, st);
    return a.D == 64 ? launch_rows<64, 4, 8, 3>(a, st) : launch_rows<128, 4, 8, 3>(a, st);
  }
  // Two row tiles (17 to 32 query rows per kv head, e.g. 20 beams of a multi-head model).  With a six-stage ring
  // four CTAs fit an SM; a launch with more CTAs than that runs in waves, each paying the whole latency chain of a
  // CTA, so it takes a four-stage ring and a register budget that fit six.  Measured on B200, 24 sequences x 32 kv
  // heads x 20 beams (768 CTAs): 26.7 -> 17.5 us per compact-cache layer, 42.4 -> 30.8 us per prompt-cache layer;
  // with few CTAs (8 long sequences, split) the deeper ring is the faster one, 49.8 against 54.0 us.
  const long ctas = (long)a.Hkv * (a.plan.n_splits > 0 ? a.plan.n_splits : 1) * a.batch;
  const bool many = ctas > 4L * sm_count();
  if (a.D == 64) return many ? launch_rows<64, 2, 4, 6>(a, st) : launch_rows<64, 2, 6, 4>(a, st);
  return many ? launch_rows<128, 2, 4, 6>(a, st) : launch_rows<128, 2, 6, 4>(a, st);
}

}  // namespace earn
