// Decode attention (Eq. 4: append K_t, V_t, then attend over K_{1:t}) for bf16 caches.
//
// HBM-bound: every byte of the cache is read once per step, so the kernel is built around keeping
// loads in flight with few instructions, not around the tensor cores; warp-level mma.sync (m16n8k16)
// only keeps the few query rows per key (g heads x W beams, padded to 16) off the FMA pipe.
//
// This file: one CTA = (sequence b, kv head, split of the shared segment, tile of 16 query rows); one warp, or
// four warps that deal the tiles of a short list among themselves when the grid is small.  (With several row
// tiles -- beams x group size > 16 -- decode_rows.cu lets the row tiles of a CTA share one pass over the shared
// segment instead.)  The key
// list of a CTA is its chunk of the shared segment (the prompt K/V of a layer l < k read in place, or
// the compact register pages of a layer l >= k) followed -- in split 0 only -- by the generated tokens
// of the beams its rows belong to (masked per row to the row's own beam; the newest token comes
// straight from k_new / v_new, which split 0 also appends to the private segment).
//
// The list is cut into tiles of 16 positions.  The warp fetches them with 16-byte cp.async copies into
// padded shared-memory tiles (a ring of four stages = 35 KB at head_dim 128, so six CTAs share an SM; three
// stages, the whole list in flight at once, for lists of at most two tiles).  Tile size, warps per CTA and ring depth were swept on B200 at
// the 7B shapes: (16, 1, 4) gave 50.9 us per layer against 51.3-63.4 us for the other combinations.
// A long list is then consumed two tiles at a time (one softmax step, one rescale of the accumulator and one
// round of quad shuffles per 32 positions, four independent MMA chains instead of two): 49.6 -> 46.3 us per
// prompt-cache layer at the 7B shapes, 6.0 TB/s.  Deeper rings behind the pairs were slower (five stages 48.0,
// six 52.5, eight 76 us), three stages 56 us.
// Rows that are an affine function of the list position (packed prompt K/V, identity page table)
// take a fast path of pointer increments; any other tile (scattered pages, generated tokens
// behind the lineage table, a ragged last tile) first resolves one row per lane and hands the row
// offsets to the copying lanes by shuffle.  (One bulk copy per 256-byte row measured 4.0 TB/s on B200
// against 6.2 TB/s for this scheme: the row is too small a unit for the copy engine.)
// Online softmax in the log2 domain.  With a single split the CTA writes O itself; otherwise it writes a
// normalised partial + log2-domain LSE, takes a ticket, and the CTA holding the last ticket of its
// (sequence, kv head, row tile) folds the partials -- one launch, and no CTA ever waits for another.
// The fold is on the critical path of the launch (it starts when the slowest split ends), so it walks the
// splits once with a running maximum, four splits' loads in flight at a time.
#include "decode_tile.cuh"
#include "sm100_ptx.cuh"

namespace earn {
namespace {
using namespace dec;

#ifndef EARN_DECODE_STAGES
#define EARN_DECODE_STAGES 4
#endif

// how a CTA walks its key list
enum Walk {
  STREAM,   // one warp, a long list: tiles consumed two at a time behind a full ring
  SHORT,    // one warp, a list of at most two tiles: the whole list in flight from the start
  SHARED    // several warps deal the tiles round-robin and merge their states at the end
};

template <int D, int STAGES, int NWARPS>   // STAGES: cp.async ring depth per warp; NWARPS: warps per CTA, tiles dealt round-robin
struct Smem {
  static constexpr int RING_B = NWARPS * STAGES * Geo<D>::STAGE_B;
  static constexpr int MERGE_B = NWARPS * 16 * D * 4 + NWARPS * 16 * 2 * 4 + 16;
  static constexpr int BYTES = RING_B > MERGE_B ? RING_B : MERGE_B;
};

template <int D, int STAGES, int NWARPS, Walk WALK>
__global__ void __launch_bounds__(NWARPS * 32) decode_mma_kernel(DecodeArgs a) {
  static_assert((WALK == SHARED) == (NWARPS > 1) && (WALK != STREAM || STAGES >= 3), "walk");
  using G = Geo<D>;
  constexpr int NTILES = D / 8, CH = G::CH, RPI = G::RPI, NIT = KT / RPI;
  extern __shared__ __align__(128) uint8_t smem[];
  // Launched programmatically, this kernel may start while its predecessor on the stream still runs; nothing the
  // predecessor may have written is read before pdl_wait().  The shared segment (prompt K/V or register pages), the
  // block table and cu_seqlens are not among that when the host says so (prefetch_shared): the first tiles of the
  // key list are then on their way while the predecessor finishes.  The order table IS written just ahead.
  const bool early_fetch = a.prefetch_shared && a.order == nullptr;
  if (!early_fetch) {
    pdl_wait();
    // (never ahead of the wait: a kernel that lets its successor start only after its own predecessor has ended keeps
    // every kernel further back ended too, which is what the successor's early fetch relies on)
    if (a.trigger_early) pdl_launch_dependents();
  }

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // kv heads vary fastest over the grid: the CTAs that read the same rows of the packed K/V tensors (one 256-byte
  // slice each of a 2 KB row) start next to each other and walk those rows together
  // CTAs are handed out in grid order: with an order table the longest sequences start first and the launch does
  // not end on a long sequence that started late
  const int b = a.order ? a.order[blockIdx.z] : (int)blockIdx.z, kvh = blockIdx.x;
  const int row_tiles = a.plan.row_tiles;
  const int split = blockIdx.y / row_tiles, row_tile = blockIdx.y % row_tiles;
  RowMap rm;
  rm.b = b; rm.kvh = kvh; rm.row0 = row_tile * 16; rm.g = a.Hq / a.Hkv; rm.W = a.beams; rm.n_rows = rm.W * rm.g; rm.Hq = a.Hq;
  const int g = rm.g, W = rm.W, step = a.step, row0 = rm.row0;
  const int seq_lo = a.src.paged ? 0 : a.cu_seqlens[b];
  const int shared_len = a.src.paged ? a.src.n_regs : (a.cu_seqlens[b + 1] - seq_lo);
  const int key_begin = split * a.plan.chunk;
  const int n_shared = max(min(key_begin + a.plan.chunk, shared_len) - key_begin, 0);
  const int w_lo = row0 / g, w_hi = min((row0 + 15) / g, W - 1);
  const int n_priv = (split == 0) ? (w_hi - w_lo + 1) * step : 0;
  const int n_total = n_shared + n_priv;
  if (n_total == 0) {
    if (early_fetch) pdl_wait();   // a CTA never ends (which also releases the successor) before the predecessor has
    return;
  }
  const int n_tiles = (n_total + KT - 1) / KT;
  const float scale_log2 = a.scale * kLog2e;

  Sources src;
  src.k[0] = reinterpret_cast<const bf16*>(a.src.k); src.v[0] = reinterpret_cast<const bf16*>(a.src.v);
  src.k[1] = reinterpret_cast<const bf16*>(a.k_priv); src.v[1] = reinterpret_cast<const bf16*>(a.v_priv);
  src.k[2] = reinterpret_cast<const bf16*>(a.k_new); src.v[2] = reinterpret_cast<const bf16*>(a.v_new);
  const bf16 *kg = src.k[0], *vg = src.v[0];

  // ---- per-warp cp.async ring.  A copy instruction moves 32 x 16 bytes = RPI whole rows.
  const uint32_t ring = ptx::smem_u32(smem) + warp * (STAGES * G::STAGE_B);
  const int ch = lane % CH, r0 = lane / CH;
  const uint32_t dst0 = (uint32_t)r0 * G::PITCH + (uint32_t)ch * 16;
  const int64_t rowstride = (int64_t)a.Hkv * D;   // elements between consecutive rows of a tensor
  // shared rows that are affine in the list position: row(p) = row_base + key_begin + p
  const bool affine = !a.src.paged || a.src.block_table == nullptr;
  const int64_t row_base = a.src.paged ? (int64_t)b * a.src.pages_per_seq * EARN_PAGE_TOKENS : (int64_t)seq_lo;
  const int64_t fast_off = ((row_base + key_begin + r0) * a.Hkv + kvh) * D + ch * 8;

  auto issue_tile = [&](int tile, int stage) {
    const uint32_t kdst = ring + stage * G::STAGE_B + dst0, vdst = kdst + G::TILE_B;
    if (affine && (tile + 1) * KT <= n_shared) {
      const bf16* ks = kg + fast_off + (int64_t)tile * KT * rowstride;
      const bf16* vs = vg + fast_off + (int64_t)tile * KT * rowstride;
#pragma unroll
      for (int i = 0; i < NIT; ++i) {
        cp_async16(kdst + i * RPI * G::PITCH, ks + i * RPI * rowstride);
        cp_async16(vdst + i * RPI * G::PITCH, vs + i * RPI * rowstride);
      }
      return;
    }
    // general tile: lane i resolves list position KT*tile + i to (tensor, element offset of its row)
    const int p = tile * KT + lane;
    int64_t off = -1;   // -1: no such position, the row is zero-filled
    int which = 0;      // 0 shared segment, 1 private segment, 2 this step's k_new / v_new
    if (lane >= KT) {
      // no row for this lane
    } else if (p < n_shared) {
      off = (key_row(a.src, b, key_begin + p) * a.Hkv + kvh) * D;
    } else if (p < n_total) {
      off = private_row<D>(a, b, kvh, w_lo, p - n_shared, which);
    }
    copy_resolved_tile<D>(ring + stage * G::STAGE_B, off, which, src, lane);
  };

  const int n_my = (n_tiles - warp + NWARPS - 1) / NWARPS;   // tiles warp, warp + NWARPS, ...
  // The one-warp streaming variant consumes its tiles two at a time (one softmax step per 32 positions): the two
  // tiles in use plus STAGES - 2 in flight.
  constexpr bool PAIR = WALK == STREAM;
  constexpr int PRE = PAIR ? STAGES - 2 : STAGES - 1;   // tiles in flight ahead of the one(s) in use
  // tiles that lie wholly in the shared segment may be fetched ahead of the wait
  auto ahead = [&](int s) { return early_fetch && s < n_my && (warp + s * NWARPS + 1) * KT <= n_shared; };
  if (early_fetch) {
#pragma unroll
    for (int s = 0; s < PRE; ++s)
      if (ahead(s)) issue_tile(warp + s * NWARPS, s);
    pdl_wait();   // q, k_new, v_new, the private segment and the lineage table are read from here on
    if (a.trigger_early) pdl_launch_dependents();
  }
#pragma unroll
  for (int s = 0; s < PRE; ++s) {
    if (s < n_my && !ahead(s)) issue_tile(warp + s * NWARPS, s);
    cp_async_commit();   // (the first group also holds every tile fetched ahead of the wait)
  }

  // ---- Q fragments, loaded while the first tiles are in flight
  RowTile<D> t;
  t.init(reinterpret_cast<const bf16*>(a.q), rm, lane);
  // Eq. 4 append: the new row is fetched here, behind the Q loads, and stored after the key loop, so that the round
  // trip of the fetch hides under the loop (7.9 -> 7.6 us per compact-cache layer at the 7B shapes, 11.9 -> 11.5 us
  // per prompt-cache layer at the 1.5B shapes).
  AppendOne<D> app;
  app.fetch(a, rm, threadIdx.x, NWARPS * 32, split == 0);
  // list positions of the generated tokens each of the lane's two rows may see: its own beam's `step` tokens
  const int vis0 = n_shared + ((row0 + (lane >> 2)) / g - w_lo) * step, vis1 = n_shared + ((row0 + (lane >> 2) + 8) / g - w_lo) * step;

  auto visible_in = [&](int tile) {
    return [=](int c, bool second) {
      const int p = tile * KT + c, v0 = second ? vis1 : vis0;
      return p < n_shared || (p >= v0 && p < v0 + step && p < n_total);
    };
  };
  if (PAIR) {
    for (int it = 0; it < n_my; it += 2) {
#pragma unroll
      for (int u = 0; u < 2; ++u) {   // into the two stages the previous round consumed (or that were never used)
        const int nxt = it + PRE + u;
        if (nxt < n_my) issue_tile(nxt, nxt % STAGES);
        cp_async_commit();
      }
      cp_async_wait<PRE>();           // this lane's copies of tiles it and it+1 have landed ...
      __syncwarp();                   // ... and so have every other lane's
      const uint32_t ks = ring + (it % STAGES) * G::STAGE_B, vs = ks + G::TILE_B;
      const uint32_t ks2 = ring + ((it + 1) % STAGES) * G::STAGE_B, vs2 = ks2 + G::TILE_B;
      if ((it + 2) * KT <= n_shared) {
        t.attend2(ks, vs, ks2, vs2, scale_log2, lane);
      } else {
        t.attend(ks, vs, scale_log2, lane, (it + 1) * KT > n_shared, visible_in(it));
        if (it + 1 < n_my) t.attend(ks2, vs2, scale_log2, lane, true, visible_in(it + 1));
      }
      __syncwarp();   // every lane is done with these stages before the next round refills them
    }
  }
  for (int it = 0; !PAIR && it < n_my; ++it) {
    const int stage = it % STAGES;
    {
      const int nxt = it + PRE;          // into a stage that is free (consumed PRE + 1 <= STAGES iterations back, or never used)
      if (nxt < n_my) issue_tile(warp + nxt * NWARPS, nxt % STAGES);
      cp_async_commit();
      cp_async_wait<PRE>();              // this lane's copies of tile `it` have landed ...
      __syncwarp();                      // ... and so have every other lane's
    }
    const int tile = warp + it * NWARPS;
    const uint32_t ks = ring + stage * G::STAGE_B, vs = ks + G::TILE_B;
    // positions past the list, and generated tokens of other beams, are invisible
    t.attend(ks, vs, scale_log2, lane, (tile + 1) * KT > n_shared, [&](int c, bool second) {
      const int p = tile * KT + c, v0 = second ? vis1 : vis0;
      return p < n_shared || (p >= v0 && p < v0 + step && p < n_total);
    });
    __syncwarp();   // every lane is done with this stage before the next iteration refills it
  }
  cp_async_wait<0>();
  // ---- Eq. 4: append.  Split 0 stores the new K/V row of every beam whose first query row is in this tile.  Nothing
  // in this launch reads those rows (the newest token came straight from k_new / v_new), so the store waits until
  // here: a whole load-then-store round trip ahead of the Q loads delayed them by more than a microsecond.
  if (app.single) app.store(a);
  else if (split == 0) append_new_rows<D>(a, rm, threadIdx.x, NWARPS * 32);
  // The next kernel on the stream may be scheduled from here on (once every CTA of this grid is past its key
  // loop): releasing it earlier let its CTAs pile up on whichever SMs had room and unbalanced the next launch
  // (55 us against 50 us per prompt-cache layer at the 7B shapes).
  if (!a.trigger_early) pdl_launch_dependents();
  t.reduce_sums();
  __syncthreads();   // all rings are idle: reuse the shared memory

  if (NWARPS == 1) {
    if (a.plan.n_splits <= 1) {
      t.store_rows(smem, reinterpret_cast<bf16*>(a.o), rm, lane);
    } else {
      const int live_splits = max(1, min(a.plan.n_splits, (shared_len + a.plan.chunk - 1) / a.plan.chunk));
      publish_and_fold<D>(t, a, rm, split, live_splits, row_tile, lane);
    }
    return;
  }

  // ---- several warps shared the key list (unsplit launches only): merge their states through shared memory
  float* mo = reinterpret_cast<float*>(smem);                 // [NWARPS][16][D]
  float* ml = mo + NWARPS * 16 * D;                           // [NWARPS][16][2] = (m, l)
  {
    const int c2 = (lane & 3) * 2, q0 = lane >> 2, q1 = q0 + 8;
    float* base = mo + warp * 16 * D;
#pragma unroll
    for (int n = 0; n < NTILES; ++n) {
      *reinterpret_cast<float2*>(base + q0 * D + n * 8 + c2) = make_float2(t.o[n][0], t.o[n][1]);
      *reinterpret_cast<float2*>(base + q1 * D + n * 8 + c2) = make_float2(t.o[n][2], t.o[n][3]);
    }
    if ((lane & 3) == 0) {
      ml[(warp * 16 + q0) * 2] = t.m0; ml[(warp * 16 + q0) * 2 + 1] = t.l0;
      ml[(warp * 16 + q1) * 2] = t.m1; ml[(warp * 16 + q1) * 2 + 1] = t.l1;
    }
  }
  __syncthreads();
  constexpr int GROUPS = NWARPS * 32 / 16;   // threads per row
  constexpr int COLS = D / GROUPS;           // columns per thread (a multiple of 8)
  static_assert(NWARPS == 1 || COLS % 8 == 0, "merge epilogue writes 8 bf16 at a time");
  const int r = threadIdx.x / GROUPS, cg = (threadIdx.x % GROUPS) * COLS;
  const int64_t off = rm.offset(row0 + r, D);
  if (off >= 0) {
    float big = -INFINITY;
#pragma unroll
    for (int w = 0; w < NWARPS; ++w) big = fmaxf(big, ml[(w * 16 + r) * 2]);
    float wt[NWARPS], den = 0.f;
#pragma unroll
    for (int w = 0; w < NWARPS; ++w) {
      wt[w] = exp2f(ml[(w * 16 + r) * 2] - big);   // a warp without keys has m = -inf -> weight 0
      den += wt[w] * ml[(w * 16 + r) * 2 + 1];
    }
    const float inv = 1.f / den;
    bf16* dst = reinterpret_cast<bf16*>(a.o) + off + cg;
#pragma unroll
    for (int c = 0; c < COLS; c += 8) {
      float out[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        float x = 0.f;
#pragma unroll
        for (int w = 0; w < NWARPS; ++w) x += wt[w] * mo[(w * 16 + r) * D + cg + c + e];
        out[e] = x * inv;
      }
      uint4 v;
      v.x = pack2(out[0], out[1]); v.y = pack2(out[2], out[3]);
      v.z = pack2(out[4], out[5]); v.w = pack2(out[6], out[7]);
      *reinterpret_cast<uint4*>(dst + c) = v;
    }
  }
}

#ifndef EARN_DECODE_EARLY_TRIGGER_TILES
#define EARN_DECODE_EARLY_TRIGGER_TILES 8
#endif

template <int D, int ST, int NWARPS, Walk WALK>
cudaError_t launch_d(const DecodeArgs& a, cudaStream_t st) {
  constexpr int smem = Smem<D, ST, NWARPS>::BYTES;
  cudaError_t e = ensure_dynamic_smem<decode_mma_kernel<D, ST, NWARPS, WALK>>(smem);
  if (e != cudaSuccess) return e;
  const int splits = a.plan.n_splits > 0 ? a.plan.n_splits : 1;
  dim3 grid(a.Hkv, splits * a.plan.row_tiles, a.batch);
  e = launch_pdl(decode_mma_kernel<D, ST, NWARPS, WALK>, grid, dim3(NWARPS * 32), smem, st, a);
  note_launch();
  return e != cudaSuccess ? e : cudaGetLastError();
}

// order[rank] = sequence, longest prompt first (ties by index): thread c counts the sequences ahead of sequence c
__global__ void __launch_bounds__(1024) decode_order_kernel(const int32_t* cu_seqlens, int batch, int32_t* order) {
  __shared__ int len[1024];
  pdl_wait();   // the table may still be read by the kernel before this one
  const int c = threadIdx.x;
  if (c < batch) len[c] = cu_seqlens[c + 1] - cu_seqlens[c];
  __syncthreads();
  pdl_launch_dependents();
  if (c >= batch) return;
  int ahead = 0;
  for (int j = 0; j < batch; ++j) ahead += (len[j] > len[c]) || (len[j] == len[c] && j < c);
  order[ahead] = c;
}

}  // namespace

cudaError_t launch_decode_order(const int32_t* cu_seqlens, int batch, int32_t* order, cudaStream_t st) {
  const cudaError_t e = launch_pdl(decode_order_kernel, dim3(1), dim3((batch + 31) / 32 * 32), 0, st, cu_seqlens, batch, order);
  note_launch();
  return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t launch_decode_mma(const DecodeArgs& a0, int max_shared_len, cudaStream_t st) {
  DecodeArgs a = a0;
  {
    // A launch whose CTAs each walk a short list is a chain of latencies (fetch, a few tiles, store), and the next
    // launch's CTAs fit beside it: let them start at once, so that whatever they may do ahead of their wait (set-up,
    // the fetch of their shared segment) runs under this launch.  A long list keeps the late trigger: there the CTAs
    // of the next launch would only take SM resources from this one's streams.
    const int gq = a.Hq / a.Hkv;
    const int per_tile = a.beams < (16 + gq - 1) / gq + 1 ? a.beams : (16 + gq - 1) / gq + 1;
    const int chunk_len = a.plan.n_splits > 1 ? a.plan.chunk : max_shared_len;
    a.trigger_early = (chunk_len + per_tile * a.step + KT - 1) / KT <= EARN_DECODE_EARLY_TRIGGER_TILES ? 1 : 0;
  }
  // A short list under one row tile (the compact cache of a register layer): the whole list at once, see decode_short.cu
  if (decode_short_supported(a, max_shared_len)) return launch_decode_short(a, max_shared_len, st);
  // Several row tiles (beams x group size > 16): the row tiles of a CTA share one pass over the shared segment.
  if (a.plan.row_tiles > 1) return launch_decode_rows(a, st);
  // One warp per CTA with a deep ring streams best whenever the grid covers the GPU (measured on B200 at the 7B
  // shapes: 8.9 us per compact-cache layer against 13.0 us with four warps).  A short key list on a grid of less
  // than a CTA per SM is latency-bound instead: four warps take a tile or two each (5.9 against 6.8 us at the 1.5B
  // shapes).
  const int g = a.Hq / a.Hkv;
  const int beams_per_tile = a.beams < (16 + g - 1) / g + 1 ? a.beams : (16 + g - 1) / g + 1;
  const int max_tiles = (max_shared_len + beams_per_tile * a.step + KT - 1) / KT;
  const long ctas = (long)(a.plan.n_splits > 0 ? a.plan.n_splits : 1) * a.plan.row_tiles * a.Hkv * a.batch;
  const bool unsplit = a.plan.n_splits <= 1;
  const bool four_warps = unsplit && max_tiles <= 16 && ctas < sm_count();
  // a longer list on such a grid (the planner leaves it unsplit up to kDecodeUnsplitMaxLen shared positions): eight warps
  const bool eight_warps = unsplit && !four_warps && ctas < sm_count() && max_shared_len <= kDecodeUnsplitMaxLen;
  // a list of one or two tiles goes into a three-stage ring whole; anything longer is walked in pairs
  const bool two_tiles = unsplit && max_tiles <= 2;
  if (a.D == 64)
    return four_warps  ? launch_d<64, 2, 4, SHARED>(a, st)   // (the planner only leaves such a list unsplit at head_dim 128)
           : two_tiles ? launch_d<64, 3, 1, SHORT>(a, st)
                        : launch_d<64, EARN_DECODE_STAGES, 1, STREAM>(a, st);
  return four_warps    ? launch_d<128, 2, 4, SHARED>(a, st)
         : eight_warps ? launch_d<128, 2, 8, SHARED>(a, st)
         : two_tiles   ? launch_d<128, 3, 1, SHORT>(a, st)
                      : launch_d<128, EARN_DECODE_STAGES, 1, STREAM>(a, st);
}

}  // namespace earn
