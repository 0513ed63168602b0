// Decode attention (Eq. 4: append K_t, V_t, then attend over K_{1:t}) for bf16 caches.
//
// HBM-bound: every byte of the cache is read once per step, so the kernel is built around keeping
// loads in flight with few instructions, not around the tensor cores; warp-level mma.sync (m16n8k16)
// only keeps the few query rows per key (g heads x W beams, padded to 16) off the FMA pipe.
//
// One CTA = (sequence b, kv head, split of the shared segment, tile of 16 query rows); one warp, or four
// warps that deal the tiles of a short list among themselves when the grid is small.  The key
// list of a CTA is its chunk of the shared segment (the prompt K/V of a layer l < k read in place, or
// the compact register pages of a layer l >= k) followed -- in split 0 only -- by the generated tokens
// of the beams its rows belong to (masked per row to the row's own beam; the newest token comes
// straight from k_new / v_new, which split 0 also appends to the private segment).
//
// The list is cut into tiles of 16 positions.  The warp fetches them with 16-byte cp.async copies into
// padded shared-memory tiles (a ring of four stages = 35 KB at head_dim 128, so six CTAs share an SM; two
// stages for lists of at most two tiles).  Tile size, warps per CTA and ring depth were swept on B200 at
// the 7B shapes: (16, 1, 4) gave 50.9 us per layer against 51.3-63.4 us for the other combinations.
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
#include "earn_common.cuh"
#include "mma_sync.cuh"
#include "sm100_ptx.cuh"

namespace earn {
namespace {
using namespace mma;

#ifndef EARN_DECODE_KT
#define EARN_DECODE_KT 16
#endif
#ifndef EARN_DECODE_STAGES
#define EARN_DECODE_STAGES 4
#endif
constexpr int KT = EARN_DECODE_KT;           // list positions per tile (16 or 32)
constexpr int N8 = KT / 8, H16 = KT / 16;

template <int D, int STAGES, int NWARPS>   // STAGES: cp.async ring depth per warp; NWARPS: warps per CTA, tiles dealt round-robin
struct Geo {
  static constexpr int ROWB = D * 2;            // bytes of one K (or V) row
  static constexpr int PITCH = ROWB + 16;       // padded row pitch: conflict-free ldmatrix, 16-byte aligned
  static constexpr int TILE_B = KT * PITCH;     // one K (or V) tile
  static constexpr int STAGE_B = 2 * TILE_B;    // K tile + V tile
  static constexpr int RING_B = NWARPS * STAGES * STAGE_B;
  static constexpr int MERGE_B = NWARPS * 16 * D * 4 + NWARPS * 16 * 2 * 4 + 16;
  static constexpr int DATA_B = RING_B > MERGE_B ? RING_B : MERGE_B;
  static constexpr int SMEM_B = DATA_B;
};

template <int D, int STAGES, int NWARPS>
__global__ void __launch_bounds__(NWARPS * 32) decode_mma_kernel(DecodeArgs a) {
  using bf16 = __nv_bfloat16;
  using G = Geo<D, STAGES, NWARPS>;
  constexpr int KSTEPS = D / 16, NTILES = D / 8;
  extern __shared__ __align__(128) uint8_t smem[];
  pdl_wait();   // everything below reads or writes global memory

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // kv heads vary fastest over the grid: the CTAs that read the same rows of the packed K/V tensors (one 256-byte
  // slice each of a 2 KB row) start next to each other and walk those rows together
  const int b = blockIdx.z, kvh = blockIdx.x;
  const int row_tiles = a.plan.row_tiles;
  const int split = blockIdx.y / row_tiles, row0 = (blockIdx.y % row_tiles) * 16;
  const int g = a.Hq / a.Hkv, W = a.beams, n_rows = W * g, step = a.step;
  const int seq_lo = a.src.paged ? 0 : a.cu_seqlens[b];
  const int shared_len = a.src.paged ? a.src.n_regs : (a.cu_seqlens[b + 1] - seq_lo);
  const int key_begin = split * a.plan.chunk;
  const int n_shared = max(min(key_begin + a.plan.chunk, shared_len) - key_begin, 0);
  const int w_lo = row0 / g, w_hi = min((row0 + 15) / g, W - 1);
  const int n_priv = (split == 0) ? (w_hi - w_lo + 1) * step : 0;
  const int n_total = n_shared + n_priv;
  if (n_total == 0) return;
  const int n_tiles = (n_total + KT - 1) / KT;
  const float scale_log2 = a.scale * kLog2e;

  const bf16* kg = reinterpret_cast<const bf16*>(a.src.k);
  const bf16* vg = reinterpret_cast<const bf16*>(a.src.v);
  bf16* kp = reinterpret_cast<bf16*>(a.k_priv);
  bf16* vp = reinterpret_cast<bf16*>(a.v_priv);
  const bf16* kn = reinterpret_cast<const bf16*>(a.k_new);
  const bf16* vn = reinterpret_cast<const bf16*>(a.v_new);

  // ---- per-warp cp.async ring.  A copy instruction moves 32 x 16 bytes = RPI whole rows.
  constexpr int CH = G::ROWB / 16, RPI = 32 / CH, NIT = KT / RPI;
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
    // general tile: lane i resolves list position 32*tile + i to (tensor, element offset of its row)
    const int p = tile * KT + lane;
    int64_t off = -1;   // -1: no such position, the row is zero-filled
    int which = 0;      // 0 shared segment, 1 private segment, 2 this step's k_new / v_new
    if (lane >= KT) {
      // no row for this lane in a tile of fewer than 32 positions
    } else if (p < n_shared) {
      off = (key_row(a.src, b, key_begin + p) * a.Hkv + kvh) * D;
    } else if (p < n_total) {
      const int pk = p - n_shared, w = w_lo + pk / step, t = pk % step;
      const int64_t j = (int64_t)b * W + w;
      if (t == step - 1) {
        which = 2;
        off = (j * a.Hkv + kvh) * D;
      } else {
        int64_t slab = j;
        if (a.lineage) slab = min(max(a.lineage[j * a.max_new + t], 0), a.batch * W - 1);
        which = 1;
        off = ((slab * a.max_new + t) * a.Hkv + kvh) * D;
      }
    }
#pragma unroll
    for (int i = 0; i < NIT; ++i) {
      const int64_t o_r = __shfl_sync(0xffffffffu, off, r0 + i * RPI);
      const int w_r = __shfl_sync(0xffffffffu, which, r0 + i * RPI);
      const bf16* ks = (w_r == 0 ? kg : w_r == 1 ? kp : kn) + (o_r < 0 ? 0 : o_r) + ch * 8;
      const bf16* vs = (w_r == 0 ? vg : w_r == 1 ? vp : vn) + (o_r < 0 ? 0 : o_r) + ch * 8;
      const int bytes = o_r < 0 ? 0 : 16;   // 0: nothing is read, the 16 destination bytes become zero
      cp_async16(kdst + i * RPI * G::PITCH, ks, bytes);
      cp_async16(vdst + i * RPI * G::PITCH, vs, bytes);
    }
  };

  const int n_my = (n_tiles - warp + NWARPS - 1) / NWARPS;   // tiles warp, warp + NWARPS, ...
#pragma unroll
  for (int s = 0; s < STAGES - 1; ++s) {
    if (s < n_my) issue_tile(warp + s * NWARPS, s);
    cp_async_commit();
  }

  // ---- Eq. 4: append.  Split 0 stores the new K/V row of every beam whose first query row is in this tile.
  if (split == 0) {
    constexpr int CH = G::ROWB / 16;
    for (int w = w_lo; w <= w_hi; ++w) {
      if (w * g < row0) continue;   // that beam's first row belongs to the previous row tile
      const int64_t j = (int64_t)b * W + w;
      const int64_t src = (j * a.Hkv + kvh) * D, dst = ((j * a.max_new + (step - 1)) * a.Hkv + kvh) * D;
      for (int i = threadIdx.x; i < 2 * CH; i += NWARPS * 32) {
        const bf16* s = (i < CH ? kn : vn) + src + (i % CH) * 8;
        bf16* d = (i < CH ? kp : vp) + dst + (i % CH) * 8;
        *reinterpret_cast<uint4*>(d) = *reinterpret_cast<const uint4*>(s);
      }
    }
  }

  // ---- Q fragments (A operand, 16 rows x D), loaded while the first tiles are in flight; rows >= W*g are zero
  const int c2 = (lane & 3) * 2;
  const int rr0 = row0 + (lane >> 2), rr1 = rr0 + 8;
  const int beam0 = rr0 / g, beam1 = rr1 / g;
  uint32_t qf[KSTEPS][4];
  {
    const bf16* qg = reinterpret_cast<const bf16*>(a.q);
    auto qrow = [&](int rr) -> const bf16* {
      if (rr >= n_rows) return nullptr;
      return qg + (((int64_t)b * W + rr / g) * a.Hq + kvh * g + rr % g) * D;
    };
    const bf16 *q0 = qrow(rr0), *q1 = qrow(rr1);
#pragma unroll
    for (int kk = 0; kk < KSTEPS; ++kk) {
      qf[kk][0] = q0 ? *reinterpret_cast<const uint32_t*>(q0 + kk * 16 + c2) : 0u;
      qf[kk][1] = q1 ? *reinterpret_cast<const uint32_t*>(q1 + kk * 16 + c2) : 0u;
      qf[kk][2] = q0 ? *reinterpret_cast<const uint32_t*>(q0 + kk * 16 + 8 + c2) : 0u;
      qf[kk][3] = q1 ? *reinterpret_cast<const uint32_t*>(q1 + kk * 16 + 8 + c2) : 0u;
    }
  }

  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;   // running max in the scaled log2 domain
  float o[NTILES][4];
#pragma unroll
  for (int n = 0; n < NTILES; ++n) { o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f; }

  // ldmatrix lane addressing inside a tile (rows = keys, 16-byte chunks along d)
  const int mat = lane >> 3;
  const uint32_t k_lane = (uint32_t)(((mat >> 1) << 3) + (lane & 7)) * G::PITCH + (uint32_t)(mat & 1) * 16;
  const uint32_t v_lane = (uint32_t)(((mat & 1) << 3) + (lane & 7)) * G::PITCH + (uint32_t)(mat >> 1) * 16;

  for (int it = 0; it < n_my; ++it) {
    const int stage = it % STAGES;
    {
      const int nxt = it + STAGES - 1;   // refill the stage that was consumed in the previous iteration
      if (nxt < n_my) issue_tile(warp + nxt * NWARPS, nxt % STAGES);
      cp_async_commit();
      cp_async_wait<STAGES - 1>();       // this lane's copies of tile `it` have landed ...
      __syncwarp();                      // ... and so have every other lane's
    }
    const int tile = warp + it * NWARPS;
    const uint32_t ks = ring + stage * G::STAGE_B, vs = ks + G::TILE_B;

    // S = Q K^T for KT positions: n-tiles of 8
    float s[N8][4];
#pragma unroll
    for (int n = 0; n < N8; ++n) { s[n][0] = s[n][1] = s[n][2] = s[n][3] = 0.f; }
#pragma unroll
    for (int kk = 0; kk < KSTEPS; ++kk) {
#pragma unroll
      for (int h16 = 0; h16 < H16; ++h16) {
        uint32_t b0, b1, b2, b3;
        ldsm_x4(ks + k_lane + h16 * 16 * G::PITCH + kk * 32, b0, b1, b2, b3);
        mma_bf16(s[2 * h16], qf[kk], b0, b1);
        mma_bf16(s[2 * h16 + 1], qf[kk], b2, b3);
      }
    }
    // positions past the list, and generated tokens of other beams, are invisible
    if ((tile + 1) * KT > n_shared) {
#pragma unroll
      for (int n = 0; n < N8; ++n)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int p = tile * KT + n * 8 + c2 + (e & 1);
          bool vis = p < n_total;
          if (p >= n_shared) vis = vis && (w_lo + (p - n_shared) / step) == ((e < 2) ? beam0 : beam1);
          if (!vis) s[n][e] = -INFINITY;
        }
    }
    float mx0 = fmaxf(s[0][0], s[0][1]), mx1 = fmaxf(s[0][2], s[0][3]);
#pragma unroll
    for (int n = 1; n < N8; ++n) {
      mx0 = fmaxf(mx0, fmaxf(s[n][0], s[n][1]));
      mx1 = fmaxf(mx1, fmaxf(s[n][2], s[n][3]));
    }
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
    const float mn0 = fmaxf(m0, mx0 * scale_log2), mn1 = fmaxf(m1, mx1 * scale_log2);
    const float mu0 = (mn0 == -INFINITY) ? 0.f : mn0, mu1 = (mn1 == -INFINITY) ? 0.f : mn1;
    const float al0 = ex2(m0 - mu0), al1 = ex2(m1 - mu1);
    const bool grew = (mn0 != m0) || (mn1 != m1);
    m0 = mn0; m1 = mn1;
    uint32_t pf[H16][4];
    {
      float sum0 = 0.f, sum1 = 0.f;
#pragma unroll
      for (int n = 0; n < N8; ++n) {
        const float p0 = ex2(fmaf(s[n][0], scale_log2, -mu0)), p1 = ex2(fmaf(s[n][1], scale_log2, -mu0));
        const float p2 = ex2(fmaf(s[n][2], scale_log2, -mu1)), p3 = ex2(fmaf(s[n][3], scale_log2, -mu1));
        sum0 += p0 + p1; sum1 += p2 + p3;
        pf[n >> 1][(n & 1) * 2] = pack2(p0, p1);
        pf[n >> 1][(n & 1) * 2 + 1] = pack2(p2, p3);
      }
      l0 = l0 * al0 + sum0;   // per-lane partial sums; reduced over the quad at the end
      l1 = l1 * al1 + sum1;
    }
    if (__any_sync(0xffffffffu, grew)) {
#pragma unroll
      for (int n = 0; n < NTILES; ++n) { o[n][0] *= al0; o[n][1] *= al0; o[n][2] *= al1; o[n][3] *= al1; }
    }
    // O += P V
#pragma unroll
    for (int h16 = 0; h16 < H16; ++h16) {
#pragma unroll
      for (int nn = 0; nn < NTILES / 2; ++nn) {
        uint32_t b0, b1, b2, b3;
        ldsm_x4_t(vs + v_lane + h16 * 16 * G::PITCH + nn * 32, b0, b1, b2, b3);
        mma_bf16(o[2 * nn], pf[h16], b0, b1);
        mma_bf16(o[2 * nn + 1], pf[h16], b2, b3);
      }
    }
    __syncwarp();   // every lane is done with this stage before the next iteration refills it
  }
  cp_async_wait<0>();
  // The next kernel on the stream may be scheduled from here on (once every CTA of this grid is past its key
  // loop): releasing it earlier let its CTAs pile up on whichever SMs had room and unbalanced the next launch
  // (55 us against 50 us per prompt-cache layer at the 7B shapes).
  pdl_launch_dependents();
  l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
  l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
  __syncthreads();   // all rings are idle: reuse the shared memory for the merge

  if (NWARPS == 1 && a.plan.n_splits <= 1) {
    // one warp saw the whole key list: normalise, stage the 16 x D bf16 tile, 16-byte stores
    const float i0 = 1.f / l0, i1 = 1.f / l1;   // rows past W*g hold garbage and are not stored
    const int r0 = lane >> 2, r1 = r0 + 8;
#pragma unroll
    for (int n = 0; n < NTILES; ++n) {
      *reinterpret_cast<uint32_t*>(smem + r0 * G::PITCH + (n * 8 + c2) * 2) = pack2(o[n][0] * i0, o[n][1] * i0);
      *reinterpret_cast<uint32_t*>(smem + r1 * G::PITCH + (n * 8 + c2) * 2) = pack2(o[n][2] * i1, o[n][3] * i1);
    }
    const int rr = row0 + (lane & 15);   // lane r (and r + 16) resolves output row r; the store loop fetches it by shuffle
    const int64_t my_off = rr < n_rows ? (((int64_t)b * W + rr / g) * a.Hq + kvh * g + rr % g) * D : -1;
    __syncwarp();
    bf16* og = reinterpret_cast<bf16*>(a.o);
#pragma unroll
    for (int it = 0; it < 16 / RPI; ++it) {
      const int r = it * RPI + lane / CH, chunk = lane % CH;
      const int64_t off = __shfl_sync(0xffffffffu, my_off, r);
      if (off >= 0)
        *reinterpret_cast<uint4*>(og + off + chunk * 8) = *reinterpret_cast<const uint4*>(smem + r * G::PITCH + chunk * 16);
    }
    return;
  }

  if (NWARPS == 1) {
    // ---- split-KV, one warp: publish this split's normalised partial rows straight from the accumulator
    // fragments, take a ticket, and let the warp that holds the last ticket of its (sequence, kv head, row tile)
    // fold all partials.  No CTA waits for another.  The fold walks the splits once, four at a time with all
    // their loads in flight together, keeping a running maximum (what one thread per row walking the splits in
    // two passes cost: 6 to 13 us of L2 round trips at 8 to 13 splits).
    const int r0 = lane >> 2, r1 = r0 + 8;
    const int64_t prow0 = ((int64_t)(b * a.Hkv + kvh) * a.plan.n_splits + split) * a.plan.rows_pad + row0;
    {
      const float i0 = 1.f / l0, i1 = 1.f / l1;
      float* p0 = a.part_o + (prow0 + r0) * D + c2;
      float* p1 = a.part_o + (prow0 + r1) * D + c2;
      if (row0 + r0 < n_rows) {
#pragma unroll
        for (int n = 0; n < NTILES; ++n) *reinterpret_cast<float2*>(p0 + n * 8) = make_float2(o[n][0] * i0, o[n][1] * i0);
        if ((lane & 3) == 0) a.part_lse[prow0 + r0] = m0 + log2f(l0);
      }
      if (row0 + r1 < n_rows) {
#pragma unroll
        for (int n = 0; n < NTILES; ++n) *reinterpret_cast<float2*>(p1 + n * 8) = make_float2(o[n][2] * i1, o[n][3] * i1);
        if ((lane & 3) == 0) a.part_lse[prow0 + r1] = m1 + log2f(l1);
      }
    }
    __threadfence();
    __syncwarp();
    const int live_splits = max(1, min(a.plan.n_splits, (shared_len + a.plan.chunk - 1) / a.plan.chunk));
    int last = 0;
    if (lane == 0) {
      int32_t* ticket = a.tickets + ((int64_t)(b * a.Hkv + kvh) * row_tiles + blockIdx.y % row_tiles);
      const int t = atomicAdd(ticket, 1);
      last = (t == live_splits - 1);
      if (last) *ticket = 0;   // ready for the next launch on this stream
    }
    if (!__shfl_sync(0xffffffffu, last, 0)) return;
    __threadfence();
    constexpr int V4 = D / 4, RPP = 4 * 32 / V4;   // float4 per row; rows per pass (4 float4 per lane)
    const int live_rows = min(16, n_rows - row0);
    const int64_t fold0 = (int64_t)(b * a.Hkv + kvh) * a.plan.n_splits * a.plan.rows_pad + row0;   // split 0, first row
    bf16* og = reinterpret_cast<bf16*>(a.o);
    for (int rbase = 0; rbase < live_rows; rbase += RPP) {
      float4 acc[4];
      float mx[4], den[4];
      int rk[4], ck[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int idx = lane + 32 * k;
        rk[k] = rbase + idx / V4;
        ck[k] = idx % V4;
        acc[k] = make_float4(0.f, 0.f, 0.f, 0.f);
        mx[k] = -INFINITY;
        den[k] = 0.f;
      }
      for (int s0 = 0; s0 < live_splits; s0 += 4) {
        float lse_b[4][4];
        float4 x_b[4][4];
#pragma unroll
        for (int u = 0; u < 4; ++u)
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const bool ok = s0 + u < live_splits && rk[k] < live_rows;
            const int64_t prow = fold0 + (int64_t)(s0 + u) * a.plan.rows_pad + rk[k];
            lse_b[u][k] = ok ? __ldcg(a.part_lse + prow) : -INFINITY;
            x_b[u][k] = ok ? __ldcg(reinterpret_cast<const float4*>(a.part_o + prow * D) + ck[k]) : make_float4(0.f, 0.f, 0.f, 0.f);
          }
#pragma unroll
        for (int u = 0; u < 4; ++u)
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const float mn = fmaxf(mx[k], lse_b[u][k]);
            const float sc = mn == -INFINITY ? 1.f : exp2f(mx[k] - mn), wt = mn == -INFINITY ? 0.f : exp2f(lse_b[u][k] - mn);
            acc[k].x = acc[k].x * sc + wt * x_b[u][k].x;
            acc[k].y = acc[k].y * sc + wt * x_b[u][k].y;
            acc[k].z = acc[k].z * sc + wt * x_b[u][k].z;
            acc[k].w = acc[k].w * sc + wt * x_b[u][k].w;
            den[k] = den[k] * sc + wt;
            mx[k] = mn;
          }
      }
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        if (rk[k] < live_rows) {
          const int rr = row0 + rk[k];
          const float inv = 1.f / den[k];
          uint2 v;
          v.x = pack2(acc[k].x * inv, acc[k].y * inv);
          v.y = pack2(acc[k].z * inv, acc[k].w * inv);
          *reinterpret_cast<uint2*>(og + (((int64_t)b * W + rr / g) * a.Hq + kvh * g + rr % g) * D + ck[k] * 4) = v;
        }
      }
    }
    return;
  }

  float* mo = reinterpret_cast<float*>(smem);                 // [NWARPS][16][D]
  float* ml = mo + NWARPS * 16 * D;                           // [NWARPS][16][2] = (m, l)
  {
    const int r0 = lane >> 2, r1 = r0 + 8;
    float* base = mo + warp * 16 * D;
#pragma unroll
    for (int n = 0; n < NTILES; ++n) {
      *reinterpret_cast<float2*>(base + r0 * D + n * 8 + c2) = make_float2(o[n][0], o[n][1]);
      *reinterpret_cast<float2*>(base + r1 * D + n * 8 + c2) = make_float2(o[n][2], o[n][3]);
    }
    if ((lane & 3) == 0) {
      ml[(warp * 16 + r0) * 2] = m0; ml[(warp * 16 + r0) * 2 + 1] = l0;
      ml[(warp * 16 + r1) * 2] = m1; ml[(warp * 16 + r1) * 2 + 1] = l1;
    }
  }
  __syncthreads();
  {
    constexpr int GROUPS = NWARPS * 32 / 16;   // threads per row
    constexpr int COLS = D / GROUPS;           // columns per thread (a multiple of 8)
    static_assert(COLS % 8 == 0, "merge epilogue writes 8 bf16 at a time");
    const int r = threadIdx.x / GROUPS, cg = (threadIdx.x % GROUPS) * COLS;
    const int rr = row0 + r;
    if (rr < n_rows) {
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
      float out[COLS];
#pragma unroll
      for (int c = 0; c < COLS; ++c) {
        float x = 0.f;
#pragma unroll
        for (int w = 0; w < NWARPS; ++w) x += wt[w] * mo[(w * 16 + r) * D + cg + c];
        out[c] = x * inv;
      }
      if (a.plan.n_splits <= 1) {
        bf16* dst = reinterpret_cast<bf16*>(a.o) + (((int64_t)b * W + rr / g) * a.Hq + kvh * g + rr % g) * D + cg;
#pragma unroll
        for (int c = 0; c < COLS; c += 8) {
          uint4 v;
          v.x = pack2(out[c], out[c + 1]); v.y = pack2(out[c + 2], out[c + 3]);
          v.z = pack2(out[c + 4], out[c + 5]); v.w = pack2(out[c + 6], out[c + 7]);
          *reinterpret_cast<uint4*>(dst + c) = v;
        }
      } else {
        const int64_t prow = ((int64_t)(b * a.Hkv + kvh) * a.plan.n_splits + split) * a.plan.rows_pad + rr;
        float* dst = a.part_o + prow * D + cg;
#pragma unroll
        for (int c = 0; c < COLS; c += 4) *reinterpret_cast<float4*>(dst + c) = make_float4(out[c], out[c + 1], out[c + 2], out[c + 3]);
        if (threadIdx.x % GROUPS == 0) a.part_lse[prow] = big + log2f(den);
      }
    }
    if (a.plan.n_splits <= 1) return;

    // ---- the split that finishes last folds all partials of this (sequence, kv head, row tile).
    // No CTA waits for another: each publishes its partial, takes a ticket, and only the holder of the
    // last ticket reads the others' partials (which its ticket proves complete).
    __threadfence();
    __syncthreads();
    int* is_last = reinterpret_cast<int*>(ml + NWARPS * 16 * 2);
    int32_t* ticket = a.tickets + ((int64_t)(b * a.Hkv + kvh) * row_tiles + blockIdx.y % row_tiles);
    const int live_splits = max(1, min(a.plan.n_splits, (shared_len + a.plan.chunk - 1) / a.plan.chunk));
    if (threadIdx.x == 0) {
      const int t = atomicAdd(ticket, 1);
      *is_last = (t == live_splits - 1);
      if (t == live_splits - 1) *ticket = 0;   // ready for the next launch on this stream
    }
    __syncthreads();
    if (!*is_last) return;
    __threadfence();
    // Fold: every thread of the CTA works on the valid rows of the tile (W*g is often 4 or 6 of the 16), a
    // float4 at a time, with the loads of several splits in flight at once -- one thread per row walking the
    // splits one after the other cost about 10 us of L2 round trips at 8 to 13 splits.
    __syncthreads();   // `mo` / `ml` are free again
    constexpr int NT = NWARPS * 32, V4 = D / 4;
    const int live_rows = min(16, n_rows - row0);
    const int64_t prow0 = (int64_t)(b * a.Hkv + kvh) * a.plan.n_splits * a.plan.rows_pad + row0;
    float* top_s = mo;          // [16] row maximum of the split LSEs
    float* inv_s = mo + 16;     // [16] 1 / sum of the split weights
    for (int r = threadIdx.x; r < live_rows; r += NT) {
      float top = -INFINITY, den = 0.f;
#pragma unroll 8
      for (int s = 0; s < live_splits; ++s) top = fmaxf(top, __ldcg(a.part_lse + prow0 + (int64_t)s * a.plan.rows_pad + r));
#pragma unroll 8
      for (int s = 0; s < live_splits; ++s) den += exp2f(__ldcg(a.part_lse + prow0 + (int64_t)s * a.plan.rows_pad + r) - top);
      top_s[r] = top;
      inv_s[r] = 1.f / den;
    }
    __syncthreads();
    bf16* og = reinterpret_cast<bf16*>(a.o);
    for (int idx = threadIdx.x; idx < live_rows * V4; idx += NT) {
      const int r = idx / V4, c4 = idx % V4, rr = row0 + r;
      const float top = top_s[r];
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 8
      for (int s = 0; s < live_splits; ++s) {
        const int64_t prow = prow0 + (int64_t)s * a.plan.rows_pad + r;
        const float wt = exp2f(__ldcg(a.part_lse + prow) - top);
        const float4 x = __ldcg(reinterpret_cast<const float4*>(a.part_o + prow * D) + c4);
        acc.x += wt * x.x; acc.y += wt * x.y; acc.z += wt * x.z; acc.w += wt * x.w;
      }
      const float inv = inv_s[r];
      uint2 v;
      v.x = pack2(acc.x * inv, acc.y * inv);
      v.y = pack2(acc.z * inv, acc.w * inv);
      *reinterpret_cast<uint2*>(og + (((int64_t)b * W + rr / g) * a.Hq + kvh * g + rr % g) * D + c4 * 4) = v;
    }
  }
}

template <int D, int ST, int NWARPS>
cudaError_t launch_d(const DecodeArgs& a, cudaStream_t st) {
  constexpr int smem = Geo<D, ST, NWARPS>::SMEM_B;
  cudaError_t e = ensure_dynamic_smem<decode_mma_kernel<D, ST, NWARPS>>(smem);
  if (e != cudaSuccess) return e;
  const int splits = a.plan.n_splits > 0 ? a.plan.n_splits : 1;
  dim3 grid(a.Hkv, splits * a.plan.row_tiles, a.batch);
  e = launch_pdl(decode_mma_kernel<D, ST, NWARPS>, grid, dim3(NWARPS * 32), smem, st, a);
  note_launch();
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace

cudaError_t launch_decode_mma(const DecodeArgs& a, int max_shared_len, cudaStream_t st) {
  // One warp per CTA with a deep ring streams best whenever the grid covers the GPU (measured on B200 at the 7B
  // shapes: 8.9 us per compact-cache layer against 13.0 us with four warps).  A short key list on a grid of less
  // than a CTA per SM is latency-bound instead: four warps take a tile or two each (5.9 against 6.8 us at the 1.5B
  // shapes).  A list of at most two tiles needs no deep ring either way.
  const int g = a.Hq / a.Hkv;
  const int beams_per_tile = a.beams < (16 + g - 1) / g + 1 ? a.beams : (16 + g - 1) / g + 1;
  const int max_tiles = (max_shared_len + beams_per_tile * a.step + KT - 1) / KT;
  const long ctas = (long)(a.plan.n_splits > 0 ? a.plan.n_splits : 1) * a.plan.row_tiles * a.Hkv * a.batch;
  const bool unsplit = a.plan.n_splits <= 1;
  const bool four_warps = unsplit && max_tiles <= 16 && ctas < 148;
  const bool small = unsplit && max_tiles <= 2;
  if (a.D == 64)
    return four_warps ? launch_d<64, 2, 4>(a, st) : small ? launch_d<64, 2, 1>(a, st) : launch_d<64, EARN_DECODE_STAGES, 1>(a, st);
  return four_warps ? launch_d<128, 2, 4>(a, st) : small ? launch_d<128, 2, 1>(a, st) : launch_d<128, EARN_DECODE_STAGES, 1>(a, st);
}

}  // namespace earn
