// Warp-level pieces shared by the decode kernels (Eq. 4 attention of 16 query rows against tiles of 16 cache
// positions held in shared memory): the online-softmax tile update on mma.sync m16n8k16, and the two ways a warp
// finishes -- writing its rows, or publishing a split-KV partial and folding all partials if it came last.
#pragma once
#include "earn_common.cuh"
#include "mma_sync.cuh"

namespace earn {
namespace dec {
using namespace mma;
using bf16 = __nv_bfloat16;

constexpr int KT = 16;   // cache positions per tile

template <int D>
struct Geo {
  static constexpr int ROWB = D * 2;            // bytes of one K (or V) row
  static constexpr int PITCH = ROWB + 16;       // padded row pitch: conflict-free ldmatrix, 16-byte aligned
  static constexpr int TILE_B = KT * PITCH;     // one K (or V) tile
  static constexpr int STAGE_B = 2 * TILE_B;    // K tile + V tile
  static constexpr int CH = ROWB / 16;          // 16-byte chunks per row
  static constexpr int RPI = 32 / CH;           // rows one 16-byte access of a whole warp covers
};

// Which query rows a warp owns: rows row0 .. row0+15 of the W*g rows of one (sequence, kv head);
// row rr is beam rr / g, head kvh*g + rr % g.
struct RowMap {
  int b, kvh, row0, n_rows, g, W, Hq;
  __device__ __forceinline__ int64_t offset(int rr, int D) const {   // element offset of row rr in q / o, -1 if absent
    return rr < n_rows ? (((int64_t)b * W + rr / g) * Hq + kvh * g + rr % g) * D : -1;
  }
};

// One warp's 16 query rows: Q fragments, running maximum / sum (scaled log2 domain) and the output accumulator.
// Lane l holds rows l/4 and l/4 + 8, columns 2*(l%4) + {0,1} of every 8-column block.
template <int D>
struct RowTile {
  static constexpr int KSTEPS = D / 16, NTILES = D / 8;
  uint32_t qf[KSTEPS][4];
  float m0, m1, l0, l1;
  float o[NTILES][4];

  __device__ __forceinline__ void init(const bf16* q, const RowMap& rm, int lane) {
    const int c2 = (lane & 3) * 2;
    const int64_t off0 = rm.offset(rm.row0 + (lane >> 2), D), off1 = rm.offset(rm.row0 + (lane >> 2) + 8, D);
#pragma unroll
    for (int kk = 0; kk < KSTEPS; ++kk) {   // rows past W*g are zero
      qf[kk][0] = off0 >= 0 ? *reinterpret_cast<const uint32_t*>(q + off0 + kk * 16 + c2) : 0u;
      qf[kk][1] = off1 >= 0 ? *reinterpret_cast<const uint32_t*>(q + off1 + kk * 16 + c2) : 0u;
      qf[kk][2] = off0 >= 0 ? *reinterpret_cast<const uint32_t*>(q + off0 + kk * 16 + 8 + c2) : 0u;
      qf[kk][3] = off1 >= 0 ? *reinterpret_cast<const uint32_t*>(q + off1 + kk * 16 + 8 + c2) : 0u;
    }
    m0 = m1 = -INFINITY;
    l0 = l1 = 0.f;
#pragma unroll
    for (int n = 0; n < NTILES; ++n) o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f;
  }

  // One tile of KT positions: S = Q K^T, online softmax, O += P V.  ks / vs: shared-memory addresses of the K and V
  // tiles.  When `masked`, visible(column, second_row) says whether position `column` of the tile counts for the
  // lane's first (false) or second (true) row.
  template <typename Vis>
  __device__ __forceinline__ void attend(uint32_t ks, uint32_t vs, float scale_log2, int lane, bool masked, Vis visible) {
    constexpr int PITCH = Geo<D>::PITCH;
    const int c2 = (lane & 3) * 2, mat = lane >> 3;
    const uint32_t k_lane = (uint32_t)(((mat >> 1) << 3) + (lane & 7)) * PITCH + (uint32_t)(mat & 1) * 16;
    const uint32_t v_lane = (uint32_t)(((mat & 1) << 3) + (lane & 7)) * PITCH + (uint32_t)(mat >> 1) * 16;
    // two accumulator sets per 8-column block (even / odd k-steps) halve the chain of dependent MMAs
    float s[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}}, s2[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
    for (int kk = 0; kk < KSTEPS; kk += 2) {
      uint32_t b0, b1, b2, b3, c0, c1, c2_, c3;
      ldsm_x4(ks + k_lane + kk * 32, b0, b1, b2, b3);
      ldsm_x4(ks + k_lane + (kk + 1) * 32, c0, c1, c2_, c3);
      mma_bf16(s[0], qf[kk], b0, b1);
      mma_bf16(s[1], qf[kk], b2, b3);
      mma_bf16(s2[0], qf[kk + 1], c0, c1);
      mma_bf16(s2[1], qf[kk + 1], c2_, c3);
    }
#pragma unroll
    for (int n = 0; n < 2; ++n)
#pragma unroll
      for (int e = 0; e < 4; ++e) s[n][e] += s2[n][e];
    if (masked) {
#pragma unroll
      for (int n = 0; n < 2; ++n)
#pragma unroll
        for (int e = 0; e < 4; ++e)
          if (!visible(n * 8 + c2 + (e & 1), e >= 2)) s[n][e] = -INFINITY;
    }
    float mx0 = fmaxf(fmaxf(s[0][0], s[0][1]), fmaxf(s[1][0], s[1][1]));
    float mx1 = fmaxf(fmaxf(s[0][2], s[0][3]), fmaxf(s[1][2], s[1][3]));
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
    const float mn0 = fmaxf(m0, mx0 * scale_log2), mn1 = fmaxf(m1, mx1 * scale_log2);
    const float mu0 = (mn0 == -INFINITY) ? 0.f : mn0, mu1 = (mn1 == -INFINITY) ? 0.f : mn1;
    const float al0 = ex2(m0 - mu0), al1 = ex2(m1 - mu1);
    const bool grew = (mn0 != m0) || (mn1 != m1);
    m0 = mn0;
    m1 = mn1;
    uint32_t pf[4];
    {
      float sum0 = 0.f, sum1 = 0.f;
#pragma unroll
      for (int n = 0; n < 2; ++n) {
        const float p0 = ex2(fmaf(s[n][0], scale_log2, -mu0)), p1 = ex2(fmaf(s[n][1], scale_log2, -mu0));
        const float p2 = ex2(fmaf(s[n][2], scale_log2, -mu1)), p3 = ex2(fmaf(s[n][3], scale_log2, -mu1));
        sum0 += p0 + p1;
        sum1 += p2 + p3;
        pf[n * 2] = pack2(p0, p1);
        pf[n * 2 + 1] = pack2(p2, p3);
      }
      l0 = l0 * al0 + sum0;   // per-lane partial sums; reduced over the quad by finish()
      l1 = l1 * al1 + sum1;
    }
    if (__any_sync(0xffffffffu, grew)) {
#pragma unroll
      for (int n = 0; n < NTILES; ++n) { o[n][0] *= al0; o[n][1] *= al0; o[n][2] *= al1; o[n][3] *= al1; }
    }
#pragma unroll
    for (int nn = 0; nn < NTILES / 2; ++nn) {
      uint32_t b0, b1, b2, b3;
      ldsm_x4_t(vs + v_lane + nn * 32, b0, b1, b2, b3);
      mma_bf16(o[2 * nn], pf, b0, b1);
      mma_bf16(o[2 * nn + 1], pf, b2, b3);
    }
  }

  // Two whole tiles (2 * KT positions, every one visible to every row) in one softmax step: four independent chains
  // of MMAs instead of two, one rescale of the accumulator and one round of quad shuffles per 32 positions.
  __device__ __forceinline__ void attend2(uint32_t ksa, uint32_t vsa, uint32_t ksb, uint32_t vsb, float scale_log2, int lane) {
    constexpr int PITCH = Geo<D>::PITCH;
    const int mat = lane >> 3;
    const uint32_t k_lane = (uint32_t)(((mat >> 1) << 3) + (lane & 7)) * PITCH + (uint32_t)(mat & 1) * 16;
    const uint32_t v_lane = (uint32_t)(((mat & 1) << 3) + (lane & 7)) * PITCH + (uint32_t)(mat >> 1) * 16;
    float s[4][4];
#pragma unroll
    for (int n = 0; n < 4; ++n) s[n][0] = s[n][1] = s[n][2] = s[n][3] = 0.f;
#pragma unroll
    for (int kk = 0; kk < KSTEPS; ++kk) {
      uint32_t b0, b1, b2, b3, c0, c1, c2_, c3;
      ldsm_x4(ksa + k_lane + kk * 32, b0, b1, b2, b3);
      ldsm_x4(ksb + k_lane + kk * 32, c0, c1, c2_, c3);
      mma_bf16(s[0], qf[kk], b0, b1);
      mma_bf16(s[1], qf[kk], b2, b3);
      mma_bf16(s[2], qf[kk], c0, c1);
      mma_bf16(s[3], qf[kk], c2_, c3);
    }
    float mx0 = fmaxf(fmaxf(fmaxf(s[0][0], s[0][1]), fmaxf(s[1][0], s[1][1])), fmaxf(fmaxf(s[2][0], s[2][1]), fmaxf(s[3][0], s[3][1])));
    float mx1 = fmaxf(fmaxf(fmaxf(s[0][2], s[0][3]), fmaxf(s[1][2], s[1][3])), fmaxf(fmaxf(s[2][2], s[2][3]), fmaxf(s[3][2], s[3][3])));
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
    const float mn0 = fmaxf(m0, mx0 * scale_log2), mn1 = fmaxf(m1, mx1 * scale_log2);   // finite: every position is visible
    const float al0 = ex2(m0 - mn0), al1 = ex2(m1 - mn1);
    const bool grew = (mn0 != m0) || (mn1 != m1);
    m0 = mn0;
    m1 = mn1;
    uint32_t pf[2][4];
    {
      float sum0 = 0.f, sum1 = 0.f;
#pragma unroll
      for (int n = 0; n < 4; ++n) {
        const float p0 = ex2(fmaf(s[n][0], scale_log2, -mn0)), p1 = ex2(fmaf(s[n][1], scale_log2, -mn0));
        const float p2 = ex2(fmaf(s[n][2], scale_log2, -mn1)), p3 = ex2(fmaf(s[n][3], scale_log2, -mn1));
        sum0 += p0 + p1;
        sum1 += p2 + p3;
        pf[n >> 1][(n & 1) * 2] = pack2(p0, p1);
        pf[n >> 1][(n & 1) * 2 + 1] = pack2(p2, p3);
      }
      l0 = l0 * al0 + sum0;
      l1 = l1 * al1 + sum1;
    }
    if (__any_sync(0xffffffffu, grew)) {
#pragma unroll
      for (int n = 0; n < NTILES; ++n) { o[n][0] *= al0; o[n][1] *= al0; o[n][2] *= al1; o[n][3] *= al1; }
    }
#pragma unroll
    for (int nn = 0; nn < NTILES / 2; ++nn) {
      uint32_t b0, b1, b2, b3, c0, c1, c2_, c3;
      ldsm_x4_t(vsa + v_lane + nn * 32, b0, b1, b2, b3);
      ldsm_x4_t(vsb + v_lane + nn * 32, c0, c1, c2_, c3);
      mma_bf16(o[2 * nn], pf[0], b0, b1);
      mma_bf16(o[2 * nn + 1], pf[0], b2, b3);
      mma_bf16(o[2 * nn], pf[1], c0, c1);
      mma_bf16(o[2 * nn + 1], pf[1], c2_, c3);
    }
  }

  __device__ __forceinline__ void reduce_sums() {
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
    l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
  }

  // The warp saw the whole key list: normalise, stage the 16 x D bf16 tile in `stage` (16 * PITCH bytes of shared
  // memory that only this warp uses), 16-byte stores.  Call after reduce_sums().
  __device__ __forceinline__ void store_rows(uint8_t* stage, bf16* og, const RowMap& rm, int lane) const {
    constexpr int PITCH = Geo<D>::PITCH, CH = Geo<D>::CH, RPI = Geo<D>::RPI;
    const int c2 = (lane & 3) * 2, r0 = lane >> 2, r1 = r0 + 8;
    const float i0 = 1.f / l0, i1 = 1.f / l1;   // rows past W*g hold garbage and are not stored
#pragma unroll
    for (int n = 0; n < NTILES; ++n) {
      *reinterpret_cast<uint32_t*>(stage + r0 * PITCH + (n * 8 + c2) * 2) = pack2(o[n][0] * i0, o[n][1] * i0);
      *reinterpret_cast<uint32_t*>(stage + r1 * PITCH + (n * 8 + c2) * 2) = pack2(o[n][2] * i1, o[n][3] * i1);
    }
    const int64_t my_off = rm.offset(rm.row0 + (lane & 15), D);   // lane r resolves output row r; fetched by shuffle below
    __syncwarp();
#pragma unroll
    for (int it = 0; it < 16 / RPI; ++it) {
      const int r = it * RPI + lane / CH, chunk = lane % CH;
      const int64_t off = __shfl_sync(0xffffffffu, my_off, r);
      if (off >= 0)
        *reinterpret_cast<uint4*>(og + off + chunk * 8) = *reinterpret_cast<const uint4*>(stage + r * PITCH + chunk * 16);
    }
  }
};

// Split-KV finish of one warp: publish this split's normalised partial rows straight from the accumulator
// fragments, take a ticket, and -- if this warp holds the last ticket of its (sequence, kv head, row tile) -- fold
// all partials into the output.  No warp waits for another.  The fold starts when the slowest split ends, so it is
// on the critical path of the launch: it walks the splits once with a running maximum, four splits' loads in
// flight at a time (one thread per row walking the splits in two passes cost 6 to 13 us of L2 round trips at
// 8 to 13 splits on B200).  Call after reduce_sums().
//   part_o [.., n_splits, rows_pad, D] fp32, part_lse [.., n_splits, rows_pad] (log2 domain); unit = b*Hkv + kvh.
template <int D>
__device__ __forceinline__ void publish_and_fold(const RowTile<D>& t, const DecodeArgs& a, const RowMap& rm, int split,
                                                 int live_splits, int row_tile, int lane) {
  constexpr int NTILES = D / 8;
  const int c2 = (lane & 3) * 2, r0 = lane >> 2, r1 = r0 + 8;
  const int64_t unit = (int64_t)rm.b * a.Hkv + rm.kvh;
  const int64_t prow0 = (unit * a.plan.n_splits + split) * a.plan.rows_pad + rm.row0;
  {
    const float i0 = 1.f / t.l0, i1 = 1.f / t.l1;
    float* p0 = a.part_o + (prow0 + r0) * D + c2;
    float* p1 = a.part_o + (prow0 + r1) * D + c2;
    if (rm.row0 + r0 < rm.n_rows) {
#pragma unroll
      for (int n = 0; n < NTILES; ++n) *reinterpret_cast<float2*>(p0 + n * 8) = make_float2(t.o[n][0] * i0, t.o[n][1] * i0);
      if ((lane & 3) == 0) a.part_lse[prow0 + r0] = t.m0 + log2f(t.l0);
    }
    if (rm.row0 + r1 < rm.n_rows) {
#pragma unroll
      for (int n = 0; n < NTILES; ++n) *reinterpret_cast<float2*>(p1 + n * 8) = make_float2(t.o[n][2] * i1, t.o[n][3] * i1);
      if ((lane & 3) == 0) a.part_lse[prow0 + r1] = t.m1 + log2f(t.l1);
    }
  }
  __threadfence();
  __syncwarp();
  int last = 0;
  if (lane == 0) {
    int32_t* ticket = a.tickets + (unit * a.plan.row_tiles + row_tile);
    const int tk = atomicAdd(ticket, 1);
    last = (tk == live_splits - 1);
    if (last) *ticket = 0;   // ready for the next launch on this stream
  }
  if (!__shfl_sync(0xffffffffu, last, 0)) return;
  __threadfence();
  constexpr int V4 = D / 4, RPP = 4 * 32 / V4;   // float4 per row; rows per pass (4 float4 per lane)
  const int live_rows = min(16, rm.n_rows - rm.row0);
  const int64_t fold0 = unit * a.plan.n_splits * a.plan.rows_pad + rm.row0;   // split 0, first row
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
        const float inv = 1.f / den[k];
        uint2 v;
        v.x = pack2(acc[k].x * inv, acc[k].y * inv);
        v.y = pack2(acc[k].z * inv, acc[k].w * inv);
        *reinterpret_cast<uint2*>(og + rm.offset(rm.row0 + rk[k], D) + ck[k] * 4) = v;
      }
    }
  }
}

// Where position pk of a row tile's generated-token list lives: beam w_lo + pk / step, token pk % step; the newest
// token comes straight from k_new / v_new, older ones from the private segment through the lineage table.
// Returns the element offset of the row (for kv head kvh) and sets `which`: 1 private segment, 2 k_new / v_new.
template <int D>
__device__ __forceinline__ int64_t private_row(const DecodeArgs& a, int b, int kvh, int w_lo, int pk, int& which) {
  const int w = w_lo + pk / a.step, t = pk % a.step;
  const int64_t j = (int64_t)b * a.beams + w;
  if (t == a.step - 1) {
    which = 2;
    return (j * a.Hkv + kvh) * D;
  }
  int64_t slab = j;
  if (a.lineage) slab = min(max(a.lineage[j * a.max_new + t], 0), a.batch * a.beams - 1);
  which = 1;
  return (priv_row(a, slab, t) * a.Hkv + kvh) * D;
}

// The three tensors a cache position can live in: 0 shared segment, 1 private segment, 2 this step's k_new / v_new.
struct Sources {
  const bf16* k[3];
  const bf16* v[3];
};

// Copy one tile whose rows were resolved one per lane (lane lane_base + i, i < KT, holds the element offset `off` of
// position i's row, -1 for "no such position", and the tensor `which`): the copying lanes fetch offset and tensor by
// shuffle.  stage = shared-memory address of the K tile; the V tile follows it.  Missing rows are zero-filled.
template <int D>
__device__ __forceinline__ void copy_resolved_tile(uint32_t stage, int64_t off, int which, const Sources& src, int lane,
                                                   int lane_base = 0) {
  using G = Geo<D>;
  const int ch = lane % G::CH, r0 = lane / G::CH;
  const uint32_t kdst = stage + (uint32_t)r0 * G::PITCH + (uint32_t)ch * 16, vdst = kdst + G::TILE_B;
#pragma unroll
  for (int i = 0; i < KT / G::RPI; ++i) {
    const int64_t o_r = __shfl_sync(0xffffffffu, off, lane_base + r0 + i * G::RPI);
    const int w_r = __shfl_sync(0xffffffffu, which, lane_base + r0 + i * G::RPI);
    const bf16* ks = (w_r == 0 ? src.k[0] : w_r == 1 ? src.k[1] : src.k[2]) + (o_r < 0 ? 0 : o_r) + ch * 8;
    const bf16* vs = (w_r == 0 ? src.v[0] : w_r == 1 ? src.v[1] : src.v[2]) + (o_r < 0 ? 0 : o_r) + ch * 8;
    const int bytes = o_r < 0 ? 0 : 16;   // 0: nothing is read, the 16 destination bytes become zero
    cp_async16(kdst + i * G::RPI * G::PITCH, ks, bytes);
    cp_async16(vdst + i * G::RPI * G::PITCH, vs, bytes);
  }
}

// Eq. 4, append, for the common case of at most one 16-byte piece per thread (one beam per row tile): fetch() early,
// store() after the key loop, so that the round trip of the fetch hides under the loop.  When the row tile holds more
// pieces than threads, active() is false and the caller falls back on append_new_rows().
template <int D>
struct AppendOne {
  uint4 piece;
  int64_t dst;      // element offset in the private segment, -1: nothing to store
  bool is_v, single;
  __device__ __forceinline__ void fetch(const DecodeArgs& a, const RowMap& rm, int tid, int n_threads, bool enabled) {
    constexpr int CH = Geo<D>::CH;
    const int w_first = (rm.row0 + rm.g - 1) / rm.g, w_last = min((rm.row0 + 15) / rm.g, rm.W - 1);
    const int n_items = max(w_last - w_first + 1, 0) * 2 * CH;
    single = n_items <= n_threads;
    dst = -1;
    if (enabled && single && tid < n_items) {
      const int64_t j = (int64_t)rm.b * rm.W + w_first + tid / (2 * CH);
      const int c = tid % (2 * CH);
      is_v = c >= CH;
      piece = *reinterpret_cast<const uint4*>(reinterpret_cast<const bf16*>(is_v ? a.v_new : a.k_new) + (j * a.Hkv + rm.kvh) * D + (c % CH) * 8);
      dst = (priv_row(a, j, a.step - 1) * a.Hkv + rm.kvh) * D + (c % CH) * 8;
    }
  }
  __device__ __forceinline__ void store(const DecodeArgs& a) const {
    if (dst >= 0) *reinterpret_cast<uint4*>(reinterpret_cast<bf16*>(is_v ? a.v_priv : a.k_priv) + dst) = piece;
  }
};

// Eq. 4, append: store the new K/V row of every beam whose first query row lies in rows row0 .. row0+15
// (`n_threads` threads with index `tid` share the copy).  The 16-byte pieces are fetched eight at a time before any
// of them is stored: one round trip to memory per eight pieces instead of one per piece.
template <int D>
__device__ __forceinline__ void append_new_rows(const DecodeArgs& a, const RowMap& rm, int tid, int n_threads) {
  constexpr int CH = Geo<D>::CH, BATCH = 8;
  const bf16* kn = reinterpret_cast<const bf16*>(a.k_new);
  const bf16* vn = reinterpret_cast<const bf16*>(a.v_new);
  bf16* kp = reinterpret_cast<bf16*>(a.k_priv);
  bf16* vp = reinterpret_cast<bf16*>(a.v_priv);
  const int w_first = (rm.row0 + rm.g - 1) / rm.g;   // a beam whose first row belongs to the previous tile is appended there
  const int w_last = min((rm.row0 + 15) / rm.g, rm.W - 1);
  const int n_items = max(w_last - w_first + 1, 0) * 2 * CH;   // item = (beam, K or V, 16-byte piece)
  if (n_items <= n_threads) {   // one beam per tile and the like: a single piece per thread
    if (tid < n_items) {
      const int64_t j = (int64_t)rm.b * rm.W + w_first + tid / (2 * CH);
      const int c = tid % (2 * CH);
      *reinterpret_cast<uint4*>((c < CH ? kp : vp) + (priv_row(a, j, a.step - 1) * a.Hkv + rm.kvh) * D + (c % CH) * 8) =
          *reinterpret_cast<const uint4*>((c < CH ? kn : vn) + (j * a.Hkv + rm.kvh) * D + (c % CH) * 8);
    }
    return;
  }
  for (int i0 = tid; i0 < n_items; i0 += BATCH * n_threads) {
    uint4 r[BATCH];
#pragma unroll
    for (int u = 0; u < BATCH; ++u) {
      const int i = i0 + u * n_threads;
      if (i < n_items) {
        const int64_t j = (int64_t)rm.b * rm.W + w_first + i / (2 * CH);
        const int c = i % (2 * CH);
        r[u] = __ldg(reinterpret_cast<const uint4*>((c < CH ? kn : vn) + (j * a.Hkv + rm.kvh) * D + (c % CH) * 8));
      }
    }
#pragma unroll
    for (int u = 0; u < BATCH; ++u) {
      const int i = i0 + u * n_threads;
      if (i < n_items) {
        const int64_t j = (int64_t)rm.b * rm.W + w_first + i / (2 * CH);
        const int c = i % (2 * CH);
        *reinterpret_cast<uint4*>((c < CH ? kp : vp) + (priv_row(a, j, a.step - 1) * a.Hkv + rm.kvh) * D + (c % CH) * 8) = r[u];
      }
    }
  }
}

}  // namespace dec
}  // namespace earn
