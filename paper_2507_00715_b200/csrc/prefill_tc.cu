// Full causal prefill attention (Eq. 3 + causal mask, layers l < k) on the Blackwell tensor cores.
// bf16 Q/K/V, head_dim 128, fp32 logits / softmax / accumulation, bf16 output.
//
// Work item = two "M-tiles" of 128 query rows that share every K/V tile: two query heads of one kv group on the
// same rows (even GQA group size), or two consecutive query tiles of one head (odd group size, multi-head
// attention; the first tile sits out the last key tile, which lies wholly past its diagonal).
// A small planning kernel lists the (sequence, query tile) pairs of the batch, longest key range first;
// the main kernel is persistent (one CTA per SM) and CTA c takes items c, c + gridDim, ... of that list,
// so every SM gets the same mix of long and short items and the pipeline below never drains between items.
//
//   warp 0     TMA: K and V tiles -> shared memory (128-byte swizzle), a ring of 32 KB entries K0 V0 K1 V1 ..
//              that runs on across item boundaries
//   warp 2     TMA: the Q tiles of the next item, as soon as the last S of the current item has read them
//   warp 1     one thread issues tcgen05.mma: S_x = Q_x K^T into tensor memory, O_x += P_x V with P_x read
//              from tensor memory; after the last P V of an item it goes straight on to the first S of the next
//   warps 4..  one softmax warpgroup per M-tile, one query row per thread: S_x from TMEM in 32-column chunks,
//              online softmax in the log2 domain in ONE pass per tile (the reference maximum of the row is the one
//              the earlier tiles left; the first tile of an item takes the maximum of its first 32 columns), packed
//              fp32x2 arithmetic, P_x kept in registers until the reference is known to hold and then written as
//              bf16 over the first 64 columns of S_x; the same warps normalise O_x when the item ends, stage their
//              32 rows each in shared memory and hand them to the copy engine (TMA store), while the tensor core
//              already works on the next item
// With two M-tiles the tensor core works on one while the other is in its softmax (S_A, S_B, O_A, O_B fill
// the 512 TMEM columns).  The running output stays in TMEM.  The softmax reference maximum is only raised
// when a tile's sum of exponentials exceeds 2^8 (no term can exceed that bound otherwise); then the owning warp
// rescales its 32 rows of O in TMEM and redoes the tile (S_x is still intact).  Exact after the final division
// by the row sum.
//
// Every mbarrier wait is bounded; when one runs out the CTA raises its abort flag, writes
// EARN_ERR_TIMEOUT to the status word, drains what it has in flight, frees its TMEM and returns.
#include <algorithm>
#include <type_traits>

#include "earn_common.cuh"
#include "sm100_ptx.cuh"
#include "tc_maps.cuh"

namespace earn {
namespace {
using namespace ptx;

constexpr int BM = 128, BN = 128, HD = 128;
constexpr int TILE = BM * HD * 2;   // bytes of one 128 x 128 bf16 tile
constexpr int HALF = TILE / 2;      // one 64-column block of it (128 rows x 128 B)
constexpr long long WAIT_LIMIT = 2000000000LL;     // about one second of SM clocks

constexpr int NT = 2;   // M-tiles per work item

struct Cfg {
  static constexpr int NSTAGE = 3;                          // ring entries (K and V tiles alternate); four and five measured the same
  static constexpr int OFF_Q = 0;
  static constexpr int OFF_RING = OFF_Q + NT * TILE;
  static constexpr int OFF_OUT = OFF_RING + NSTAGE * TILE;  // per M-tile: the 128 x 128 bf16 tile of O on its way out
  static constexpr int OFF_BAR = OFF_OUT + NT * TILE;
  static constexpr int SMEM_BYTES = OFF_BAR + 512 + 1024;   // + alignment slack
  static constexpr int TMEM_COLS = NT * 256;                // S_x (and P_x over it) at x*128, O_x at (NT + x)*128
  static constexpr int THREADS = 32 * (4 + 4 * NT);
  // barriers
  static constexpr int BAR_FULL = 0, BAR_EMPTY = BAR_FULL + NSTAGE, BAR_QFULL = BAR_EMPTY + NSTAGE,
                       BAR_QFREE = BAR_QFULL + NT, BAR_S = BAR_QFREE + NT, BAR_P = BAR_S + NT, BAR_O = BAR_P + NT,
                       BAR_DRAIN = BAR_O + NT, N_BARS = BAR_DRAIN + 1;
  static_assert(8 * N_BARS + 16 <= 512, "barrier block");
};

struct TcParams {
  void* o;
  float* lse;
  const int4* plan;        // one entry per (sequence, query tile): {first global row, rows of the sequence from there, tile index, sequence}
  int32_t* status;
  int Hq, g, total, n_items, n_hp;   // n_hp work items per plan entry
  float scale_log2;
};

struct Item {
  int key0;      // global row of the sequence's first key
  int n_tiles;   // key tiles both M-tiles are run over: 0 .. the later diagonal
  int kvh;       // kv head
  int row0[NT];  // global row of the first query of M-tile x
  int rows[NT];  // rows of the sequence from there on; the tile holds min(rows, 128) valid rows (none if <= 0)
  int head[NT];  // query head of M-tile x
  int diag[NT];  // key tile that holds M-tile x's diagonal; later tiles are invisible to it
};

// Plan entry {first global row, rows of the sequence from there, level, sequence} -> work item i.
//   two heads of a group (even group size): level = query tile; both M-tiles have the same rows and the same diagonal;
//   two query tiles of one head (odd group size, multi-head attention): level = pair of query tiles; the first
//   M-tile's diagonal is one key tile earlier, and it sits out the last key tile (all of it is masked for it).
template <bool PAIR_TILES>   // false: the two M-tiles are two heads of a kv group; true: two consecutive query tiles of one head
__device__ __forceinline__ Item load_item(const TcParams& p, int i) {
  const int e = i / p.n_hp, hp = i - e * p.n_hp;
  const int4 t = __ldg(p.plan + e);
  Item it;
  if (!PAIR_TILES) {
    it.key0 = t.x - t.z * BM;
    it.n_tiles = t.z + 1;
#pragma unroll
    for (int x = 0; x < NT; ++x) { it.row0[x] = t.x; it.rows[x] = t.y; it.head[x] = hp * NT + x; it.diag[x] = t.z; }
  } else {
    it.key0 = t.x - t.z * (NT * BM);
    it.n_tiles = NT * t.z + NT;
#pragma unroll
    for (int x = 0; x < NT; ++x) { it.row0[x] = t.x + x * BM; it.rows[x] = t.y - x * BM; it.head[x] = hp; it.diag[x] = NT * t.z + x; }
  }
  it.kvh = it.head[0] / p.g;
  return it;
}

// ---- packed fp32 pairs (one instruction for two lanes of the row) and three-input max
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
__device__ __forceinline__ void fma2(float& d0, float& d1, float a0, float a1, float b, float c) {   // d = a * b + c
  asm("{\n\t.reg .b64 ra, rb, rc, rd;\n\tmov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %4};\n\tmov.b64 rc, {%5, %5};\n\t"
      "fma.rn.ftz.f32x2 rd, ra, rb, rc;\n\tmov.b64 {%0, %1}, rd;\n\t}"
      : "=f"(d0), "=f"(d1) : "f"(a0), "f"(a1), "f"(b), "f"(c));
}
__device__ __forceinline__ void add2(float& d0, float& d1, float a0, float a1) {   // d += a
  asm("{\n\t.reg .b64 ra, rd;\n\tmov.b64 ra, {%2, %3};\n\tmov.b64 rd, {%0, %1};\n\tadd.rn.ftz.f32x2 rd, rd, ra;\n\t"
      "mov.b64 {%0, %1}, rd;\n\t}"
      : "+f"(d0), "+f"(d1) : "f"(a0), "f"(a1));
}
template <bool PAIR_TILES>
__global__ void __launch_bounds__(Cfg::THREADS, 1)
prefill_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                  const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_o, TcParams p) {
  using C = Cfg;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;    // swizzled tiles need 1024-byte alignment
  uint8_t* gen = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t sQ = base + C::OFF_Q, sRing = base + C::OFF_RING;
  const uint32_t bars = base + C::OFF_BAR;
  auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gen + C::OFF_BAR + 8 * C::N_BARS);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gen + C::OFF_BAR + 8 * C::N_BARS + 8);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < C::NSTAGE; ++s) {
      mbar_init(bar(C::BAR_FULL + s), 1);
      mbar_init(bar(C::BAR_EMPTY + s), 1);
    }
    for (int x = 0; x < NT; ++x) {
      mbar_init(bar(C::BAR_QFULL + x), 1);
      mbar_init(bar(C::BAR_QFREE + x), 1);
      mbar_init(bar(C::BAR_S + x), 1);
      mbar_init(bar(C::BAR_P + x), 128);
      mbar_init(bar(C::BAR_O + x), 1);
    }
    mbar_init(bar(C::BAR_DRAIN), 1);
    *abort_flag = 0;
    fence_barrier_init();
    tma_prefetch_desc(&map_q);
    tma_prefetch_desc(&map_k);
    tma_prefetch_desc(&map_v);
    tma_prefetch_desc(&map_o);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), C::TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  // This CTA's items: the plan is dealt to the CTAs in passes of gridDim.x items, forwards and backwards in turn (the
  // plan is sorted longest first, so dealing every pass in the same direction gives the low-numbered CTAs the longer
  // item of every pass: 3 % more work than the mean on the long-history shapes, 15 % on the 1.5B ones).
  const int n_cta = gridDim.x;
  auto item_at = [&](int k) { return k * n_cta + ((k & 1) ? n_cta - 1 - (int)blockIdx.x : (int)blockIdx.x); };
  pdl_launch_dependents();
  pdl_wait();   // the plan (written by the kernel launched just before this one) and every tensor are read below

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer: K/V ring
    if (lane == 0) {
      int e = 0;   // ring entries issued so far, over all items
      bool ok = true;
      for (int k = 0, i = item_at(0); i < p.n_items && ok; i = item_at(++k)) {
        const Item it = load_item<PAIR_TILES>(p, i);
        const int kvh = it.kvh;
        for (int t = 0; t < 2 * it.n_tiles; ++t, ++e) {
          const int st = e % C::NSTAGE;
          if (e >= C::NSTAGE &&
              !mbar_wait_bounded(bar(C::BAR_EMPTY + st), ((e / C::NSTAGE) - 1) & 1, abort_flag, WAIT_LIMIT)) {
            ok = false;
            break;
          }
          const CUtensorMap* map = (t & 1) ? &map_v : &map_k;
          mbar_expect_tx(bar(C::BAR_FULL + st), TILE);
          tma_load_3d(sRing + st * TILE, map, bar(C::BAR_FULL + st), 0, kvh, it.key0 + (t >> 1) * BN);
          tma_load_3d(sRing + st * TILE + HALF, map, bar(C::BAR_FULL + st), 64, kvh, it.key0 + (t >> 1) * BN);
        }
      }
      if (*abort_flag) {
        // let the copies already in flight land before the CTA gives its shared memory back
        int none = 0;
        for (int f = max(e - C::NSTAGE, 0); f < e; ++f)
          mbar_wait_bounded(bar(C::BAR_FULL + f % C::NSTAGE), (f / C::NSTAGE) & 1, &none, WAIT_LIMIT);
      }
    }
  } else if (warp == 2) {
    // ------------------------------------------------------------------ TMA producer: Q tiles
    if (lane == 0) {
      int n = 0;   // items loaded so far
      bool ok = true;
      for (int i = item_at(0); i < p.n_items && ok; i = item_at(++n)) {
        const Item it = load_item<PAIR_TILES>(p, i);
        for (int x = 0; x < NT; ++x) {
          if (n > 0 && !mbar_wait_bounded(bar(C::BAR_QFREE + x), (n - 1) & 1, abort_flag, WAIT_LIMIT)) {
            ok = false;
            break;
          }
          mbar_expect_tx(bar(C::BAR_QFULL + x), TILE);
          tma_load_3d(sQ + x * TILE, &map_q, bar(C::BAR_QFULL + x), 0, it.head[x], it.row0[x]);
          tma_load_3d(sQ + x * TILE + HALF, &map_q, bar(C::BAR_QFULL + x), 64, it.head[x], it.row0[x]);
        }
      }
      if (*abort_flag && n > 0) {
        int none = 0;
        for (int x = 0; x < NT; ++x) mbar_wait_bounded(bar(C::BAR_QFULL + x), (n - 1) & 1, &none, WAIT_LIMIT);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    // The whole warp runs the loop (so that every descriptor is warp-uniform arithmetic and nothing but the
    // tcgen05.mma instructions themselves sits between two of them); lane 0 issues.
    {
      const bool leader = lane == 0;
      constexpr uint32_t idesc_s = idesc_bf16_f32(BM, BN, 0, 0);   // Q (K-major) x K^T (K-major)
      constexpr uint32_t idesc_o = idesc_bf16_f32(BM, HD, 0, 1);   // P (TMEM) x V (MN-major)
      constexpr uint32_t desc_hi = smem_desc_hi_sw128(1024);
      const uint32_t q_lo = smem_desc_lo(sQ, 16), k_lo = smem_desc_lo(sRing, 16), v_lo = smem_desc_lo(sRing, HALF);
      auto wait = [&](int b, int parity) {   // warp-uniform result
        return __all_sync(0xffffffffu, mbar_wait_bounded(bar(b), (uint32_t)parity & 1u, abort_flag, WAIT_LIMIT));
      };
      auto wait_full = [&](int e) { return wait(C::BAR_FULL + e % C::NSTAGE, e / C::NSTAGE); };
      // S_x = Q_x K^T with the K tile of ring entry e; `last` = no later S of this item reads Q_x
      auto issue_s = [&](int x, int e, bool last) {
        const uint32_t a0 = q_lo + x * (TILE >> 4), b0 = k_lo + (e % C::NSTAGE) * (TILE >> 4);
        if (leader) {
#pragma unroll
          for (int kk = 0; kk < HD / 16; ++kk) {
            const uint32_t off = ((kk >> 2) * HALF + (kk & 3) * 32) >> 4;
            umma_ss_lohi(tmem + x * 128, a0 + off, desc_hi, b0 + off, desc_hi, idesc_s, kk > 0);
          }
          umma_commit(bar(C::BAR_S + x));
          if (last) umma_commit(bar(C::BAR_QFREE + x));
          if (x == NT - 1) umma_commit(bar(C::BAR_EMPTY + e % C::NSTAGE));   // K tile free once the last S has read it
        }
      };
      // O_x (+)= P_x V with P_x in tensor memory (bf16 pairs over the first 64 columns of S_x) and the V tile of entry e
      auto issue_pv = [&](int x, int e, bool first_tile) {
        const uint32_t b0 = v_lo + (e % C::NSTAGE) * (TILE >> 4);
        if (leader) {
#pragma unroll
          for (int kk = 0; kk < BN / 16; ++kk)
            umma_ts_lohi(tmem + (NT + x) * 128, tmem + x * 128 + kk * 8, b0 + kk * (2048 >> 4), desc_hi, idesc_o,
                         (!first_tile || kk > 0) ? 1u : 0u);
          if (x == NT - 1) umma_commit(bar(C::BAR_EMPTY + e % C::NSTAGE));   // V tile free once the last P V has read it
        }
      };
      int eb = 0;       // ring entry of the current item's K_0
      int n_item = 0;   // items started so far
      int n_p[NT];      // P_x phases consumed so far
      for (int x = 0; x < NT; ++x) n_p[x] = 0;
      bool ok = item_at(0) < p.n_items;
      Item cur{};
      if (ok) {
        cur = load_item<PAIR_TILES>(p, item_at(0));
        for (int x = 0; x < NT && ok; ++x) {
          ok = wait(C::BAR_QFULL + x, 0) && (x > 0 || wait_full(0));
          if (!ok) break;
          tc_fence_after();
          issue_s(x, 0, cur.n_tiles == 1);
        }
      }
      for (int i = item_at(0); i < p.n_items && ok; i = item_at(++n_item)) {
        const bool has_next = item_at(n_item + 1) < p.n_items;
        Item nxt{};
        if (has_next) nxt = load_item<PAIR_TILES>(p, item_at(n_item + 1));
        const int n = cur.n_tiles;
        for (int j = 0; j < n && ok; ++j) {
          for (int x = 0; x < NT && ok; ++x) {
            ok = wait(C::BAR_P + x, n_p[x]);   // P_x(j) written, S_x consumed
            ++n_p[x];
            if (ok && x == 0) ok = wait_full(eb + 2 * j + 1);
            if (!ok) break;
            tc_fence_after();
            issue_pv(x, eb + 2 * j + 1, j == 0);
            if (j < n - 1) {
              if (x == 0) ok = wait_full(eb + 2 * j + 2);
              if (!ok) break;
              tc_fence_after();
              issue_s(x, eb + 2 * j + 2, j + 1 == n - 1);
            } else {
              if (leader) umma_commit(bar(C::BAR_O + x));
              if (has_next) {   // straight on to the next item: its Q_x and first K tile are on their way already
                ok = wait(C::BAR_QFULL + x, n_item + 1);
                if (ok && x == 0) ok = wait_full(eb + 2 * n);
                if (!ok) break;
                tc_fence_after();
                issue_s(x, eb + 2 * n, nxt.n_tiles == 1);
              }
            }
          }
        }
        eb += 2 * n;
        cur = nxt;
      }
      if (leader && *abort_flag) {
        int none = 0;
        umma_commit(bar(C::BAR_DRAIN));   // everything this thread issued has retired once this fires
        mbar_wait_bounded(bar(C::BAR_DRAIN), 0, &none, WAIT_LIMIT);
      }
      __syncwarp();
    }
  } else if (warp >= 4) {
    // ------------------------------------------------------------------ softmax warpgroup x, one row per thread
    const int x = (warp - 4) >> 2;
    const int wq = warp & 3;            // a warp may only touch TMEM lanes 32*(warp % 4) ..
    const int row = wq * 32 + lane;
    const uint32_t t_s = tmem + ((uint32_t)(wq * 32) << 16) + x * 128;   // S_x; P_x goes over its first 64 columns
    const uint32_t t_o = tmem + ((uint32_t)(wq * 32) << 16) + (NT + x) * 128;
    const float sl2 = p.scale_log2;
    int n_s = 0, n_item = 0;
    bool ok = true;
    for (int i = item_at(0); i < p.n_items && ok; i = item_at(++n_item)) {
      const Item it = load_item<PAIR_TILES>(p, i);
      // this M-tile's share of the item, in registers (x is not a compile-time index)
      const int h = x ? it.head[1] : it.head[0], my_diag = x ? it.diag[1] : it.diag[0];
      const int my_row0 = x ? it.row0[1] : it.row0[0], my_rows = x ? it.rows[1] : it.rows[0];
      float m_ref = 0.f, l0 = 0.f, l1 = 0.f;
      for (int j = 0; j < it.n_tiles; ++j, ++n_s) {
        ok = __all_sync(0xffffffffu, mbar_wait_bounded(bar(C::BAR_S + x), n_s & 1, abort_flag, WAIT_LIMIT));   // warp-uniform
        if (!ok) break;
        tc_fence_after();
        const bool diag = j == my_diag;               // key column c of this tile is visible to row r iff c <= r
        // 32-column chunks with a visible key for this warp's rows (none in a tile past the diagonal)
        const int n_chunks = diag ? wq + 1 : (!PAIR_TILES || j < my_diag) ? 4 : 0;
        uint32_t a[32], b[32], pk[4][16];
        // row maximum of the visible part of S_x(j), scaled into the log2 domain (a pass of its own over TMEM)
        auto row_max_all = [&]() {
          float mx = -INFINITY;
          tmem_ld_32x32(t_s, a);
          if (n_chunks > 1) tmem_ld_32x32(t_s + 32, b);
          tmem_wait_ld(a);
          tmem_wait_ld(b);
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            if (q < n_chunks) {
              uint32_t(&cur)[32] = (q & 1) ? b : a;
              if (diag && q == wq) {
#pragma unroll
                for (int c = 0; c < 32; ++c)
                  if (c > lane) cur[c] = 0xff800000u;   // -inf
              }
              float m1 = -INFINITY;
#pragma unroll
              for (int c = 0; c < 32; c += 4) {
                mx = max3(mx, __uint_as_float(cur[c]), __uint_as_float(cur[c + 1]));
                m1 = max3(m1, __uint_as_float(cur[c + 2]), __uint_as_float(cur[c + 3]));
              }
              mx = fmaxf(mx, m1);
            }
            if (q == 1 && n_chunks > 2) {
              tmem_ld_32x32(t_s + 64, a);
              if (n_chunks > 3) tmem_ld_32x32(t_s + 96, b);
              tmem_wait_ld(a);
              tmem_wait_ld(b);
            }
          }
          return mx * sl2;
        };
        // ---- P = 2^(S * scale - m_ref) as bf16 pairs (kept in registers until the reference is known to hold) and
        //      their row sum, in one pass.  The reference is the one earlier tiles left.  If this tile's sum of
        //      exponentials exceeds 2^8 some logit may have outgrown the reference by more than the threshold
        //      (rare: with the reference at the running maximum every term is <= 1 and the sum <= 128): then find
        //      the tile's own maximum, raise the reference, rescale what has been accumulated, and redo the pass.
        //      S_x is still intact because nothing has been written over it.  No term ever exceeds 2^8.
        float ls0, ls1;
#pragma unroll 1
        for (int attempt = 0;; ++attempt) {
          ls0 = ls1 = 0.f;
          tmem_ld_32x32(t_s, a);
          tmem_wait_ld(a);
          if (j == 0 && attempt == 0) {
            // First tile of an item: the reference is the largest visible logit among the row's first 32 keys (the
            // start of the sequence; column 0 is visible to every row).  A later column that outgrows it by more
            // than the threshold shows in the sum below and sends the tile through the redo path like any other.
            // (A pass of its own over all 128 columns for the exact row maximum cost 26 us per 7B-class layer.)
            float mx = -INFINITY, m1 = -INFINITY;
#pragma unroll
            for (int c = 0; c < 32; c += 4) {
              const bool d0 = diag && wq == 0;   // on the diagonal chunk column c counts for row `lane` iff c <= lane
              mx = max3(mx, (d0 && c > lane) ? -INFINITY : __uint_as_float(a[c]), (d0 && c + 1 > lane) ? -INFINITY : __uint_as_float(a[c + 1]));
              m1 = max3(m1, (d0 && c + 2 > lane) ? -INFINITY : __uint_as_float(a[c + 2]), (d0 && c + 3 > lane) ? -INFINITY : __uint_as_float(a[c + 3]));
            }
            m_ref = fmaxf(mx, m1) * sl2;
          }
          const float neg_m = -m_ref;
          // Two copies of the loop over the four chunks: an interior tile (all 128 columns visible, the usual case) takes
          // the one without a test per chunk, which the compiler schedules as one block of straight-line code -- the end
          // of one chunk's arithmetic overlaps the start of the next -- where the tests cut it into four.
          auto chunks = [&](auto interior_tag) {
            constexpr bool INTERIOR = decltype(interior_tag)::value;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              if (INTERIOR || q < n_chunks) {
                uint32_t(&cur)[32] = (q & 1) ? b : a;
                uint32_t(&nxt)[32] = (q & 1) ? a : b;
                if (q + 1 < 4 && (INTERIOR || q + 1 < n_chunks)) tmem_ld_32x32(t_s + (q + 1) * 32, nxt);
                if (!INTERIOR && diag && q == wq) {
#pragma unroll
                  for (int c = 0; c < 32; ++c)
                    if (c > lane) cur[c] = 0xff800000u;
                }
#pragma unroll
                for (int c = 0; c < 32; c += 2) {
                  float e0, e1;
                  fma2(e0, e1, __uint_as_float(cur[c]), __uint_as_float(cur[c + 1]), sl2, neg_m);
                  e0 = ex2(e0);   // all on the special-function unit: a cubic on the FMA pipe for a share of them costs
                  e1 = ex2(e1);   // more issue slots than it frees on the unit
                  add2(ls0, ls1, e0, e1);
                  pk[q][c >> 1] = pack_bf16(e0, e1);
                }
                if (q + 1 < 4 && (INTERIOR || q + 1 < n_chunks)) tmem_wait_ld(nxt);
              } else {
#pragma unroll
                for (int c = 0; c < 16; ++c) pk[q][c] = 0u;
              }
            }
          };
          if (n_chunks == 4 && !diag) chunks(std::true_type{});
          else chunks(std::false_type{});
          const bool grow = !(ls0 + ls1 <= 256.f);   // also catches a sum that overflowed
          if (attempt > 0 || !__any_sync(0xffffffffu, grow)) break;
          // S_x(j) was issued after P_x V of tile j-1, so the commit that signalled it covers that too: O_x is quiescent
          // the whole warp repeats the pass (the TMEM accesses are warp-wide), but only the rows that grew take a new
          // reference: a row's result depends on its own logits alone, whatever its neighbours in the tile do
          const float mx_all = row_max_all();   // every lane takes part in the loads
          const float mxs = grow ? mx_all : m_ref;
          const float alpha = mxs > m_ref ? ex2(m_ref - mxs) : 1.f;
          m_ref = fmaxf(m_ref, mxs);
          l0 *= alpha;
          l1 *= alpha;
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            tmem_ld_32x32(t_o + q * 32, a);
            tmem_wait_ld(a);
#pragma unroll
            for (int c = 0; c < 32; ++c) a[c] = __float_as_uint(__uint_as_float(a[c]) * alpha);
            tmem_st_32x32(t_o + q * 32, a);
          }
        }
        l0 += ls0;
        l1 += ls1;
#pragma unroll
        for (int q = 0; q < 4; ++q) tmem_st_32x16(t_s + q * 16, pk[q]);
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(bar(C::BAR_P + x));
      }
      if (!ok) break;
      // ---- end of the item: O_x / l -> global memory (the tensor core is already on the next item's S)
      ok = __all_sync(0xffffffffu, mbar_wait_bounded(bar(C::BAR_O + x), n_item & 1, abort_flag, WAIT_LIMIT));
      if (!ok) break;
      tc_fence_after();
      const float l = l0 + l1;
      const float inv = 1.f / l;
      const bool valid = row < my_rows;
      __nv_bfloat16* orow = reinterpret_cast<__nv_bfloat16*>(p.o) + ((int64_t)(my_row0 + row) * p.Hq + h) * HD;
      uint32_t a[32], b[32];
      if (my_rows >= BM) {
        // A whole tile of this sequence goes out through shared memory and the copy engine (each thread writing its
        // own 256-byte row with 16-byte stores took 3600 clocks per item: 4096 half-sector writes through one
        // load/store unit).  Lane r of a warp writes 16-byte chunk c of its row at chunk c ^ (r % 8) of the row's
        // 128-byte line, the 128-byte swizzle the tensor map expects.
        // Each warp stages and sends its own 32 rows (two blocks of 32 x 64), so no warp waits for another.
        const uint32_t out = base + C::OFF_OUT + x * TILE + (uint32_t)wq * (32 * 128);
        // 32-column chunks, the next one in flight while this one is scaled, packed and staged
        if (lane == 0) bulk_wait_read0();   // this warp's previous copies have left its staging rows (long ago)
        tmem_ld_32x32(t_o, a);
        tmem_wait_ld(a);
        __syncwarp();
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          uint32_t(&cur)[32] = (q & 1) ? b : a;
          uint32_t(&nxt)[32] = (q & 1) ? a : b;
          if (q + 1 < 4) tmem_ld_32x32(t_o + (q + 1) * 32, nxt);
#pragma unroll
          for (int c = 0; c < 4; ++c) {   // chunk c of this quarter = 16-byte chunk (q % 2) * 4 + c of block q / 2
            const uint32_t w0 = pack_bf16(__uint_as_float(cur[c * 8 + 0]) * inv, __uint_as_float(cur[c * 8 + 1]) * inv);
            const uint32_t w1 = pack_bf16(__uint_as_float(cur[c * 8 + 2]) * inv, __uint_as_float(cur[c * 8 + 3]) * inv);
            const uint32_t w2 = pack_bf16(__uint_as_float(cur[c * 8 + 4]) * inv, __uint_as_float(cur[c * 8 + 5]) * inv);
            const uint32_t w3 = pack_bf16(__uint_as_float(cur[c * 8 + 6]) * inv, __uint_as_float(cur[c * 8 + 7]) * inv);
            const int ch = (q & 1) * 4 + c;
            st_shared_v4(out + (q >> 1) * HALF + (uint32_t)lane * 128 + (uint32_t)((ch ^ (lane & 7)) << 4), w0, w1, w2, w3);
          }
          if (q + 1 < 4) tmem_wait_ld(nxt);
        }
        fence_async_smem();
        __syncwarp();
        if (lane == 0) {
          tma_store_3d(&map_o, out, 0, h, my_row0 + wq * 32);
          tma_store_3d(&map_o, out + HALF, 64, h, my_row0 + wq * 32);
          bulk_commit();
        }
      } else {
      tmem_ld_32x32(t_o, a);
      tmem_wait_ld(a);
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        uint32_t(&cur)[32] = (q & 1) ? b : a;
        uint32_t(&nxt)[32] = (q & 1) ? a : b;
        if (q + 1 < 4) tmem_ld_32x32(t_o + (q + 1) * 32, nxt);
        if (valid) {
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            uint4 w;
            w.x = pack_bf16(__uint_as_float(cur[c * 8 + 0]) * inv, __uint_as_float(cur[c * 8 + 1]) * inv);
            w.y = pack_bf16(__uint_as_float(cur[c * 8 + 2]) * inv, __uint_as_float(cur[c * 8 + 3]) * inv);
            w.z = pack_bf16(__uint_as_float(cur[c * 8 + 4]) * inv, __uint_as_float(cur[c * 8 + 5]) * inv);
            w.w = pack_bf16(__uint_as_float(cur[c * 8 + 6]) * inv, __uint_as_float(cur[c * 8 + 7]) * inv);
            *reinterpret_cast<uint4*>(orow + q * 32 + c * 8) = w;
          }
        }
        if (q + 1 < 4) tmem_wait_ld(nxt);
      }
      }
      if (valid && p.lse != nullptr) p.lse[(int64_t)h * p.total + my_row0 + row] = (m_ref + log2f(l)) * kLn2;
      tc_fence_before();   // the next item's first P V overwrites O_x; it is issued after this warp's next arrive on P_x
    }
  }

  if (warp >= 4 && lane == 0) bulk_wait_all0();   // this thread's output copies have completed
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) atomicExch(p.status, (int32_t)EARN_ERR_TIMEOUT);
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, C::TMEM_COLS);
  }
}

// ------------------------------------------------------------------------------------------------
// planning kernel: one entry per (sequence, block of `rows` query rows), blocks with the longest key range first
// (rows = 128: one query tile; rows = 256: a pair of query tiles)
// ------------------------------------------------------------------------------------------------
constexpr int PLAN_THREADS = 1024;
constexpr int PLAN_MAX_LEVELS = 2048;   // query tiles per sequence the planner can order (256 K tokens)

__global__ void __launch_bounds__(PLAN_THREADS) prefill_plan_kernel(const int32_t* cu_seqlens, int batch, int max_tiles,
                                                                    int rows, int group_seqs, int4* plan) {
  // The sequences are taken in groups of `group_seqs` (the K/V rows of one group fit the L2 cache with room to spare:
  // the items of a group re-read them once per tile level) and the groups' entries follow one another.  Within a
  // group, level t holds every sequence with more than t blocks; levels are laid out from the highest down.
  __shared__ int cnt[PLAN_MAX_LEVELS];      // sequences per level, then the level's cursor
  __shared__ int off[PLAN_MAX_LEVELS];      // first entry of the level
  __shared__ int base;                      // entries of the groups before this one
  pdl_launch_dependents();
  pdl_wait();   // the plan area may still be read by the kernel before this one
  if (threadIdx.x == 0) base = 0;
  const int gs = group_seqs > 0 ? group_seqs : batch;
  for (int g0 = 0; g0 < batch; g0 += gs) {
    const int g1 = min(g0 + gs, batch);
    __syncthreads();   // (the last group's cursors are done with)
    for (int t = threadIdx.x; t < max_tiles; t += PLAN_THREADS) cnt[t] = 0;
    __syncthreads();
    for (int b = g0 + threadIdx.x; b < g1; b += PLAN_THREADS) {
      const int n = (cu_seqlens[b + 1] - cu_seqlens[b] + rows - 1) / rows;
      if (n > 0) atomicAdd(&cnt[min(n, max_tiles) - 1], 1);   // histogram by tile count first
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      int seqs = 0, entries = base;
      for (int t = max_tiles - 1; t >= 0; --t) {
        seqs += cnt[t];          // sequences with more than t tiles
        off[t] = entries;
        entries += seqs;
        cnt[t] = 0;
      }
      base = entries;
    }
    __syncthreads();
    for (int b = g0 + threadIdx.x; b < g1; b += PLAN_THREADS) {
      const int lo = cu_seqlens[b], len = cu_seqlens[b + 1] - lo;
      const int n = min((len + rows - 1) / rows, max_tiles);
      for (int t = 0; t < n; ++t) plan[off[t] + atomicAdd(&cnt[t], 1)] = make_int4(lo + t * rows, len - t * rows, t, b);
    }
  }
}

// ------------------------------------------------------------------------------------------------
// host side: tensor maps over the packed [total, H, 128] bf16 tensors, box = 64 columns x 1 head x 128 tokens
// ------------------------------------------------------------------------------------------------
using tcmap::make_map;

}  // namespace

cudaError_t launch_tile_plan(const int32_t* cu_seqlens, int batch, int max_seqlen, int rows, int group_seqs, void* plan,
                             cudaStream_t st) {
  const cudaError_t e = launch_pdl(prefill_plan_kernel, dim3(1), dim3(PLAN_THREADS), 0, st, cu_seqlens, batch,
                                   (max_seqlen + rows - 1) / rows, rows, group_seqs, reinterpret_cast<int4*>(plan));
  note_launch();
  return e != cudaSuccess ? e : cudaGetLastError();
}

int prefill_rows_per_entry(int n_q_heads, int n_kv_heads) {
  // an even group: the two M-tiles of an item are two heads on the same 128 rows; otherwise two consecutive query tiles
  return (n_q_heads / n_kv_heads) % 2 == 0 ? BM : NT * BM;
}

int prefill_plan_entries(const earn_batch_t& b, int rows) {
  int64_t n = 0;
  for (int i = 0; i < b.batch; ++i) n += (b.cu_seqlens_host[i + 1] - b.cu_seqlens_host[i] + rows - 1) / rows;
  return n > INT32_MAX ? INT32_MAX : (int)n;
}

bool prefill_tc_supported(const PrefillArgs& a, int total_tokens) {
  return a.dtype == EARN_BF16 && a.D == HD && total_tokens >= BM && (a.max_seqlen + BM - 1) / BM <= PLAN_MAX_LEVELS;
}

cudaError_t launch_prefill_tc(const PrefillArgs& a, int total_tokens, int plan_entries, void* plan, int32_t* status_word,
                              cudaStream_t st) {
  CUtensorMap mq, mk, mv, mo;
  if (!make_map(&mq, a.q, a.Hq, total_tokens, BM) || !make_map(&mk, a.k, a.Hkv, total_tokens, BM) ||
      !make_map(&mv, a.v, a.Hkv, total_tokens, BM) || !make_map(&mo, a.o, a.Hq, total_tokens, 32))   // O leaves in slabs of 32 rows, one per warp
    return cudaErrorInvalidValue;
  if (plan_entries <= 0) return cudaSuccess;
  const int rows = prefill_rows_per_entry(a.Hq, a.Hkv);
  // sequences per group of the plan: about 32 MB of K and V rows (a quarter of the L2 cache; measured at the 7B
  // shapes: 596 us per layer with groups of 8 sequences, 600 with 16, 612 with 32, 615 with the whole batch as one)
  const int64_t kv_bytes_per_seq = (int64_t)total_tokens / (a.batch > 0 ? a.batch : 1) * a.Hkv * HD * 2 * 2;
  const int group_seqs = (int)std::max<int64_t>(1, (32LL << 20) / std::max<int64_t>(kv_bytes_per_seq, 1));
  cudaError_t e = launch_tile_plan(a.cu_seqlens, a.batch, a.max_seqlen, rows, group_seqs, plan, st);
  if (e != cudaSuccess) return e;
  TcParams p{};
  p.o = a.o; p.lse = a.lse; p.plan = reinterpret_cast<const int4*>(plan); p.status = status_word;
  p.Hq = a.Hq; p.g = a.Hq / a.Hkv; p.total = total_tokens;
  const bool pair_tiles = rows != BM;
  p.n_hp = pair_tiles ? a.Hq : a.Hq / NT;
  p.n_items = plan_entries * p.n_hp;
  p.scale_log2 = a.scale * kLog2e;
  const int grid = p.n_items < sm_count() ? p.n_items : sm_count();
  if (pair_tiles) {
    e = ensure_dynamic_smem<prefill_tc_kernel<true>>(Cfg::SMEM_BYTES);
    if (e == cudaSuccess)
      e = launch_pdl(prefill_tc_kernel<true>, dim3(grid), dim3(Cfg::THREADS), Cfg::SMEM_BYTES, st, mq, mk, mv, mo, p);
  } else {
    e = ensure_dynamic_smem<prefill_tc_kernel<false>>(Cfg::SMEM_BYTES);
    if (e == cudaSuccess)
      e = launch_pdl(prefill_tc_kernel<false>, dim3(grid), dim3(Cfg::THREADS), Cfg::SMEM_BYTES, st, mq, mk, mv, mo, p);
  }
  note_launch();
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace earn
