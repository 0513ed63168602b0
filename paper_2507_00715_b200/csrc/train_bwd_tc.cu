// Backward of full causal attention (the layers l < k of a training sample, Section 3.2 "Training") on the Blackwell
// tensor cores.  bf16 Q/K/V/O/dO, head_dim 128, fp32 accumulation, bf16 gradients.
//
//   P = exp(S c - LSE),   dV = P^T dO,   dP = dO V^T,   dS = P o (dP - delta),   dQ = dS K c,   dK = dS^T Q c
// with S = Q K^T, c the logit scale, LSE the forward's log-sum-exp and delta = rowsum(dO o O) (a small kernel ahead).
//
// Two launches of one kernel, each deterministic and free of atomics (S and dP are computed in both):
//   MODE_KV  one CTA per (sequence, tile of 128 keys, kv head): K_j, V_j stay in shared memory; the Q_i, dO_i tiles of
//            every query head of the group and every query tile i >= j stream through a two-stage ring; dV_j and dK_j
//            accumulate in tensor memory over the whole loop (the heads of a group add up there).
//   MODE_Q   one CTA per (sequence, tile of 128 queries, query head): Q_i, dO_i stay; K_j, V_j (j <= i) stream; dQ_i
//            accumulates in tensor memory.
// The two modes are the same pipeline with rows and keys exchanged.  "Left" = the resident pair (L0, L1), "streamed" =
// the ring pair (T0, T1); lane l of tensor memory is row l of the left tile, columns run over the streamed tile:
//   X  = L0 T0^T   (S^T = K Q^T  or  S = Q K^T)        Y = L1 T1^T   (dP^T = V dO^T  or  dP = dO V^T)
//   softmax warpgroup, one lane per thread: p = exp2(X c log2e - LSE), ds = p (Y - delta), both written back to tensor
//   memory as bf16 over the first 64 columns of X and of Y
//   MODE_KV: acc0 += p T1 (dV += P^T dO)      both modes: acc1 += ds T0 (dK += dS^T Q  or  dQ += dS K)
// so every tensor-core product has the shapes and operand layouts of the forward kernel's two (left operand K-major
// from shared memory, or from tensor memory; right operand K-major or MN-major from a TMA-loaded tile).
//   warp 0  TMA producer    warp 1  tcgen05.mma issuer (and TMEM owner)    warps 4-11  two softmax warpgroups, 64 columns each
// All 512 TMEM columns are taken (X, Y, acc0, acc1), so there is no second X / Y to work ahead on; the overlap comes from
// the issue order Y(u) | acc0(u) | X(u+1) | acc1(u): the warpgroups turn X(u) into p while the tensor core does acc1(u-1)
// and Y(u), and Y(u) into ds while it does acc0(u) and X(u+1); X(u+1) only waits for p(u) to have been handed over
// (issued tile by tile as X Y, then acc0 acc1, the tensor core and the warpgroups took turns).
// Every mbarrier wait is bounded as in the forward kernel.
#include <type_traits>

#include "earn_common.cuh"
#include "sm100_ptx.cuh"
#include "tc_maps.cuh"

namespace earn {
namespace {
using namespace ptx;

constexpr int BM = 128, HD = 128;
constexpr int TILE = BM * HD * 2, HALF = TILE / 2;
constexpr long long WAIT_LIMIT = 2000000000LL;
constexpr int MODE_KV = 0, MODE_Q = 1;

struct BCfg {
  static constexpr int NSTAGE = 2;
  static constexpr int OFF_L = 0;                                   // L0, L1
  static constexpr int OFF_T = OFF_L + 2 * TILE;                    // NSTAGE x (T0, T1)
  static constexpr int OFF_STAT = OFF_T + NSTAGE * 2 * TILE;        // NSTAGE x (lse2[128], delta[128]) fp32
  static constexpr int OFF_BAR = OFF_STAT + NSTAGE * 2 * BM * 4;
  static constexpr int SMEM_BYTES = OFF_BAR + 256 + 1024;           // + alignment slack
  static constexpr int TMEM_COLS = 512;                             // X 0, Y 128, acc0 256, acc1 384
  static constexpr int THREADS = 384;                               // TMA, MMA, two idle warps, two softmax warpgroups
  static constexpr int BAR_RES = 0, BAR_FULL = 1, BAR_EMPTY = BAR_FULL + NSTAGE, BAR_X = BAR_EMPTY + NSTAGE,
                       BAR_Y = BAR_X + 1, BAR_P = BAR_Y + 1, BAR_DS = BAR_P + 1, BAR_ACC = BAR_DS + 1,
                       BAR_DRAIN = BAR_ACC + 1, N_BARS = BAR_DRAIN + 1;
};

struct BwdParams {
  const int4* plan;       // {first global row of the tile, rows of the sequence from there, tile index, sequence}
  const float* lse2;      // [Hq, total] log2-domain LSE
  const float* delta;     // [Hq, total]
  void *dq, *dk, *dv;
  int32_t* status;
  int Hq, Hkv, g, total, n_entries;
  float scale, scale_log2;
};

// what one CTA works on
struct Job {
  int left_row0;    // global row of the left (resident) tile
  int left_valid;   // rows of it that belong to the sequence (1..128)
  int n_iter;       // streamed tiles
  int n_t;          // streamed tiles per head (MODE_KV: query tiles i >= j; MODE_Q: key tiles j <= i)
  int t_row0;       // global row of the first streamed tile
  int rows_left;    // rows of the sequence from t_row0 on (MODE_KV: bounds the valid query rows of streamed tile u)
  int head0;        // MODE_KV: first query head of the group; MODE_Q: the query head
  int kvh;
};

template <int MODE>
__device__ __forceinline__ Job make_job(const BwdParams& p) {
  Job j;
  // The plan is sequence-major (all tiles of sequence 0, then of sequence 1, ...), low tile indices first: the CTAs that
  // run at the same time then work on two or three sequences, whose Q / dO (MODE_KV) or K / V (MODE_Q) tiles they share
  // through L2.  (Ordered by tile index over the whole batch, longest items first, the dK / dV launch read 5.2 GB from
  // DRAM for a 7B-class layer whose Q and dO are 1.07 GB: every key tile's CTA fetched its query tiles afresh.)
  if (MODE == MODE_KV) {
    const int e = (int)blockIdx.x / p.Hkv;
    const int4 t = __ldg(p.plan + e);
    j.kvh = blockIdx.x % p.Hkv;
    j.head0 = j.kvh * p.g;
    j.left_row0 = t.x;
    j.left_valid = min(t.y, BM);
    j.n_t = (t.y + BM - 1) / BM;
    j.n_iter = j.n_t * p.g;
    j.t_row0 = t.x;
    j.rows_left = t.y;
  } else {
    // entry (sequence, tile z) stands for query tile nt - 1 - z here: within a sequence the long items come first
    const int e = (int)blockIdx.x / p.Hq;
    const int4 t = __ldg(p.plan + e);
    const int lo = t.x - t.z * BM, len = t.y + t.z * BM, i = (len + BM - 1) / BM - 1 - t.z;
    j.head0 = blockIdx.x % p.Hq;
    j.kvh = j.head0 / p.g;
    j.left_row0 = lo + i * BM;
    j.left_valid = min(len - i * BM, BM);
    j.n_t = i + 1;
    j.n_iter = j.n_t;
    j.t_row0 = lo;
    j.rows_left = len;
  }
  return j;
}

template <int MODE>
__global__ void __launch_bounds__(BCfg::THREADS, 1)
train_bwd_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                    const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_do,
                    const __grid_constant__ CUtensorMap map_out0, const __grid_constant__ CUtensorMap map_out1, BwdParams p) {
  // map_out0 / map_out1: MODE_KV dV and dK, MODE_Q unused and dQ (boxes of 32 rows x 64 columns, one per warp)
  using C = BCfg;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t sL = base + C::OFF_L, sT = base + C::OFF_T, bars = base + C::OFF_BAR;
  float* stat = reinterpret_cast<float*>(gen + C::OFF_STAT);
  auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gen + C::OFF_BAR + 8 * C::N_BARS);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gen + C::OFF_BAR + 8 * C::N_BARS + 8);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    mbar_init(bar(C::BAR_RES), 1);
    for (int s = 0; s < C::NSTAGE; ++s) {
      mbar_init(bar(C::BAR_FULL + s), 1);
      mbar_init(bar(C::BAR_EMPTY + s), 1);
    }
    mbar_init(bar(C::BAR_X), 1);
    mbar_init(bar(C::BAR_Y), 1);
    mbar_init(bar(C::BAR_P), 256);
    mbar_init(bar(C::BAR_DS), 256);
    mbar_init(bar(C::BAR_ACC), 1);
    mbar_init(bar(C::BAR_DRAIN), 1);
    *abort_flag = 0;
    fence_barrier_init();
    tma_prefetch_desc(&map_q);
    tma_prefetch_desc(&map_k);
    tma_prefetch_desc(&map_v);
    tma_prefetch_desc(&map_do);
    tma_prefetch_desc(&map_out0);
    tma_prefetch_desc(&map_out1);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), C::TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  pdl_launch_dependents();
  pdl_wait();   // the plan, delta and the log2-domain LSE come from the kernels launched just before this one
  const Job job = make_job<MODE>(p);
  // the left pair and the streamed pair: (K, V) and (Q, dO), one way round or the other
  const CUtensorMap* mapL0 = MODE == MODE_KV ? &map_k : &map_q;
  const CUtensorMap* mapL1 = MODE == MODE_KV ? &map_v : &map_do;
  const CUtensorMap* mapT0 = MODE == MODE_KV ? &map_q : &map_k;
  const CUtensorMap* mapT1 = MODE == MODE_KV ? &map_do : &map_v;
  // streamed tile of iteration u: MODE_KV head head0 + u / n_t, query tile u % n_t; MODE_Q kv head, key tile u
  auto t_head = [&](int u) { return MODE == MODE_KV ? job.head0 + u / job.n_t : job.kvh; };
  auto t_row = [&](int u) { return job.t_row0 + (MODE == MODE_KV ? u % job.n_t : u) * BM; };

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      const int lh = MODE == MODE_KV ? job.kvh : job.head0;
      mbar_expect_tx(bar(C::BAR_RES), 2 * TILE);
      tma_load_3d(sL, mapL0, bar(C::BAR_RES), 0, lh, job.left_row0);
      tma_load_3d(sL + HALF, mapL0, bar(C::BAR_RES), 64, lh, job.left_row0);
      tma_load_3d(sL + TILE, mapL1, bar(C::BAR_RES), 0, lh, job.left_row0);
      tma_load_3d(sL + TILE + HALF, mapL1, bar(C::BAR_RES), 64, lh, job.left_row0);
      int u = 0;
      for (; u < job.n_iter; ++u) {
        const int st = u % C::NSTAGE;
        if (u >= C::NSTAGE && !mbar_wait_bounded(bar(C::BAR_EMPTY + st), ((u / C::NSTAGE) - 1) & 1, abort_flag, WAIT_LIMIT)) break;
        const uint32_t dst = sT + st * 2 * TILE;
        mbar_expect_tx(bar(C::BAR_FULL + st), 2 * TILE);
        tma_load_3d(dst, mapT0, bar(C::BAR_FULL + st), 0, t_head(u), t_row(u));
        tma_load_3d(dst + HALF, mapT0, bar(C::BAR_FULL + st), 64, t_head(u), t_row(u));
        tma_load_3d(dst + TILE, mapT1, bar(C::BAR_FULL + st), 0, t_head(u), t_row(u));
        tma_load_3d(dst + TILE + HALF, mapT1, bar(C::BAR_FULL + st), 64, t_head(u), t_row(u));
      }
      if (*abort_flag) {   // let the copies already in flight land before the CTA gives its shared memory back
        int none = 0;
        mbar_wait_bounded(bar(C::BAR_RES), 0, &none, WAIT_LIMIT);
        for (int f = max(u - C::NSTAGE, 0); f < u; ++f)
          mbar_wait_bounded(bar(C::BAR_FULL + f % C::NSTAGE), (f / C::NSTAGE) & 1, &none, WAIT_LIMIT);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (the whole warp runs the loop, lane 0 issues)
    const bool leader = lane == 0;
    constexpr uint32_t idesc_xy = idesc_bf16_f32(BM, BM, 0, 0);    // left (K-major) x streamed^T (K-major)
    constexpr uint32_t idesc_acc = idesc_bf16_f32(BM, HD, 0, 1);   // p / ds (tensor memory) x streamed tile (MN-major)
    constexpr uint32_t desc_hi = smem_desc_hi_sw128(1024);
    const uint32_t l_lo = smem_desc_lo(sL, 16);
    auto wait = [&](int b, int parity) {
      return __all_sync(0xffffffffu, mbar_wait_bounded(bar(b), (uint32_t)parity & 1u, abort_flag, WAIT_LIMIT));
    };
    // D = A B^T over the 128-wide inner dimension, both operands K-major tiles (two 64-column halves)
    auto issue_xy = [&](uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo) {
      if (leader) {
#pragma unroll
        for (int kk = 0; kk < HD / 16; ++kk) {
          const uint32_t off = ((kk >> 2) * HALF + (kk & 3) * 32) >> 4;
          umma_ss_lohi(d_tmem, a_lo + off, desc_hi, b_lo + off, desc_hi, idesc_xy, kk > 0);
        }
      }
    };
    // D (+)= A B with A = 128 x 128 bf16 in tensor memory (64 columns) and B a [128 inner x 128] tile, MN-major
    auto issue_acc = [&](uint32_t d_tmem, uint32_t a_tmem, uint32_t b_addr, bool first) {
      const uint32_t b_lo = smem_desc_lo(b_addr, HALF);
      if (leader) {
#pragma unroll
        for (int kk = 0; kk < BM / 16; ++kk)
          umma_ts_lohi(d_tmem, a_tmem + kk * 8, b_lo + kk * (2048 >> 4), desc_hi, idesc_acc, (!first || kk > 0) ? 1u : 0u);
      }
    };
    // Order on the tensor core, per streamed tile u:  Y(u) | acc0(u) | X(u+1) | acc1(u)  -- the softmax warpgroups turn
    // X(u) into p while acc1(u-1) and Y(u) run, and Y(u) into ds while acc0(u) and X(u+1) run.  One thread's tensor-core
    // instructions run in the order they were issued, which is what lets X(u+1) go over the columns acc0(u) reads p
    // from, and Y(u+1) over the columns acc1(u) reads ds from.
    bool ok = wait(C::BAR_RES, 0) && wait(C::BAR_FULL + 0, 0);
    if (ok) {
      tc_fence_after();
      issue_xy(tmem + 0, l_lo, smem_desc_lo(sT, 16));
      if (leader) umma_commit(bar(C::BAR_X));
      issue_xy(tmem + 128, l_lo + (TILE >> 4), smem_desc_lo(sT + TILE, 16));
      if (leader) umma_commit(bar(C::BAR_Y));
    }
    for (int u = 0; u < job.n_iter && ok; ++u) {
      const int st = u % C::NSTAGE, sn = (u + 1) % C::NSTAGE;
      const uint32_t t0 = sT + st * 2 * TILE, t1 = t0 + TILE, n0 = sT + sn * 2 * TILE, n1 = n0 + TILE;
      const bool more = u + 1 < job.n_iter;
      // P(u) released: MODE_KV p is in tensor memory; MODE_Q every softmax thread has its part of X(u) in registers
      ok = wait(C::BAR_P, u);
      if (ok && more) ok = wait(C::BAR_FULL + sn, (u + 1) / C::NSTAGE);
      if (!ok) break;
      tc_fence_after();
      if (MODE == MODE_KV) issue_acc(tmem + 256, tmem + 0, t1, u == 0);      // dV += P^T dO
      if (more) {   // X(u+1) runs while the warpgroups are still on ds(u)
        issue_xy(tmem + 0, l_lo, smem_desc_lo(n0, 16));
        if (leader) umma_commit(bar(C::BAR_X));
      }
      ok = wait(C::BAR_DS, u);
      if (!ok) break;
      tc_fence_after();
      issue_acc(tmem + 384, tmem + 128, t0, u == 0);      // dK += dS^T Q   or   dQ += dS K
      if (leader) {
        umma_commit(bar(C::BAR_EMPTY + st));
        if (!more) umma_commit(bar(C::BAR_ACC));
      }
      if (more) {
        issue_xy(tmem + 128, l_lo + (TILE >> 4), smem_desc_lo(n1, 16));
        if (leader) umma_commit(bar(C::BAR_Y));
      }
    }
    if (leader && *abort_flag) {
      int none = 0;
      umma_commit(bar(C::BAR_DRAIN));
      mbar_wait_bounded(bar(C::BAR_DRAIN), 0, &none, WAIT_LIMIT);
    }
    __syncwarp();
  } else if (warp >= 4) {
    // ------------------------------------------------------------------ two softmax warpgroups: thread = lane l of tensor
    // memory; warpgroup wg takes columns 64 wg .. 64 wg + 63 of X and of Y (one warpgroup over all 128 columns was bound
    // by the instructions one warp per scheduler can issue: about 1900 clocks per pass)
    const int wq = warp & 3, l = wq * 32 + lane, wg = (warp - 4) >> 2, c0 = wg * 64;
    const uint32_t t_lane = tmem + ((uint32_t)(wq * 32) << 16);
    const uint32_t t_x = t_lane + c0, t_y = t_lane + 128 + c0;
    const float sl2 = p.scale_log2;
    // MODE_Q: the thread's own query row has one LSE and one delta for the whole item
    float my_lse = 0.f, my_delta = 0.f;
    if (MODE == MODE_Q && l < job.left_valid) {
      const int64_t at = (int64_t)job.head0 * p.total + job.left_row0 + l;
      my_lse = __ldg(p.lse2 + at);
      my_delta = __ldg(p.delta + at);
    }
    // MODE_KV: LSE and delta belong to the streamed query rows: thread l of the first warpgroup fetches those of row l
    // of the tile one iteration ahead and both warpgroups read them from shared memory
    auto fetch_stat = [&](int u, float& a_lse, float& a_delta) {
      a_lse = 0.f;
      a_delta = 0.f;
      if (MODE == MODE_KV && wg == 0 && u < job.n_iter) {
        const int it = u % job.n_t;
        if (it * BM + l < job.rows_left) {
          const int64_t at = (int64_t)t_head(u) * p.total + t_row(u) + l;
          a_lse = __ldg(p.lse2 + at);
          a_delta = __ldg(p.delta + at);
        }
      }
    };
    float nx_lse, nx_delta;
    fetch_stat(0, nx_lse, nx_delta);
    bool ok = true;
    for (int u = 0; u < job.n_iter && ok; ++u) {
      const int st = u % C::NSTAGE;
      const float* s_lse = stat + st * 2 * BM;
      const float* s_delta = s_lse + BM;
      // streamed tile index within the sequence relative to the left tile (0 = the diagonal tile), valid columns
      const int rel = MODE == MODE_KV ? u % job.n_t : job.n_t - 1 - u;
      const bool diag = rel == 0;
      const int col_valid = MODE == MODE_KV ? min(job.rows_left - rel * BM, BM) : BM;   // MODE_KV: query rows of the sequence in this tile
      const bool masked = diag || col_valid < BM;   // warp-uniform: interior tiles take the path without compares
      if (MODE == MODE_KV) {
        if (wg == 0) {
          stat[st * 2 * BM + l] = nx_lse;
          stat[st * 2 * BM + BM + l] = nx_delta;
        }
        asm volatile("bar.sync 1, 256;" ::: "memory");   // the softmax warps' own barrier
        fetch_stat(u + 1, nx_lse, nx_delta);
      }
      ok = __all_sync(0xffffffffu, mbar_wait_bounded(bar(C::BAR_X), u & 1, abort_flag, WAIT_LIMIT));
      if (!ok) break;
      tc_fence_after();
      // column c of the tile pairs with this lane iff both belong to the sequence and the key is not after the query:
      //   MODE_KV: lane = key, column = query row: c >= l on the diagonal tile, c < col_valid always
      //   MODE_Q : lane = query row, column = key: c <= l on the diagonal tile (keys past the sequence lie past every valid row)
      uint32_t a[32], b[32], pk[2][16];
      // ---- p = 2^(x c log2e - LSE) as bf16 pairs.  p goes over the first 64 columns of X, so the second warpgroup's
      // share lands on columns the first one reads: everybody has X in registers before anybody writes.
      tmem_ld_32x32(t_x, a);
      tmem_ld_32x32(t_x + 32, b);
      tmem_wait_ld(a);
      tmem_wait_ld(b);
      if (MODE == MODE_KV) {
        asm volatile("bar.sync 2, 256;" ::: "memory");
      } else {   // X(u) has been read (p stays in registers): the next X may go over it
        tc_fence_before();
        mbar_arrive(bar(C::BAR_P));
      }
      // Two copies of the loop, chosen once per tile: with the test for `masked` inside it, every group of four
      // columns became a basic block of its own and the pass ran at the latency of one group after another (1900
      // clocks for an interior tile, 6000 for a masked one, against 1300 for the loop without the test).
      // the columns this lane pairs with are vis_lo .. vis_lo + vis_n - 1
      const int vis_lo = (MODE == MODE_KV && diag) ? l : 0;
      const int vis_hi = MODE == MODE_KV ? col_valid : (diag ? l + 1 : BM);
      const uint32_t vis_n = (uint32_t)max(vis_hi - vis_lo, 0);
      auto p_pass = [&](auto masked_tag) {
        constexpr bool MASKED = decltype(masked_tag)::value;
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          uint32_t(&cur)[32] = q ? b : a;
#pragma unroll
          for (int c = 0; c < 32; c += 4) {
            const int col = c0 + q * 32 + c;
            float4 ls = make_float4(my_lse, my_lse, my_lse, my_lse);
            if (MODE == MODE_KV) ls = *reinterpret_cast<const float4*>(s_lse + col);
            float e[4];
            e[0] = ex2(fmaf(__uint_as_float(cur[c + 0]), sl2, -ls.x));
            e[1] = ex2(fmaf(__uint_as_float(cur[c + 1]), sl2, -ls.y));
            e[2] = ex2(fmaf(__uint_as_float(cur[c + 2]), sl2, -ls.z));
            e[3] = ex2(fmaf(__uint_as_float(cur[c + 3]), sl2, -ls.w));
            if (MASKED) {
#pragma unroll
              for (int z = 0; z < 4; ++z)   // one unsigned compare: vis_lo <= column < vis_lo + vis_n
                e[z] = (uint32_t)(col + z - vis_lo) < vis_n ? e[z] : 0.f;
            }
            pk[q][c >> 1] = pack_bf16(e[0], e[1]);
            pk[q][(c >> 1) + 1] = pack_bf16(e[2], e[3]);
          }
        }
      };
      if (masked) p_pass(std::true_type{});
      else p_pass(std::false_type{});
      ok = __all_sync(0xffffffffu, mbar_wait_bounded(bar(C::BAR_Y), u & 1, abort_flag, WAIT_LIMIT));
      if (!ok) break;
      tc_fence_after();
      tmem_ld_32x32(t_y, a);        // Y on its way while p is stored
      tmem_ld_32x32(t_y + 32, b);
      if (MODE == MODE_KV) {
        tmem_st_32x16(t_lane + wg * 32, pk[0]);
        tmem_st_32x16(t_lane + wg * 32 + 16, pk[1]);
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(bar(C::BAR_P));
      }
      tmem_wait_ld(a);
      tmem_wait_ld(b);
      asm volatile("bar.sync 3, 256;" ::: "memory");   // everybody has Y in registers before ds goes over its first 64 columns
      // ---- ds = p (y - delta) as bf16 pairs (p is exactly zero where the pair is masked; the difference is finite there:
      // every operand is real data or zero fill)
      uint32_t dsk[2][16];
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        uint32_t(&cur)[32] = q ? b : a;
#pragma unroll
        for (int c = 0; c < 32; c += 4) {
          const int col = c0 + q * 32 + c;
          float4 dl = make_float4(my_delta, my_delta, my_delta, my_delta);
          if (MODE == MODE_KV) dl = *reinterpret_cast<const float4*>(s_delta + col);
          const uint32_t pw0 = pk[q][c >> 1], pw1 = pk[q][(c >> 1) + 1];
          dsk[q][c >> 1] = pack_bf16(__uint_as_float(pw0 << 16) * (__uint_as_float(cur[c + 0]) - dl.x),
                                     __uint_as_float(pw0 & 0xffff0000u) * (__uint_as_float(cur[c + 1]) - dl.y));
          dsk[q][(c >> 1) + 1] = pack_bf16(__uint_as_float(pw1 << 16) * (__uint_as_float(cur[c + 2]) - dl.z),
                                           __uint_as_float(pw1 & 0xffff0000u) * (__uint_as_float(cur[c + 3]) - dl.w));
        }
      }
      tmem_st_32x16(t_lane + 128 + wg * 32, dsk[0]);
      tmem_st_32x16(t_lane + 128 + wg * 32 + 16, dsk[1]);
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(bar(C::BAR_DS));
    }
    // ---- the item's accumulators -> global memory (each warpgroup its half of the columns)
    if (ok) ok = __all_sync(0xffffffffu, mbar_wait_bounded(bar(C::BAR_ACC), 0, abort_flag, WAIT_LIMIT));
    if (ok) {
      tc_fence_after();
      const bool valid = l < job.left_valid;
      uint32_t a[32];
      auto store_rows = [&](uint32_t t_acc, void* out, int heads, int head, float mul) {
        __nv_bfloat16* orow = reinterpret_cast<__nv_bfloat16*>(out) + ((int64_t)(job.left_row0 + l) * heads + head) * HD + c0;
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          tmem_ld_32x32(t_acc + c0 + q * 32, a);
          tmem_wait_ld(a);
          if (valid) {
#pragma unroll
            for (int c = 0; c < 4; ++c) {
              uint4 w;
              w.x = pack_bf16(__uint_as_float(a[c * 8 + 0]) * mul, __uint_as_float(a[c * 8 + 1]) * mul);
              w.y = pack_bf16(__uint_as_float(a[c * 8 + 2]) * mul, __uint_as_float(a[c * 8 + 3]) * mul);
              w.z = pack_bf16(__uint_as_float(a[c * 8 + 4]) * mul, __uint_as_float(a[c * 8 + 5]) * mul);
              w.w = pack_bf16(__uint_as_float(a[c * 8 + 6]) * mul, __uint_as_float(a[c * 8 + 7]) * mul);
              *reinterpret_cast<uint4*>(orow + q * 32 + c * 8) = w;
            }
          }
        }
      };
      // A whole tile of the sequence leaves through shared memory and the copy engine instead (each thread writing its
      // own row with 16-byte stores puts 2048 half-sector writes per accumulator through the SM's one load/store unit:
      // about 3600 clocks, a quarter of a dQ item).  The resident pair's 64 KB are free once the last product has
      // retired: warp (wg, wq) stages its 32 rows x 64 columns there, 128-byte swizzled, and its first lane hands the
      // slab to the copy engine.  `slot` tells the two accumulators of MODE_KV apart.
      auto store_tile = [&](uint32_t t_acc, const CUtensorMap* map, int head, float mul, int slot) {
        const uint32_t out = sL + (uint32_t)(slot * 8 + (warp - 4)) * (32 * 128);
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          tmem_ld_32x32(t_acc + c0 + q * 32, a);
          tmem_wait_ld(a);
#pragma unroll
          for (int c = 0; c < 4; ++c) {   // 16-byte chunk q * 4 + c of the lane's 128-byte row, at chunk ^ (row % 8)
            const uint32_t w0 = pack_bf16(__uint_as_float(a[c * 8 + 0]) * mul, __uint_as_float(a[c * 8 + 1]) * mul);
            const uint32_t w1 = pack_bf16(__uint_as_float(a[c * 8 + 2]) * mul, __uint_as_float(a[c * 8 + 3]) * mul);
            const uint32_t w2 = pack_bf16(__uint_as_float(a[c * 8 + 4]) * mul, __uint_as_float(a[c * 8 + 5]) * mul);
            const uint32_t w3 = pack_bf16(__uint_as_float(a[c * 8 + 6]) * mul, __uint_as_float(a[c * 8 + 7]) * mul);
            const int ch = q * 4 + c;
            st_shared_v4(out + (uint32_t)lane * 128 + (uint32_t)((ch ^ (lane & 7)) << 4), w0, w1, w2, w3);
          }
        }
        fence_async_smem();
        __syncwarp();
        if (lane == 0) {
          tma_store_3d(map, out, c0, head, job.left_row0 + wq * 32);
          bulk_commit();
        }
      };
      if (job.left_valid == BM) {
        if (MODE == MODE_KV) {
          store_tile(t_lane + 256, &map_out0, job.kvh, 1.f, 0);
          store_tile(t_lane + 384, &map_out1, job.kvh, p.scale, 1);
        } else {
          store_tile(t_lane + 384, &map_out1, job.head0, p.scale, 0);
        }
        if (lane == 0) bulk_wait_all0();   // the copies have completed before the CTA gives its shared memory back
      } else
      if (MODE == MODE_KV) {
        store_rows(t_lane + 256, p.dv, p.Hkv, job.kvh, 1.f);
        store_rows(t_lane + 384, p.dk, p.Hkv, job.kvh, p.scale);
      } else {
        store_rows(t_lane + 384, p.dq, p.Hq, job.head0, p.scale);
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) atomicExch(p.status, (int32_t)EARN_ERR_TIMEOUT);
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, C::TMEM_COLS);
  }
}

// Sequence-major plan: entry (sequence b, tile z) = {first global row of the tile, rows of the sequence from there, z, b}
// at index (tiles of the sequences before b) + z.  One CTA; the sequences are scanned 1024 at a time.
__global__ void __launch_bounds__(1024) train_plan_kernel(const int32_t* cu_seqlens, int batch, int4* plan) {
  __shared__ int scan[1024];
  __shared__ int carry;
  pdl_launch_dependents();
  pdl_wait();   // the plan area may still be read by the kernel before this one
  if (threadIdx.x == 0) carry = 0;
  __syncthreads();
  for (int b0 = 0; b0 < batch; b0 += 1024) {
    const int b = b0 + threadIdx.x;
    const int lo = b < batch ? cu_seqlens[b] : 0, len = b < batch ? cu_seqlens[b + 1] - lo : 0;
    const int nt = (len + BM - 1) / BM;
    scan[threadIdx.x] = nt;
    __syncthreads();
    for (int off = 1; off < 1024; off <<= 1) {   // inclusive scan
      const int add = threadIdx.x >= off ? scan[threadIdx.x - off] : 0;
      __syncthreads();
      scan[threadIdx.x] += add;
      __syncthreads();
    }
    const int first = carry + scan[threadIdx.x] - nt;
    for (int z = 0; z < nt; ++z) plan[first + z] = make_int4(lo + z * BM, len - z * BM, z, b);
    __syncthreads();
    if (threadIdx.x == 1023) carry += scan[1023];
    __syncthreads();
  }
}

// delta[h][row] = sum_d dO[row, h, d] * O[row, h, d] and the forward's LSE moved into the log2 domain: one warp per (row, head)
__global__ void __launch_bounds__(256) train_bwd_prep_kernel(const __nv_bfloat16* o, const __nv_bfloat16* d_o, const float* lse,
                                                             float* delta, float* lse2, int total, int Hq) {
  pdl_launch_dependents();
  pdl_wait();
  const int64_t w = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (w >= (int64_t)total * Hq) return;
  const int row = (int)(w / Hq), h = (int)(w % Hq);
  const uint2 x = *reinterpret_cast<const uint2*>(o + w * HD + lane * 4);
  const uint2 y = *reinterpret_cast<const uint2*>(d_o + w * HD + lane * 4);
  float s = __uint_as_float(x.x << 16) * __uint_as_float(y.x << 16) +
            __uint_as_float(x.x & 0xffff0000u) * __uint_as_float(y.x & 0xffff0000u) +
            __uint_as_float(x.y << 16) * __uint_as_float(y.y << 16) +
            __uint_as_float(x.y & 0xffff0000u) * __uint_as_float(y.y & 0xffff0000u);
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
  if (lane == 0) {
    delta[(int64_t)h * total + row] = s;
    lse2[(int64_t)h * total + row] = lse[(int64_t)h * total + row] * kLog2e;
  }
}

}  // namespace

bool train_bwd_tc_supported(const TrainArgs& a) {
  return a.dtype == EARN_BF16 && a.D == HD && a.cu_seqlens != nullptr && a.total >= BM && (a.max_seqlen + BM - 1) / BM <= 2048;
}

cudaError_t launch_train_bwd_tc(const TrainArgs& a, const earn_batch_t& b, void* plan, cudaStream_t st) {
  using tcmap::make_map;
  CUtensorMap mq, mk, mv, mdo, mdq, mdk, mdv;
  if (!make_map(&mq, a.q, a.Hq, a.total, BM) || !make_map(&mk, a.k, a.Hkv, a.total, BM) ||
      !make_map(&mv, a.v, a.Hkv, a.total, BM) || !make_map(&mdo, a.d_o, a.Hq, a.total, BM) ||
      !make_map(&mdq, a.dq, a.Hq, a.total, 32) || !make_map(&mdk, a.dk, a.Hkv, a.total, 32) ||
      !make_map(&mdv, a.dv, a.Hkv, a.total, 32))   // gradients leave in slabs of 32 rows, one per warp
    return cudaErrorInvalidValue;
  const int n_entries = prefill_plan_entries(b, BM);
  if (n_entries <= 0) return cudaSuccess;
  cudaError_t e = launch_pdl(train_plan_kernel, dim3(1), dim3(1024), 0, st, a.cu_seqlens, a.batch, reinterpret_cast<int4*>(plan));
  note_launch();
  if (e == cudaSuccess) e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  const int64_t warps = (int64_t)a.total * a.Hq;
  e = launch_pdl(train_bwd_prep_kernel, dim3((unsigned)((warps + 7) / 8)), dim3(256), 0, st,
                 reinterpret_cast<const __nv_bfloat16*>(a.o), reinterpret_cast<const __nv_bfloat16*>(a.d_o),
                 (const float*)a.lse, a.delta, a.lse2, a.total, a.Hq);
  note_launch();
  if (e == cudaSuccess) e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  BwdParams p{};
  p.plan = reinterpret_cast<const int4*>(plan); p.lse2 = a.lse2; p.delta = a.delta;
  p.dq = a.dq; p.dk = a.dk; p.dv = a.dv; p.status = a.status;
  p.Hq = a.Hq; p.Hkv = a.Hkv; p.g = a.Hq / a.Hkv; p.total = a.total; p.n_entries = n_entries;
  p.scale = a.scale; p.scale_log2 = a.scale * kLog2e;
  e = ensure_dynamic_smem<train_bwd_tc_kernel<MODE_KV>>(BCfg::SMEM_BYTES);
  if (e == cudaSuccess)
    e = launch_pdl(train_bwd_tc_kernel<MODE_KV>, dim3((unsigned)((int64_t)n_entries * a.Hkv)), dim3(BCfg::THREADS),
                   BCfg::SMEM_BYTES, st, mq, mk, mv, mdo, mdv, mdk, p);
  note_launch();
  if (e == cudaSuccess) e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  e = ensure_dynamic_smem<train_bwd_tc_kernel<MODE_Q>>(BCfg::SMEM_BYTES);
  if (e == cudaSuccess)
    e = launch_pdl(train_bwd_tc_kernel<MODE_Q>, dim3((unsigned)((int64_t)n_entries * a.Hq)), dim3(BCfg::THREADS),
                   BCfg::SMEM_BYTES, st, mq, mk, mv, mdo, mdq, mdq, p);
  note_launch();
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace earn
