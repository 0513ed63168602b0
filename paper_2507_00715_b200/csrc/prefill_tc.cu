// Full causal prefill attention (Eq. 3 + causal mask, layers l < k) on the Blackwell tensor cores.
// bf16 Q/K/V, head_dim 128, fp32 logits / softmax / accumulation, bf16 output.
//
// One CTA = 128 query rows of NT query heads that share a kv head (NT = 2 when the GQA group size is
// even, else 1): NT "M-tiles" with the same rows and the same key range, so they share every K/V tile
// and finish together.  Per 128-key tile:
//   warp 0     TMA: K and V tiles -> shared memory (128-byte swizzle), a ring of 32 KB entries K0 V0 K1 V1 ..
//   warp 1     one thread issues tcgen05.mma: S_x = Q_x K^T into tensor memory, later O_x += P_x V
//   warps 4..  one softmax warpgroup per M-tile, one query row per thread: read S_x from TMEM, online softmax
//              in the log2 domain, write P_x as bf16 into swizzled shared memory
// With two M-tiles the tensor core works on one while the other is in its softmax (S_A, S_B, O_A, O_B fill
// the 512 TMEM columns).  The running output stays in TMEM.  The softmax reference maximum is only raised
// when the row maximum grows by more than 2^8; then the owning warp rescales its 32 rows of O in TMEM.
// Exact after the final division by the row sum.
//
// Every mbarrier wait is bounded; when one runs out the CTA raises its abort flag, writes
// EARN_ERR_TIMEOUT to the status word, drains what it has in flight, frees its TMEM and returns.
#include <cudaTypedefs.h>

#include "earn_common.cuh"
#include "sm100_ptx.cuh"

namespace earn {
namespace {
using namespace ptx;

constexpr int BM = 128, BN = 128, HD = 128;
constexpr int TILE = BM * HD * 2;   // bytes of one 128 x 128 bf16 tile
constexpr int HALF = TILE / 2;      // one 64-column block of it (128 rows x 128 B)
constexpr long long WAIT_LIMIT = 2000000000LL;     // about one second of SM clocks
constexpr float RESCALE_THRESHOLD = 8.f;           // log2 units

template <int NT>
struct Cfg {
  static constexpr int NSTAGE = NT == 1 ? 4 : 3;            // ring entries (K and V tiles alternate)
  static constexpr int OFF_Q = 0;
  static constexpr int OFF_RING = OFF_Q + NT * TILE;
  static constexpr int OFF_P = OFF_RING + NSTAGE * TILE;
  static constexpr int OFF_BAR = OFF_P + NT * TILE;
  static constexpr int SMEM_BYTES = OFF_BAR + 256 + 1024;   // + alignment slack
  static constexpr int TMEM_COLS = NT * 256;                // S_x at x*128, O_x at (NT + x)*128
  static constexpr int THREADS = 32 * (4 + 4 * NT);
  // barriers
  static constexpr int BAR_Q = 0, BAR_FULL = 1, BAR_EMPTY = BAR_FULL + NSTAGE, BAR_S = BAR_EMPTY + NSTAGE,
                       BAR_P = BAR_S + NT, BAR_O = BAR_P + NT, BAR_DRAIN = BAR_O + NT, N_BARS = BAR_DRAIN + 1;
};

struct TcParams {
  void* o;
  float* lse;
  const int32_t* cu_seqlens;
  int32_t* status;
  int Hq, g, total;
  float scale_log2;
};

template <int NT>
__global__ void __launch_bounds__(Cfg<NT>::THREADS, 1)
prefill_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                  const __grid_constant__ CUtensorMap map_v, TcParams p) {
  using C = Cfg<NT>;
  const int b = blockIdx.z, h0 = blockIdx.y * NT;
  const int lo = p.cu_seqlens[b], L = p.cu_seqlens[b + 1] - lo;
  const int q0 = ((int)gridDim.x - 1 - (int)blockIdx.x) * BM;   // longest tiles first
  if (q0 >= L) return;
  const int n_tiles = q0 / BN + 1;                                // causal: key tiles 0 .. diagonal
  const int kvh = h0 / p.g;

  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;    // swizzled tiles need 1024-byte alignment
  uint8_t* gen = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t sQ = base + C::OFF_Q, sRing = base + C::OFF_RING, sP = base + C::OFF_P;
  const uint32_t bars = base + C::OFF_BAR;
  auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gen + C::OFF_BAR + 8 * C::N_BARS);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gen + C::OFF_BAR + 8 * C::N_BARS + 8);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    mbar_init(bar(C::BAR_Q), 1);
    for (int s = 0; s < C::NSTAGE; ++s) {
      mbar_init(bar(C::BAR_FULL + s), 1);
      mbar_init(bar(C::BAR_EMPTY + s), 1);
    }
    for (int x = 0; x < NT; ++x) {
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
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), C::TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const int n_entries = 2 * n_tiles;   // ring entries: K_0 V_0 K_1 V_1 ...

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      mbar_expect_tx(bar(C::BAR_Q), NT * TILE);
      for (int x = 0; x < NT; ++x) {
        tma_load_3d(sQ + x * TILE, &map_q, bar(C::BAR_Q), 0, h0 + x, lo + q0);
        tma_load_3d(sQ + x * TILE + HALF, &map_q, bar(C::BAR_Q), 64, h0 + x, lo + q0);
      }
      int issued = 0;
      for (int e = 0; e < n_entries; ++e) {
        const int st = e % C::NSTAGE;
        if (e >= C::NSTAGE &&
            !mbar_wait_bounded(bar(C::BAR_EMPTY + st), ((e / C::NSTAGE) - 1) & 1, abort_flag, WAIT_LIMIT))
          break;
        const CUtensorMap* map = (e & 1) ? &map_v : &map_k;
        mbar_expect_tx(bar(C::BAR_FULL + st), TILE);
        tma_load_3d(sRing + st * TILE, map, bar(C::BAR_FULL + st), 0, kvh, lo + (e >> 1) * BN);
        tma_load_3d(sRing + st * TILE + HALF, map, bar(C::BAR_FULL + st), 64, kvh, lo + (e >> 1) * BN);
        issued = e + 1;
      }
      if (*abort_flag) {
        // let the copies already in flight land before the CTA gives its shared memory back
        int none = 0;
        mbar_wait_bounded(bar(C::BAR_Q), 0, &none, WAIT_LIMIT);
        for (int e = max(issued - C::NSTAGE, 0); e < issued; ++e)
          mbar_wait_bounded(bar(C::BAR_FULL + e % C::NSTAGE), (e / C::NSTAGE) & 1, &none, WAIT_LIMIT);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_s = idesc_bf16_f32(BM, BN, 0, 0);   // Q (K-major) x K^T (K-major)
      constexpr uint32_t idesc_o = idesc_bf16_f32(BM, HD, 0, 1);   // P (K-major) x V (MN-major)
      auto wait_full = [&](int e) {
        return mbar_wait_bounded(bar(C::BAR_FULL + e % C::NSTAGE), (e / C::NSTAGE) & 1, abort_flag, WAIT_LIMIT);
      };
      auto issue_s = [&](int x, int e) {   // S_x = Q_x K^T with the K tile of ring entry e
        const uint32_t sK = sRing + (e % C::NSTAGE) * TILE;
#pragma unroll
        for (int kk = 0; kk < HD / 16; ++kk) {
          const uint32_t off = (kk >> 2) * HALF + (kk & 3) * 32;
          umma_ss(tmem + x * 128, smem_desc_sw128(sQ + x * TILE + off, 16, 1024), smem_desc_sw128(sK + off, 16, 1024),
                  idesc_s, kk > 0);
        }
        umma_commit(bar(C::BAR_S + x));
        if (x == NT - 1) umma_commit(bar(C::BAR_EMPTY + e % C::NSTAGE));   // K tile free once the last S has read it
      };
      auto issue_pv = [&](int x, int e, bool first) {   // O_x (+)= P_x V with the V tile of ring entry e
        const uint32_t sV = sRing + (e % C::NSTAGE) * TILE;
#pragma unroll
        for (int kk = 0; kk < BN / 16; ++kk) {
          const uint32_t offp = (kk >> 2) * HALF + (kk & 3) * 32;
          umma_ss(tmem + (NT + x) * 128, smem_desc_sw128(sP + x * TILE + offp, 16, 1024),
                  smem_desc_sw128(sV + kk * 2048, HALF, 1024), idesc_o, (!first || kk > 0) ? 1u : 0u);
        }
        if (x == NT - 1) umma_commit(bar(C::BAR_EMPTY + e % C::NSTAGE));   // V tile free once the last P V has read it
      };
      bool ok = mbar_wait_bounded(bar(C::BAR_Q), 0, abort_flag, WAIT_LIMIT) && wait_full(0);
      if (ok) {
        tc_fence_after();
        for (int x = 0; x < NT; ++x) issue_s(x, 0);
      }
      for (int j = 0; j < n_tiles && ok; ++j) {
        for (int x = 0; x < NT && ok; ++x) {
          ok = mbar_wait_bounded(bar(C::BAR_P + x), j & 1, abort_flag, WAIT_LIMIT);   // P_x(j) written, S_x free
          if (ok && x == 0) ok = wait_full(2 * j + 1);
          if (!ok) break;
          tc_fence_after();
          issue_pv(x, 2 * j + 1, j == 0);
          if (j == n_tiles - 1) {
            umma_commit(bar(C::BAR_O + x));
          } else {
            if (x == 0) ok = wait_full(2 * j + 2);
            if (!ok) break;
            tc_fence_after();
            issue_s(x, 2 * j + 2);
          }
        }
      }
      if (*abort_flag) {
        int none = 0;
        umma_commit(bar(C::BAR_DRAIN));   // everything this thread issued has retired once this fires
        mbar_wait_bounded(bar(C::BAR_DRAIN), 0, &none, WAIT_LIMIT);
      }
    }
  } else if (warp >= 4) {
    // ------------------------------------------------------------------ softmax warpgroup x, one row per thread
    const int x = (warp - 4) >> 2;
    const int h = h0 + x;
    const int wq = warp & 3;            // a warp may only touch TMEM lanes 32*(warp % 4) ..
    const int row = wq * 32 + lane;
    const uint32_t t_s = tmem + ((uint32_t)(wq * 32) << 16) + x * 128;
    const uint32_t t_o = tmem + ((uint32_t)(wq * 32) << 16) + (NT + x) * 128;
    const uint32_t p_row = sP + x * TILE + row * 128;
    const uint32_t sw = (uint32_t)(row & 7);
    float m_ref = 0.f, l = 0.f;
    bool ok = true;
    for (int j = 0; j < n_tiles; ++j) {
      ok = __all_sync(0xffffffffu, mbar_wait_bounded(bar(C::BAR_S + x), j & 1, abort_flag, WAIT_LIMIT));   // warp-uniform
      if (!ok) break;
      tc_fence_after();
      uint32_t s[4][32];
#pragma unroll
      for (int q = 0; q < 4; ++q) tmem_ld_32x32(t_s + q * 32, s[q]);
      tmem_wait_ld();
      if (j == n_tiles - 1) {   // diagonal tile: key column c is visible to row r iff c <= r
#pragma unroll
        for (int q = 0; q < 4; ++q)
#pragma unroll
          for (int c = 0; c < 32; ++c)
            if (q * 32 + c > row) s[q][c] = 0xff800000u;   // -inf
      }
      float mx = -INFINITY;
#pragma unroll
      for (int q = 0; q < 4; ++q)
#pragma unroll
        for (int c = 0; c < 32; ++c) mx = fmaxf(mx, __uint_as_float(s[q][c]));
      mx *= p.scale_log2;
      float alpha = 1.f;
      bool grow = false;
      if (j == 0) {
        m_ref = mx;
      } else if (mx > m_ref + RESCALE_THRESHOLD) {
        alpha = ex2(m_ref - mx);
        m_ref = mx;
        grow = true;
      }
      if (__any_sync(0xffffffffu, grow)) {
        // S_x(j) was issued after P_x V of tile j-1, so the commit that signalled it covers that too: O_x is quiescent
        l *= alpha;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          uint32_t o[32];
          tmem_ld_32x32(t_o + q * 32, o);
          tmem_wait_ld();
#pragma unroll
          for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * alpha);
          tmem_st_32x32(t_o + q * 32, o);
        }
        tmem_wait_st();
      }
      float sum = 0.f;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
#pragma unroll
        for (int c8 = 0; c8 < 4; ++c8) {
          float e[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            e[i] = ex2(fmaf(__uint_as_float(s[q][c8 * 8 + i]), p.scale_log2, -m_ref));
            sum += e[i];
          }
          const uint32_t chunk = (uint32_t)((q & 1) * 4 + c8);
          const uint32_t addr = p_row + (q >> 1) * HALF + ((chunk ^ sw) << 4);
          asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(pack_bf16(e[0], e[1])),
                       "r"(pack_bf16(e[2], e[3])), "r"(pack_bf16(e[4], e[5])), "r"(pack_bf16(e[6], e[7]))
                       : "memory");
        }
      }
      l += sum;
      fence_async_smem();   // P was written through the generic proxy; the tensor core reads it through the async proxy
      tc_fence_before();
      mbar_arrive(bar(C::BAR_P + x));
    }
    if (ok) ok = __all_sync(0xffffffffu, mbar_wait_bounded(bar(C::BAR_O + x), 0, abort_flag, WAIT_LIMIT));
    if (ok) {
      tc_fence_after();
      const float inv = 1.f / l;
      const bool valid = q0 + row < L;
      __nv_bfloat16* orow = reinterpret_cast<__nv_bfloat16*>(p.o) + ((int64_t)(lo + q0 + row) * p.Hq + h) * HD;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        uint32_t o[32];
        tmem_ld_32x32(t_o + q * 32, o);
        tmem_wait_ld();
        if (valid) {
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            uint4 w;
            w.x = pack_bf16(__uint_as_float(o[c * 8 + 0]) * inv, __uint_as_float(o[c * 8 + 1]) * inv);
            w.y = pack_bf16(__uint_as_float(o[c * 8 + 2]) * inv, __uint_as_float(o[c * 8 + 3]) * inv);
            w.z = pack_bf16(__uint_as_float(o[c * 8 + 4]) * inv, __uint_as_float(o[c * 8 + 5]) * inv);
            w.w = pack_bf16(__uint_as_float(o[c * 8 + 6]) * inv, __uint_as_float(o[c * 8 + 7]) * inv);
            *reinterpret_cast<uint4*>(orow + q * 32 + c * 8) = w;
          }
        }
      }
      if (valid && p.lse != nullptr) p.lse[(int64_t)h * p.total + lo + q0 + row] = (m_ref + log2f(l)) * kLn2;
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

// ------------------------------------------------------------------------------------------------
// host side: tensor maps over the packed [total, H, 128] bf16 tensors, box = 64 columns x 1 head x 128 tokens
// ------------------------------------------------------------------------------------------------
PFN_cuTensorMapEncodeTiled_v12000 encode_fn() {
  static PFN_cuTensorMapEncodeTiled_v12000 fn = [] {
    void* f = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      f = nullptr;
    return reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(f);
  }();
  return fn;
}

bool make_map(CUtensorMap* map, const void* ptr, int heads, int total) {
  auto fn = encode_fn();
  if (fn == nullptr) return false;
  cuuint64_t dims[3] = {(cuuint64_t)HD, (cuuint64_t)heads, (cuuint64_t)total};
  cuuint64_t strides[2] = {(cuuint64_t)HD * 2, (cuuint64_t)heads * HD * 2};
  cuuint32_t box[3] = {64, 1, (cuuint32_t)BM};
  cuuint32_t estr[3] = {1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int NT>
cudaError_t launch_nt(const PrefillArgs& a, const CUtensorMap& mq, const CUtensorMap& mk, const CUtensorMap& mv,
                      const TcParams& p, cudaStream_t st) {
  cudaError_t e = ensure_dynamic_smem<prefill_tc_kernel<NT>>(Cfg<NT>::SMEM_BYTES);
  if (e != cudaSuccess) return e;
  dim3 grid((a.max_seqlen + BM - 1) / BM, a.Hq / NT, a.batch);
  prefill_tc_kernel<NT><<<grid, Cfg<NT>::THREADS, Cfg<NT>::SMEM_BYTES, st>>>(mq, mk, mv, p);
  note_launch();
  return cudaGetLastError();
}

}  // namespace

bool prefill_tc_supported(const PrefillArgs& a, int total_tokens) {
  return a.dtype == EARN_BF16 && a.D == HD && total_tokens >= BM;
}

cudaError_t launch_prefill_tc(const PrefillArgs& a, int total_tokens, int32_t* status_word, cudaStream_t st) {
  CUtensorMap mq, mk, mv;
  if (!make_map(&mq, a.q, a.Hq, total_tokens) || !make_map(&mk, a.k, a.Hkv, total_tokens) ||
      !make_map(&mv, a.v, a.Hkv, total_tokens))
    return cudaErrorInvalidValue;
  TcParams p{};
  p.o = a.o; p.lse = a.lse; p.cu_seqlens = a.cu_seqlens; p.status = status_word;
  p.Hq = a.Hq; p.g = a.Hq / a.Hkv; p.total = total_tokens;
  p.scale_log2 = a.scale * kLog2e;
  // two query heads of one kv head per CTA when the group size allows it
  return (p.g % 2 == 0) ? launch_nt<2>(a, mq, mk, mv, p, st) : launch_nt<1>(a, mq, mk, mv, p, st);
}

}  // namespace earn
