// Full causal prefill attention (Eq. 3 + causal mask, layers l < k) on the Blackwell tensor cores.
// bf16 Q/K/V, head_dim 128, fp32 logits / softmax / accumulation, bf16 output.
//
// One CTA = 128 query rows of one (sequence, query head).  Per 128-key tile:
//   TMA      : K and V tiles -> shared memory (128-byte swizzle), two stages
//   tcgen05  : S = Q K^T into tensor memory (TMEM columns 0..127), issued by one thread
//   softmax  : 128 threads, one query row each: read S from TMEM, online softmax in the log2 domain,
//              write P as bf16 into swizzled shared memory
//   tcgen05  : O += P V into TMEM columns 128..255
// The running output stays in TMEM.  The softmax reference maximum is only raised when the row maximum
// grows by more than 2^8; then the owning warp rescales its 32 rows of O in TMEM.  Exact after the
// final division by the row sum.
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
constexpr int KV_STAGES = 2;
constexpr int OFF_Q = 0;
constexpr int OFF_K = OFF_Q + TILE;
constexpr int OFF_V = OFF_K + KV_STAGES * TILE;
constexpr int OFF_P = OFF_V + KV_STAGES * TILE;
constexpr int OFF_BAR = OFF_P + TILE;
constexpr int SMEM_BYTES = OFF_BAR + 256 + 1024;   // + alignment slack
constexpr int TMEM_COLS = 256;
constexpr long long WAIT_LIMIT = 2000000000LL;     // about one second of SM clocks
constexpr float RESCALE_THRESHOLD = 8.f;           // log2 units

enum { BAR_Q = 0, BAR_K = 1, BAR_V = 3, BAR_KV_EMPTY = 5, BAR_S = 7, BAR_P = 8, BAR_O = 9, BAR_DRAIN = 10, N_BARS = 11 };

struct TcParams {
  void* o;
  float* lse;
  const int32_t* cu_seqlens;
  int32_t* status;
  int Hq, g, total;
  float scale_log2;
};

__global__ void __launch_bounds__(192, 1)
prefill_tc_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                  const __grid_constant__ CUtensorMap map_v, TcParams p) {
  const int b = blockIdx.z, h = blockIdx.y;
  const int lo = p.cu_seqlens[b], L = p.cu_seqlens[b + 1] - lo;
  const int q0 = ((int)gridDim.x - 1 - (int)blockIdx.x) * BM;   // longest tiles first
  if (q0 >= L) return;
  const int n_tiles = q0 / BN + 1;                                // causal: key tiles 0 .. diagonal
  const int kvh = h / p.g;

  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;    // swizzled tiles need 1024-byte alignment
  uint8_t* gen = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t sQ = base + OFF_Q, sK = base + OFF_K, sV = base + OFF_V, sP = base + OFF_P;
  const uint32_t bars = base + OFF_BAR;
  auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gen + OFF_BAR + 8 * N_BARS);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gen + OFF_BAR + 8 * N_BARS + 8);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    mbar_init(bar(BAR_Q), 1);
    for (int s = 0; s < KV_STAGES; ++s) {
      mbar_init(bar(BAR_K + s), 1);
      mbar_init(bar(BAR_V + s), 1);
      mbar_init(bar(BAR_KV_EMPTY + s), 1);
    }
    mbar_init(bar(BAR_S), 1);
    mbar_init(bar(BAR_P), 128);
    mbar_init(bar(BAR_O), 1);
    mbar_init(bar(BAR_DRAIN), 1);
    *abort_flag = 0;
    fence_barrier_init();
    tma_prefetch_desc(&map_q);
    tma_prefetch_desc(&map_k);
    tma_prefetch_desc(&map_v);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      mbar_expect_tx(bar(BAR_Q), TILE);
      tma_load_3d(sQ, &map_q, bar(BAR_Q), 0, h, lo + q0);
      tma_load_3d(sQ + HALF, &map_q, bar(BAR_Q), 64, h, lo + q0);
      int issued = 0;
      bool ok = true;
      for (int j = 0; j < n_tiles && ok; ++j) {
        const int st = j % KV_STAGES;
        if (j >= KV_STAGES) ok = mbar_wait_bounded(bar(BAR_KV_EMPTY + st), ((j / KV_STAGES) - 1) & 1, abort_flag, WAIT_LIMIT);
        if (!ok) break;
        mbar_expect_tx(bar(BAR_K + st), TILE);
        tma_load_3d(sK + st * TILE, &map_k, bar(BAR_K + st), 0, kvh, lo + j * BN);
        tma_load_3d(sK + st * TILE + HALF, &map_k, bar(BAR_K + st), 64, kvh, lo + j * BN);
        mbar_expect_tx(bar(BAR_V + st), TILE);
        tma_load_3d(sV + st * TILE, &map_v, bar(BAR_V + st), 0, kvh, lo + j * BN);
        tma_load_3d(sV + st * TILE + HALF, &map_v, bar(BAR_V + st), 64, kvh, lo + j * BN);
        issued = j + 1;
      }
      if (*abort_flag) {
        // let the copies already in flight land before the CTA gives its shared memory back
        int none = 0;
        mbar_wait_bounded(bar(BAR_Q), 0, &none, WAIT_LIMIT);
        for (int j = max(issued - KV_STAGES, 0); j < issued; ++j) {
          mbar_wait_bounded(bar(BAR_K + j % KV_STAGES), (j / KV_STAGES) & 1, &none, WAIT_LIMIT);
          mbar_wait_bounded(bar(BAR_V + j % KV_STAGES), (j / KV_STAGES) & 1, &none, WAIT_LIMIT);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_s = idesc_bf16_f32(BM, BN, 0, 0);   // Q (K-major) x K^T (K-major)
      constexpr uint32_t idesc_o = idesc_bf16_f32(BM, HD, 0, 1);   // P (K-major) x V (MN-major)
      bool ok = mbar_wait_bounded(bar(BAR_Q), 0, abort_flag, WAIT_LIMIT);
      for (int j = 0; j < n_tiles && ok; ++j) {
        const int st = j % KV_STAGES, ph = (j / KV_STAGES) & 1;
        ok = mbar_wait_bounded(bar(BAR_K + st), ph, abort_flag, WAIT_LIMIT);
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < HD / 16; ++kk) {
          const uint32_t off = (kk >> 2) * HALF + (kk & 3) * 32;
          umma_ss(tmem, smem_desc_sw128(sQ + off, 16, 1024), smem_desc_sw128(sK + st * TILE + off, 16, 1024), idesc_s, kk > 0);
        }
        umma_commit(bar(BAR_S));
        ok = mbar_wait_bounded(bar(BAR_P), j & 1, abort_flag, WAIT_LIMIT) &&
             mbar_wait_bounded(bar(BAR_V + st), ph, abort_flag, WAIT_LIMIT);
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int kk = 0; kk < BN / 16; ++kk) {
          const uint32_t offp = (kk >> 2) * HALF + (kk & 3) * 32;
          umma_ss(tmem + 128, smem_desc_sw128(sP + offp, 16, 1024), smem_desc_sw128(sV + st * TILE + kk * 2048, HALF, 1024),
                  idesc_o, (j > 0 || kk > 0) ? 1u : 0u);
        }
        umma_commit(bar(BAR_KV_EMPTY + st));
        if (j == n_tiles - 1) umma_commit(bar(BAR_O));
      }
      if (*abort_flag) {
        int none = 0;
        umma_commit(bar(BAR_DRAIN));   // everything this thread issued has retired once this fires
        mbar_wait_bounded(bar(BAR_DRAIN), 0, &none, WAIT_LIMIT);
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax: warps 2..5, one row per thread
    const int wq = warp & 3;            // a warp may only touch TMEM lanes 32*(warp % 4) ..
    const int row = wq * 32 + lane;
    const uint32_t t_row = tmem + ((uint32_t)(wq * 32) << 16);
    const uint32_t p_row = sP + row * 128;
    const uint32_t sw = (uint32_t)(row & 7);
    float m_ref = 0.f, l = 0.f;
    bool ok = true;
    for (int j = 0; j < n_tiles; ++j) {
      ok = __all_sync(0xffffffffu, mbar_wait_bounded(bar(BAR_S), j & 1, abort_flag, WAIT_LIMIT));   // warp-uniform
      if (!ok) break;
      tc_fence_after();
      uint32_t s[4][32];
#pragma unroll
      for (int q = 0; q < 4; ++q) tmem_ld_32x32(t_row + q * 32, s[q]);
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
        // the commit that signalled S_j also covers P V of tile j-1, so O is quiescent here
        l *= alpha;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          uint32_t o[32];
          tmem_ld_32x32(t_row + 128 + q * 32, o);
          tmem_wait_ld();
#pragma unroll
          for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * alpha);
          tmem_st_32x32(t_row + 128 + q * 32, o);
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
      mbar_arrive(bar(BAR_P));
    }
    if (ok) ok = __all_sync(0xffffffffu, mbar_wait_bounded(bar(BAR_O), 0, abort_flag, WAIT_LIMIT));
    if (ok) {
      tc_fence_after();
      const float inv = 1.f / l;
      const bool valid = q0 + row < L;
      __nv_bfloat16* orow = reinterpret_cast<__nv_bfloat16*>(p.o) + ((int64_t)(lo + q0 + row) * p.Hq + h) * HD;
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        uint32_t o[32];
        tmem_ld_32x32(t_row + 128 + q * 32, o);
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
    tmem_dealloc(tmem, TMEM_COLS);
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

}  // namespace

bool prefill_tc_supported(const PrefillArgs& a, int total_tokens) {
  return a.dtype == EARN_BF16 && a.D == HD && total_tokens >= BM;
}

cudaError_t launch_prefill_tc(const PrefillArgs& a, int total_tokens, int32_t* status_word, cudaStream_t st) {
  CUtensorMap mq, mk, mv;
  if (!make_map(&mq, a.q, a.Hq, total_tokens) || !make_map(&mk, a.k, a.Hkv, total_tokens) ||
      !make_map(&mv, a.v, a.Hkv, total_tokens))
    return cudaErrorInvalidValue;
  cudaError_t e = ensure_dynamic_smem<prefill_tc_kernel>(SMEM_BYTES);
  if (e != cudaSuccess) return e;
  TcParams p{};
  p.o = a.o; p.lse = a.lse; p.cu_seqlens = a.cu_seqlens; p.status = status_word;
  p.Hq = a.Hq; p.g = a.Hq / a.Hkv; p.total = total_tokens;
  p.scale_log2 = a.scale * kLog2e;
  dim3 grid((a.max_seqlen + BM - 1) / BM, a.Hq, a.batch);
  prefill_tc_kernel<<<grid, 192, SMEM_BYTES, st>>>(mq, mk, mv, p);
  note_launch();
  return cudaGetLastError();
}

}  // namespace earn
