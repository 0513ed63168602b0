// The register-focused process as the paper states it (Section 3.2, inference): the hidden state entering a layer
// l >= k is cut down to the register rows, X -> X' = [X_prefix; X_suffix], and only those rows are projected
// (Eq. 2).  Per layer: gather the R register rows of every sequence, RMS-normalise them, multiply by W_qkv^T on the
// tensor cores, rotate Q and K by the registers' ORIGINAL positions, and write Q' to q_reg and K', V' straight into
// the pages of the compact cache -- the full-length K/V of such a layer are never computed, let alone read.
//
// Two kernels:
//   gather_norm_kernel   one CTA per register row: 16-byte loads, fp32 sum of squares, bf16 row of
//                        X_n = x / rms(x) * w_norm into a [B*R, d_model] scratch; also writes reg_idx.
//   register_qkv_kernel  persistent tcgen05 GEMM  C[B*R, (Hq+2Hkv)*D] = X_n W_qkv^T  with 128 x 256 tiles (two heads):
//                          warp 0    TMA: X_n and W_qkv k-blocks of 64 columns -> shared memory (128-byte swizzle), 4 stages
//                          warp 1    one thread issues tcgen05.mma 128x256x16 into one of two TMEM accumulators
//                          warps 4-7 epilogue, one output row per thread: TMEM -> registers, rotary embedding from the
//                                    caller's cos / sin tables (pairs (i, i + D/2) sit in the same thread), bf16, 256-byte
//                                    rows to q_reg or to the cache page of that register, while the tensor core fills
//                                    the other accumulator.
// Every mbarrier wait is bounded; a wait that runs out sets EARN_ERR_TIMEOUT in the status word and the CTA leaves.
#include <cudaTypedefs.h>

#include "earn_common.cuh"
#include "sm100_ptx.cuh"

namespace earn {
namespace {
using namespace ptx;

constexpr int BM = 128, BK = 64, HD = 128;
constexpr int A_BYTES = BM * BK * 2;
// Tile geometry for an output tile of BN columns (256: two heads; 128: one head, for grids that would otherwise leave
// most SMs without a tile): ring of 192 KB either way.
template <int BN>
struct Tile {
  static constexpr int B_BYTES = BN * BK * 2, STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int NSTAGE = BN == 256 ? 4 : 6;
  static constexpr int SMEM_BYTES = NSTAGE * STAGE_BYTES + 256 + 1024;
  static constexpr int BAR_FULL = 0, BAR_EMPTY = NSTAGE, BAR_ACC_FULL = 2 * NSTAGE, BAR_ACC_EMPTY = BAR_ACC_FULL + 2,
                       BAR_DRAIN = BAR_ACC_EMPTY + 2, N_BARS = BAR_DRAIN + 1;
  static_assert(8 * N_BARS + 16 <= 256, "barrier block");
};
constexpr int THREADS = 256;
constexpr long long WAIT_LIMIT = 2000000000LL;

struct QkvParams {
  void* q_reg;
  KeySource cache;                 // compact pages (k, v are written here)
  const int32_t* cu_seqlens;
  const float* rope_cos;
  const float* rope_sin;
  int32_t* status;
  int M, K, n_heads, Hq, Hkv, R, r_head, r_tail, m_tiles, n_tiles, max_pos;
};

__device__ __forceinline__ int register_position(int m, int len, int r_head, int r_tail) {
  return m < r_head ? m : len - r_tail + (m - r_head);
}

// ---------------------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) gather_norm_kernel(const __nv_bfloat16* x, int x_is_compact, const __nv_bfloat16* w_norm,
                                                          __nv_bfloat16* xn, const int32_t* cu_seqlens, int32_t* reg_idx,
                                                          int R, int r_head, int r_tail, int d_model, float eps) {
  pdl_launch_dependents();
  pdl_wait();
  const int row = blockIdx.x, b = row / R, m = row % R;
  const int lo = cu_seqlens[b], len = cu_seqlens[b + 1] - lo;
  const int pos = register_position(m, len, r_head, r_tail);
  if (reg_idx != nullptr && threadIdx.x == 0) reg_idx[row] = pos;
  const uint4* src = reinterpret_cast<const uint4*>(x + (x_is_compact ? (int64_t)row : (int64_t)lo + pos) * d_model);
  const uint4* wsrc = reinterpret_cast<const uint4*>(w_norm);
  uint4* dst = reinterpret_cast<uint4*>(xn + (int64_t)row * d_model);
  const int n_vec = d_model / 8;
  float ss = 0.f;
  for (int i = threadIdx.x; i < n_vec; i += blockDim.x) {
    const uint4 v = __ldg(src + i);
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float2 f = __bfloat1622float2(h[e]);
      ss += f.x * f.x + f.y * f.y;
    }
  }
  __shared__ float red[8];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int i = 0; i < 8; ++i) tot += red[i];
  const float inv = rsqrtf(tot / (float)d_model + eps);
  for (int i = threadIdx.x; i < n_vec; i += blockDim.x) {
    const uint4 v = __ldg(src + i), wv = __ldg(wsrc + i);
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&v);
    const __nv_bfloat162* wh = reinterpret_cast<const __nv_bfloat162*>(&wv);
    uint4 out;
    uint32_t* oh = reinterpret_cast<uint32_t*>(&out);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float2 f = __bfloat1622float2(h[e]), g = __bfloat1622float2(wh[e]);
      oh[e] = pack_bf16(f.x * inv * g.x, f.y * inv * g.y);
    }
    dst[i] = out;
  }
}

// ---------------------------------------------------------------------------------------------------------------
template <int BN>
__global__ void __launch_bounds__(THREADS, 1)
register_qkv_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, QkvParams p) {
  using T = Tile<BN>;
  constexpr int NSTAGE = T::NSTAGE, STAGE_BYTES = T::STAGE_BYTES, N_BARS = T::N_BARS;
  constexpr int BAR_FULL = T::BAR_FULL, BAR_EMPTY = T::BAR_EMPTY, BAR_ACC_FULL = T::BAR_ACC_FULL,
                BAR_ACC_EMPTY = T::BAR_ACC_EMPTY, BAR_DRAIN = T::BAR_DRAIN;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* gen = smem_raw + (base - smem_u32(smem_raw));
  const uint32_t bars = base + NSTAGE * STAGE_BYTES;
  auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(gen + NSTAGE * STAGE_BYTES + 8 * N_BARS);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(gen + NSTAGE * STAGE_BYTES + 8 * N_BARS + 8);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < NSTAGE; ++s) {
      mbar_init(bar(BAR_FULL + s), 1);
      mbar_init(bar(BAR_EMPTY + s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(bar(BAR_ACC_FULL + a), 1);
      mbar_init(bar(BAR_ACC_EMPTY + a), 128);
    }
    mbar_init(bar(BAR_DRAIN), 1);
    *abort_flag = 0;
    fence_barrier_init();
    tma_prefetch_desc(&map_a);
    tma_prefetch_desc(&map_b);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), 2 * BN);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const int n_tiles_total = p.m_tiles * p.n_tiles, k_blocks = p.K / BK;
  pdl_launch_dependents();
  pdl_wait();   // X_n comes from the kernel launched just before this one

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer
    if (lane == 0) {
      int e = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < n_tiles_total && ok; t += gridDim.x) {
        const int mt = t % p.m_tiles, nt = t / p.m_tiles;   // consecutive CTAs share a block of W_qkv
        for (int kb = 0; kb < k_blocks; ++kb, ++e) {
          const int st = e % NSTAGE;
          if (e >= NSTAGE && !mbar_wait_bounded(bar(BAR_EMPTY + st), ((e / NSTAGE) - 1) & 1, abort_flag, WAIT_LIMIT)) {
            ok = false;
            break;
          }
          mbar_expect_tx(bar(BAR_FULL + st), STAGE_BYTES);
          tma_load_2d(base + st * STAGE_BYTES, &map_a, bar(BAR_FULL + st), kb * BK, mt * BM);
          tma_load_2d(base + st * STAGE_BYTES + A_BYTES, &map_b, bar(BAR_FULL + st), kb * BK, nt * BN);
        }
      }
      if (*abort_flag) {
        int none = 0;
        for (int f = max(e - NSTAGE, 0); f < e; ++f)
          mbar_wait_bounded(bar(BAR_FULL + f % NSTAGE), (f / NSTAGE) & 1, &none, WAIT_LIMIT);
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = idesc_bf16_f32(BM, BN, 0, 0);   // both operands K-major
      constexpr uint32_t desc_hi = smem_desc_hi_sw128(1024);
      int e = 0, n_acc = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < n_tiles_total && ok; t += gridDim.x, ++n_acc) {
        const int acc = n_acc & 1;
        if (n_acc >= 2) ok = mbar_wait_bounded(bar(BAR_ACC_EMPTY + acc), ((n_acc >> 1) - 1) & 1, abort_flag, WAIT_LIMIT);
        if (!ok) break;
        tc_fence_after();
        for (int kb = 0; kb < k_blocks && ok; ++kb, ++e) {
          const int st = e % NSTAGE;
          ok = mbar_wait_bounded(bar(BAR_FULL + st), (e / NSTAGE) & 1, abort_flag, WAIT_LIMIT);
          if (!ok) break;
          tc_fence_after();
          const uint32_t a_lo = smem_desc_lo(base + st * STAGE_BYTES, 16), b_lo = smem_desc_lo(base + st * STAGE_BYTES + A_BYTES, 16);
#pragma unroll
          for (int kk = 0; kk < BK / 16; ++kk)
            umma_ss_lohi(tmem + acc * BN, a_lo + kk * 2, desc_hi, b_lo + kk * 2, desc_hi, idesc, (kb > 0 || kk > 0) ? 1u : 0u);
          umma_commit(bar(BAR_EMPTY + st));
        }
        if (ok) umma_commit(bar(BAR_ACC_FULL + acc));
      }
      if (*abort_flag) {
        int none = 0;
        umma_commit(bar(BAR_DRAIN));
        mbar_wait_bounded(bar(BAR_DRAIN), 0, &none, WAIT_LIMIT);
      }
    }
  } else if (warp >= 4) {
    // ---------------------------------------------------------------- epilogue: one output row per thread
    const int wq = warp & 3, row_in_tile = wq * 32 + lane;
    int n_acc = 0;
    bool ok = true;
    for (int t = blockIdx.x; t < n_tiles_total && ok; t += gridDim.x, ++n_acc) {
      const int mt = t % p.m_tiles, nt = t / p.m_tiles, acc = n_acc & 1;
      ok = __all_sync(0xffffffffu, mbar_wait_bounded(bar(BAR_ACC_FULL + acc), (n_acc >> 1) & 1, abort_flag, WAIT_LIMIT));
      if (!ok) break;
      tc_fence_after();
      const int row = mt * BM + row_in_tile;
      const bool valid = row < p.M;
      const int b = valid ? row / p.R : 0, m = valid ? row % p.R : 0;
      const int len = p.cu_seqlens[b + 1] - p.cu_seqlens[b];
      const int pos = min(register_position(m, len, p.r_head, p.r_tail), p.max_pos - 1);
      const float* cs = p.rope_cos + (int64_t)pos * (HD / 2);
      const float* sn = p.rope_sin + (int64_t)pos * (HD / 2);
      const int64_t page_row = valid ? key_row(p.cache, b, m) : 0;
      // destination row and kind of each of the tile's two heads (0..Hq-1: Q; then Hkv K heads; then Hkv V heads)
      __nv_bfloat16* dst[BN / HD];
      bool rotate[BN / HD];
#pragma unroll
      for (int hh = 0; hh < BN / HD; ++hh) {
        const int head = nt * (BN / HD) + hh;
        dst[hh] = nullptr;
        rotate[hh] = head < p.Hq + p.Hkv;
        if (valid && head < p.n_heads) {
          if (head < p.Hq)
            dst[hh] = reinterpret_cast<__nv_bfloat16*>(p.q_reg) + ((int64_t)row * p.Hq + head) * HD;
          else if (head < p.Hq + p.Hkv)
            dst[hh] = reinterpret_cast<__nv_bfloat16*>(const_cast<void*>(p.cache.k)) + (page_row * p.Hkv + (head - p.Hq)) * HD;
          else
            dst[hh] = reinterpret_cast<__nv_bfloat16*>(const_cast<void*>(p.cache.v)) + (page_row * p.Hkv + (head - p.Hq - p.Hkv)) * HD;
        }
      }
      // Columns i and i + 64 of a head rotate together: chunk q (32 columns) is fetched with chunk q + 2.  The angles
      // depend on the row and on i only, so one fetch of cos / sin serves both heads of the tile.
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        float4 c4[8], s4[8];
        if (rotate[0]) {   // heads are ordered Q, K, V: if the first does not rotate, neither does the second
#pragma unroll
          for (int c = 0; c < 8; ++c) {
            c4[c] = __ldg(reinterpret_cast<const float4*>(cs + q * 32) + c);
            s4[c] = __ldg(reinterpret_cast<const float4*>(sn + q * 32) + c);
          }
        }
        const float* co = reinterpret_cast<const float*>(c4);
        const float* si = reinterpret_cast<const float*>(s4);
#pragma unroll
        for (int hh = 0; hh < BN / HD; ++hh) {
          const uint32_t t_acc = tmem + ((uint32_t)(wq * 32) << 16) + acc * BN + hh * HD;
          uint32_t lo[32], hi[32];
          tmem_ld_32x32(t_acc + q * 32, lo);
          tmem_ld_32x32(t_acc + (q + 2) * 32, hi);
          tmem_wait_ld(lo);
          tmem_wait_ld(hi);
          if (dst[hh] != nullptr) {
            if (rotate[hh]) {
#pragma unroll
              for (int c = 0; c < 32; ++c) {
                const float a = __uint_as_float(lo[c]), bb = __uint_as_float(hi[c]);
                lo[c] = __float_as_uint(a * co[c] - bb * si[c]);
                hi[c] = __float_as_uint(bb * co[c] + a * si[c]);
              }
            }
#pragma unroll
            for (int c = 0; c < 4; ++c) {
              uint4 w0, w1;
              w0.x = pack_bf16(__uint_as_float(lo[c * 8 + 0]), __uint_as_float(lo[c * 8 + 1]));
              w0.y = pack_bf16(__uint_as_float(lo[c * 8 + 2]), __uint_as_float(lo[c * 8 + 3]));
              w0.z = pack_bf16(__uint_as_float(lo[c * 8 + 4]), __uint_as_float(lo[c * 8 + 5]));
              w0.w = pack_bf16(__uint_as_float(lo[c * 8 + 6]), __uint_as_float(lo[c * 8 + 7]));
              w1.x = pack_bf16(__uint_as_float(hi[c * 8 + 0]), __uint_as_float(hi[c * 8 + 1]));
              w1.y = pack_bf16(__uint_as_float(hi[c * 8 + 2]), __uint_as_float(hi[c * 8 + 3]));
              w1.z = pack_bf16(__uint_as_float(hi[c * 8 + 4]), __uint_as_float(hi[c * 8 + 5]));
              w1.w = pack_bf16(__uint_as_float(hi[c * 8 + 6]), __uint_as_float(hi[c * 8 + 7]));
              *reinterpret_cast<uint4*>(dst[hh] + q * 32 + c * 8) = w0;
              *reinterpret_cast<uint4*>(dst[hh] + (q + 2) * 32 + c * 8) = w1;
            }
          }
        }
      }
      tc_fence_before();
      mbar_arrive(bar(BAR_ACC_EMPTY + acc));   // this accumulator may be overwritten
    }
  }

  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) atomicExch(p.status, (int32_t)EARN_ERR_TIMEOUT);
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, 2 * BN);
  }
}

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

// [rows, cols] bf16 row-major, box = 64 columns x box_rows rows, 128-byte swizzle; rows past the tensor read as zero
bool make_map_2d(CUtensorMap* map, const void* ptr, int rows, int cols, int box_rows) {
  auto fn = encode_fn();
  if (fn == nullptr) return false;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  cuuint32_t box[2] = {(cuuint32_t)BK, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int BN>
cudaError_t launch_gemm(const RegisterQkvArgs& a, QkvParams p, int M, int N, int sms, cudaStream_t st) {
  CUtensorMap ma, mb;
  if (!make_map_2d(&ma, a.x_norm, M, a.d_model, BM) || !make_map_2d(&mb, a.w_qkv, N, a.d_model, BN)) return cudaErrorInvalidValue;
  p.n_tiles = (N + BN - 1) / BN;
  cudaError_t e = ensure_dynamic_smem<register_qkv_kernel<BN>>(Tile<BN>::SMEM_BYTES);
  if (e != cudaSuccess) return e;
  const int tiles = p.m_tiles * p.n_tiles;
  e = launch_pdl(register_qkv_kernel<BN>, dim3(tiles < sms ? tiles : sms), dim3(THREADS), Tile<BN>::SMEM_BYTES, st, ma, mb, p);
  note_launch();
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace

cudaError_t launch_register_qkv(const RegisterQkvArgs& a, cudaStream_t st) {
  const int M = a.batch * a.R, n_heads = a.Hq + 2 * a.Hkv, N = n_heads * HD;
  cudaError_t e = launch_pdl(gather_norm_kernel, dim3(M), dim3(256), 0, st, reinterpret_cast<const __nv_bfloat16*>(a.x),
                             a.x_is_compact, reinterpret_cast<const __nv_bfloat16*>(a.w_norm),
                             reinterpret_cast<__nv_bfloat16*>(a.x_norm), a.cu_seqlens, a.reg_idx, a.R, a.r_head, a.r_tail,
                             a.d_model, a.rms_eps);
  note_launch();
  if (e == cudaSuccess) e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  QkvParams p{};
  p.q_reg = a.q_reg; p.cache = a.cache; p.cu_seqlens = a.cu_seqlens; p.rope_cos = a.rope_cos; p.rope_sin = a.rope_sin;
  p.status = a.status; p.M = M; p.K = a.d_model; p.n_heads = n_heads; p.Hq = a.Hq; p.Hkv = a.Hkv; p.R = a.R;
  p.r_head = a.r_head; p.r_tail = a.r_tail; p.max_pos = a.max_pos;
  p.m_tiles = (M + BM - 1) / BM;
  // Two heads per tile unless that leaves most of the GPU idle: with few register rows (a batch of 24 prompts with
  // two registers each is ONE row tile) the layer is a stream of W_qkv, and one-head tiles put twice as many SMs on it.
  const int sms = sm_count();
  const bool narrow = (long)p.m_tiles * ((N + 255) / 256) * 3 <= 2L * sms;
  return narrow ? launch_gemm<128>(a, p, M, N, sms, st) : launch_gemm<256>(a, p, M, N, sms, st);
}

}  // namespace earn
