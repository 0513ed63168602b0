// Training-time attention on CUDA cores (Section 3.2 "Training"; forward = Eq. 3 with the causal mask, backward = the
// chain rule through it):
//   P = softmax(S), O = P V   =>   dV = P^T dO,  dP = dO V^T,  dS = P o (dP - rowsum(dO o O)),  dQ = dS K c,  dK = dS^T Q c.
// These kernels serve the layers after the split, where only the participating rows (registers and target tokens, a few
// dozen per sequence) are left, and every shape the tensor-core kernels do not take (fp32, head_dim 64).  fp32
// arithmetic throughout; one warp per output row, no atomics, so results are reproducible from launch to launch:
//   forward    warp = (query row i, query head h): lanes take keys j <= i 32 at a time for the logits, then own
//              D / 32 output columns each for P V (online softmax in the log2 domain); writes O and LSE;
//   dQ         warp = (query row i, query head h): recomputes p_ij from LSE, dp_ij = dO_i . V_j, then dq_i = c sum_j ds_ij K_j;
//   dK, dV     warp = (key j, kv head): lanes take the rows i >= j of every query head of the group 32 at a time.
#include "earn_common.cuh"

namespace earn {
namespace {

constexpr int TW = 4;   // warps per CTA

struct Seq { int lo, len; };
__device__ __forceinline__ Seq seq_of(const TrainArgs& a, int b) {
  if (a.cu_seqlens == nullptr) return {b * a.uniform_len, a.uniform_len};
  const int lo = a.cu_seqlens[b];
  return {lo, a.cu_seqlens[b + 1] - lo};
}
// LSE of (sequence b, head h, local row i): [Hq, total] for packed sequences, [B, Hq, P] for uniform ones
__device__ __forceinline__ int64_t lse_at(const TrainArgs& a, int b, int h, int lo, int i) {
  return a.cu_seqlens == nullptr ? ((int64_t)b * a.Hq + h) * a.uniform_len + i : (int64_t)h * a.total + lo + i;
}
template <typename T>
__device__ __forceinline__ float ld1(const T* p);
template <> __device__ __forceinline__ float ld1<float>(const float* p) { return *p; }
template <> __device__ __forceinline__ float ld1<__nv_bfloat16>(const __nv_bfloat16* p) { return __bfloat162float(*p); }
template <typename T>
__device__ __forceinline__ void st1(T* p, float x);
template <> __device__ __forceinline__ void st1<float>(float* p, float x) { *p = x; }
template <> __device__ __forceinline__ void st1<__nv_bfloat16>(__nv_bfloat16* p, float x) { *p = __float2bfloat16_rn(x); }

__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}
__device__ __forceinline__ float warp_max(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
  return x;
}
// dot product of a row held in shared memory (fp32, D values) with a row of a tensor in global memory
template <typename T, int D>
__device__ __forceinline__ float dot_row(const float* s, const T* g) {
  float acc = 0.f;
#pragma unroll 8
  for (int d = 0; d < D; d += 4) {
    float x[4];
    Elem<T>::load4(g + d, x);
    acc += s[d] * x[0] + s[d + 1] * x[1] + s[d + 2] * x[2] + s[d + 3] * x[3];
  }
  return acc;
}

// ------------------------------------------------------------------------------------------------ forward
template <typename T, int D>
__global__ void __launch_bounds__(TW * 32) train_fwd_kernel(TrainArgs a) {
  constexpr int C = D / 32;
  __shared__ float sq[TW][D];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int b = blockIdx.z, h = blockIdx.y, kvh = h / (a.Hq / a.Hkv);
  const Seq s = seq_of(a, b);
  const int i = blockIdx.x * TW + warp;
  if (i >= s.len) return;
  const T* qg = reinterpret_cast<const T*>(a.q) + ((int64_t)(s.lo + i) * a.Hq + h) * D;
  const T* kg = reinterpret_cast<const T*>(a.k) + ((int64_t)s.lo * a.Hkv + kvh) * D;
  const T* vg = reinterpret_cast<const T*>(a.v) + ((int64_t)s.lo * a.Hkv + kvh) * D;
  const int64_t kv_stride = (int64_t)a.Hkv * D;
  const float sl2 = a.scale * kLog2e;
  for (int d = lane; d < D; d += 32) sq[warp][d] = ld1(qg + d) * sl2;   // logits come out in the log2 domain
  __syncwarp();
  float m = -INFINITY, l = 0.f, acc[C];
#pragma unroll
  for (int c = 0; c < C; ++c) acc[c] = 0.f;
  for (int j0 = 0; j0 <= i; j0 += 32) {
    const int j = j0 + lane;
    const float sj = j <= i ? dot_row<T, D>(sq[warp], kg + j * kv_stride) : -INFINITY;
    const float mn = fmaxf(m, warp_max(sj));     // finite: key j0 is visible
    const float alpha = exp2f(m - mn), pj = exp2f(sj - mn);
    l = l * alpha + warp_sum(pj);
    m = mn;
#pragma unroll
    for (int c = 0; c < C; ++c) acc[c] *= alpha;
    const int n = min(32, i - j0 + 1);
    for (int t = 0; t < n; ++t) {
      const float pt = __shfl_sync(0xffffffffu, pj, t);
      const T* vr = vg + (j0 + t) * kv_stride;
#pragma unroll
      for (int c = 0; c < C; ++c) acc[c] += pt * ld1(vr + lane + 32 * c);
    }
  }
  T* og = reinterpret_cast<T*>(a.out_o) + ((int64_t)(s.lo + i) * a.Hq + h) * D;
  const float inv = 1.f / l;
#pragma unroll
  for (int c = 0; c < C; ++c) st1(og + lane + 32 * c, acc[c] * inv);
  if (lane == 0 && a.lse != nullptr) a.lse[lse_at(a, b, h, s.lo, i)] = (m + log2f(l)) * kLn2;
}

// ------------------------------------------------------------------------------------------------ backward: dQ
template <typename T, int D>
__global__ void __launch_bounds__(TW * 32) train_dq_kernel(TrainArgs a) {
  constexpr int C = D / 32;
  __shared__ float sq[TW][D], sgo[TW][D];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int b = blockIdx.z, h = blockIdx.y, kvh = h / (a.Hq / a.Hkv);
  const Seq s = seq_of(a, b);
  const int i = blockIdx.x * TW + warp;
  if (i >= s.len) return;
  const int64_t row = ((int64_t)(s.lo + i) * a.Hq + h) * D;
  const T* kg = reinterpret_cast<const T*>(a.k) + ((int64_t)s.lo * a.Hkv + kvh) * D;
  const T* vg = reinterpret_cast<const T*>(a.v) + ((int64_t)s.lo * a.Hkv + kvh) * D;
  const int64_t kv_stride = (int64_t)a.Hkv * D;
  const float sl2 = a.scale * kLog2e;
  float part = 0.f;   // delta_i = dO_i . O_i
  for (int d = lane; d < D; d += 32) {
    const float go = ld1(reinterpret_cast<const T*>(a.d_o) + row + d);
    sq[warp][d] = ld1(reinterpret_cast<const T*>(a.q) + row + d) * sl2;
    sgo[warp][d] = go;
    part += go * ld1(reinterpret_cast<const T*>(a.o) + row + d);
  }
  const float delta = warp_sum(part);
  const float lse2 = a.lse[lse_at(a, b, h, s.lo, i)] * kLog2e;
  __syncwarp();
  float acc[C];
#pragma unroll
  for (int c = 0; c < C; ++c) acc[c] = 0.f;
  for (int j0 = 0; j0 <= i; j0 += 32) {
    const int j = j0 + lane;
    float ds = 0.f;
    if (j <= i) {
      const float p = exp2f(dot_row<T, D>(sq[warp], kg + j * kv_stride) - lse2);
      ds = p * (dot_row<T, D>(sgo[warp], vg + j * kv_stride) - delta);
    }
    const int n = min(32, i - j0 + 1);
    for (int t = 0; t < n; ++t) {
      const float dt = __shfl_sync(0xffffffffu, ds, t);
      const T* kr = kg + (j0 + t) * kv_stride;
#pragma unroll
      for (int c = 0; c < C; ++c) acc[c] += dt * ld1(kr + lane + 32 * c);
    }
  }
  T* dq = reinterpret_cast<T*>(a.dq) + row;
#pragma unroll
  for (int c = 0; c < C; ++c) st1(dq + lane + 32 * c, acc[c] * a.scale);
}

// ------------------------------------------------------------------------------------------------ backward: dK, dV
template <typename T, int D>
__global__ void __launch_bounds__(TW * 32) train_dkv_kernel(TrainArgs a) {
  constexpr int C = D / 32;
  __shared__ float sk[TW][D], sv[TW][D];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int b = blockIdx.z, kvh = blockIdx.y, g = a.Hq / a.Hkv;
  const Seq s = seq_of(a, b);
  const int j = blockIdx.x * TW + warp;
  if (j >= s.len) return;
  const int64_t krow = ((int64_t)(s.lo + j) * a.Hkv + kvh) * D;
  const float sl2 = a.scale * kLog2e;
  for (int d = lane; d < D; d += 32) {
    sk[warp][d] = ld1(reinterpret_cast<const T*>(a.k) + krow + d) * sl2;
    sv[warp][d] = ld1(reinterpret_cast<const T*>(a.v) + krow + d);
  }
  __syncwarp();
  float ak[C], av[C];
#pragma unroll
  for (int c = 0; c < C; ++c) ak[c] = av[c] = 0.f;
  for (int hh = 0; hh < g; ++hh) {          // the query heads of the group add into the kv head they share, in order
    const int h = kvh * g + hh;
    for (int i0 = j; i0 < s.len; i0 += 32) {
      const int i = i0 + lane;
      float p = 0.f, ds = 0.f;
      if (i < s.len) {
        const int64_t row = ((int64_t)(s.lo + i) * a.Hq + h) * D;
        const T* qr = reinterpret_cast<const T*>(a.q) + row;
        const T* gor = reinterpret_cast<const T*>(a.d_o) + row;
        const T* orow = reinterpret_cast<const T*>(a.o) + row;
        float delta = 0.f;
#pragma unroll 8
        for (int d = 0; d < D; d += 4) {
          float x[4], y[4];
          Elem<T>::load4(gor + d, x);
          Elem<T>::load4(orow + d, y);
          delta += x[0] * y[0] + x[1] * y[1] + x[2] * y[2] + x[3] * y[3];
        }
        p = exp2f(dot_row<T, D>(sk[warp], qr) - a.lse[lse_at(a, b, h, s.lo, i)] * kLog2e);
        ds = p * (dot_row<T, D>(sv[warp], gor) - delta);
      }
      const int n = min(32, s.len - i0);
      for (int t = 0; t < n; ++t) {
        const float pt = __shfl_sync(0xffffffffu, p, t), dt = __shfl_sync(0xffffffffu, ds, t);
        const int64_t row = ((int64_t)(s.lo + i0 + t) * a.Hq + h) * D;
        const T* qr = reinterpret_cast<const T*>(a.q) + row;
        const T* gor = reinterpret_cast<const T*>(a.d_o) + row;
#pragma unroll
        for (int c = 0; c < C; ++c) {
          av[c] += pt * ld1(gor + lane + 32 * c);
          ak[c] += dt * ld1(qr + lane + 32 * c);
        }
      }
    }
  }
  T* dk = reinterpret_cast<T*>(a.dk) + krow;
  T* dv = reinterpret_cast<T*>(a.dv) + krow;
#pragma unroll
  for (int c = 0; c < C; ++c) {
    st1(dk + lane + 32 * c, ak[c] * a.scale);
    st1(dv + lane + 32 * c, av[c]);
  }
}

template <typename T, int D>
cudaError_t launch_fwd(const TrainArgs& a, cudaStream_t st) {
  dim3 grid((a.max_seqlen + TW - 1) / TW, a.Hq, a.batch);
  train_fwd_kernel<T, D><<<grid, TW * 32, 0, st>>>(a);
  note_launch();
  return cudaGetLastError();
}
template <typename T, int D>
cudaError_t launch_bwd(const TrainArgs& a, cudaStream_t st) {
  dim3 gq((a.max_seqlen + TW - 1) / TW, a.Hq, a.batch), gk((a.max_seqlen + TW - 1) / TW, a.Hkv, a.batch);
  train_dq_kernel<T, D><<<gq, TW * 32, 0, st>>>(a);
  note_launch();
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  train_dkv_kernel<T, D><<<gk, TW * 32, 0, st>>>(a);
  note_launch();
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_train_fwd_simt(const TrainArgs& a, cudaStream_t st) {
  if (a.batch == 0 || a.max_seqlen == 0) return cudaSuccess;
  if (a.dtype == EARN_F32) return a.D == 64 ? launch_fwd<float, 64>(a, st) : launch_fwd<float, 128>(a, st);
  return a.D == 64 ? launch_fwd<__nv_bfloat16, 64>(a, st) : launch_fwd<__nv_bfloat16, 128>(a, st);
}

cudaError_t launch_train_bwd_simt(const TrainArgs& a, cudaStream_t st) {
  if (a.batch == 0 || a.max_seqlen == 0) return cudaSuccess;
  if (a.dtype == EARN_F32) return a.D == 64 ? launch_bwd<float, 64>(a, st) : launch_bwd<float, 128>(a, st);
  return a.D == 64 ? launch_bwd<__nv_bfloat16, 64>(a, st) : launch_bwd<__nv_bfloat16, 128>(a, st);
}

}  // namespace earn
