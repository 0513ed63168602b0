// Generic fp32-arithmetic tile attention on CUDA cores.
//
// One kernel template serves three uses:
//   prefill  (Eq. 3 + causal mask, layers l < k) for any dtype / head_dim the tensor-core kernel does not take,
//            and always for the fp32 debug path;
//   register (Section 3.2 register-focused process: causal attention among the R compact rows);
//   decode   (Eq. 4: W*g query rows of one (sequence, kv head) against one chunk of the shared segment,
//            written as normalised partial outputs + log2-domain LSE for the merge kernel).
//
// Tile: BM query rows x 64 keys per iteration, 256 threads as 16 x 16; thread (ty, tx) owns rows
// ty*RM.. and keys tx + 16 c of the logits and rows ty*RM.. x columns {64 c + 4 tx ..} of the output.
// Online softmax in the log2 domain (queries are pre-multiplied by scale * log2 e).
#include "earn_common.cuh"

namespace earn {
namespace {

constexpr int MODE_PREFILL = 0, MODE_REGISTER = 1, MODE_DECODE = 2;
constexpr int BN = 64;
constexpr int PS = BN + 16;   // row stride of the probability tile in shared memory

struct SimtParams {
  const void* q;
  void* o;
  float* lse;
  KeySource src;
  const int32_t* cu_seqlens;
  float* part_o;
  float* part_lse;
  int Hq, Hkv, g, R, W;
  int n_splits, chunk, rows_pad, row_tiles;
  float scale_log2;
};

template <int D, int BM>
constexpr size_t simt_smem_bytes() {
  return sizeof(float) * (size_t)(BM * D + BN * (D + 4) + BN * D + BM * PS);
}

template <typename T, int D, int BM, int MODE>
__global__ void __launch_bounds__(256) attn_simt_kernel(SimtParams p) {
  constexpr int RM = BM / 16, RN = BN / 16, KS = D + 4, NV = D / 64;
  extern __shared__ __align__(16) float smem[];
  float* sQ = smem;
  float* sK = sQ + BM * D;
  float* sV = sK + BN * KS;
  float* sP = sV + BN * D;

  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int b = blockIdx.z;
  int kvh, key_begin, key_end, row0 = 0, q_head = 0, seq_len = 0, split = 0;
  if (MODE == MODE_DECODE) {
    kvh = blockIdx.y;
    split = blockIdx.x / p.row_tiles;
    row0 = (blockIdx.x % p.row_tiles) * BM;
    seq_len = p.src.paged ? p.R : (p.cu_seqlens[b + 1] - p.cu_seqlens[b]);
    key_begin = split * p.chunk;
    key_end = min(key_begin + p.chunk, seq_len);
    if (key_begin >= key_end) return;
  } else {
    q_head = blockIdx.y;
    kvh = q_head / p.g;
    seq_len = (MODE == MODE_REGISTER) ? p.R : (p.cu_seqlens[b + 1] - p.cu_seqlens[b]);
    row0 = ((int)gridDim.x - 1 - (int)blockIdx.x) * BM;   // longest rows first
    if (row0 >= seq_len) return;
    key_begin = 0;
    key_end = min(row0 + BM, seq_len);
  }

  // pointer to the query/output row r of this tile, or null when the row does not exist
  auto row_offset = [&](int r) -> int64_t {
    int rr = row0 + r;
    if (MODE == MODE_DECODE) {
      if (rr >= p.W * p.g) return -1;
      int w = rr / p.g, gi = rr % p.g;
      return ((int64_t)(b * p.W + w) * p.Hq + kvh * p.g + gi) * D;
    }
    if (rr >= seq_len) return -1;
    int64_t tok = (MODE == MODE_REGISTER) ? (int64_t)b * p.R + rr : (int64_t)p.cu_seqlens[b] + rr;
    return (tok * p.Hq + q_head) * D;
  };

  // ---- Q tile -> shared memory, scaled into the log2 domain
  const T* qg = reinterpret_cast<const T*>(p.q);
  for (int i = tid; i < BM * (D / 4); i += 256) {
    int r = i / (D / 4), c = (i % (D / 4)) * 4;
    float x[4] = {0.f, 0.f, 0.f, 0.f};
    int64_t off = row_offset(r);
    if (off >= 0) Elem<T>::load4(qg + off + c, x);
    float* dst = sQ + r * D + c;
    dst[0] = x[0] * p.scale_log2; dst[1] = x[1] * p.scale_log2;
    dst[2] = x[2] * p.scale_log2; dst[3] = x[3] * p.scale_log2;
  }

  float m_run[RM], l_run[RM], acc[RM][NV * 4];
#pragma unroll
  for (int i = 0; i < RM; ++i) {
    m_run[i] = -INFINITY;
    l_run[i] = 0.f;
#pragma unroll
    for (int c = 0; c < NV * 4; ++c) acc[i][c] = 0.f;
  }

  const T* kg = reinterpret_cast<const T*>(p.src.k);
  const T* vg = reinterpret_cast<const T*>(p.src.v);

  for (int kb = key_begin; kb < key_end; kb += BN) {
    __syncthreads();
    for (int i = tid; i < BN * (D / 4); i += 256) {
      int r = i / (D / 4), c = (i % (D / 4)) * 4;
      float kx[4] = {0.f, 0.f, 0.f, 0.f}, vx[4] = {0.f, 0.f, 0.f, 0.f};
      if (kb + r < key_end) {
        int64_t off = (key_row(p.src, b, kb + r) * p.Hkv + kvh) * D + c;
        Elem<T>::load4(kg + off, kx);
        Elem<T>::load4(vg + off, vx);
      }
      *reinterpret_cast<float4*>(sK + r * KS + c) = make_float4(kx[0], kx[1], kx[2], kx[3]);
      *reinterpret_cast<float4*>(sV + r * D + c) = make_float4(vx[0], vx[1], vx[2], vx[3]);
    }
    __syncthreads();

    float s[RM][RN];
#pragma unroll
    for (int i = 0; i < RM; ++i)
#pragma unroll
      for (int c = 0; c < RN; ++c) s[i][c] = 0.f;
#pragma unroll 4
    for (int d = 0; d < D; d += 4) {
      float4 qv[RM], kv[RN];
#pragma unroll
      for (int i = 0; i < RM; ++i) qv[i] = *reinterpret_cast<const float4*>(sQ + (ty * RM + i) * D + d);
#pragma unroll
      for (int c = 0; c < RN; ++c) kv[c] = *reinterpret_cast<const float4*>(sK + (tx + 16 * c) * KS + d);
#pragma unroll
      for (int i = 0; i < RM; ++i)
#pragma unroll
        for (int c = 0; c < RN; ++c)
          s[i][c] += qv[i].x * kv[c].x + qv[i].y * kv[c].y + qv[i].z * kv[c].z + qv[i].w * kv[c].w;
    }

#pragma unroll
    for (int i = 0; i < RM; ++i) {
      int r = ty * RM + i;
      // keys this row may see: below key_end, and (causal modes) not after the row itself
      int limit = (MODE == MODE_DECODE) ? key_end : min(key_end, row0 + r + 1);
      float mx = -INFINITY;
#pragma unroll
      for (int c = 0; c < RN; ++c) {
        if (kb + tx + 16 * c >= limit) s[i][c] = -INFINITY;
        mx = fmaxf(mx, s[i][c]);
      }
#pragma unroll
      for (int o = 8; o >= 1; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      float m_new = fmaxf(m_run[i], mx);
      float m_use = (m_new == -INFINITY) ? 0.f : m_new;   // a row with no visible key yet keeps zeros
      float alpha = exp2f(m_run[i] - m_use);
      float sum = 0.f;
#pragma unroll
      for (int c = 0; c < RN; ++c) {
        float e = exp2f(s[i][c] - m_use);
        sum += e;
        sP[r * PS + tx + 16 * c] = e;
      }
#pragma unroll
      for (int o = 8; o >= 1; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
      l_run[i] = l_run[i] * alpha + sum;
      m_run[i] = m_new;
#pragma unroll
      for (int c = 0; c < NV * 4; ++c) acc[i][c] *= alpha;
    }
    __syncwarp();   // the 16 threads that wrote a row of sP are the ones that read it (same warp)

#pragma unroll 4
    for (int j = 0; j < BN; ++j) {
      float4 vv[NV];
#pragma unroll
      for (int c = 0; c < NV; ++c) vv[c] = *reinterpret_cast<const float4*>(sV + j * D + c * 64 + tx * 4);
#pragma unroll
      for (int i = 0; i < RM; ++i) {
        float pj = sP[(ty * RM + i) * PS + j];
#pragma unroll
        for (int c = 0; c < NV; ++c) {
          acc[i][c * 4 + 0] += pj * vv[c].x;
          acc[i][c * 4 + 1] += pj * vv[c].y;
          acc[i][c * 4 + 2] += pj * vv[c].z;
          acc[i][c * 4 + 3] += pj * vv[c].w;
        }
      }
    }
  }

  // ---- epilogue
#pragma unroll
  for (int i = 0; i < RM; ++i) {
    int r = ty * RM + i;
    int64_t off = row_offset(r);
    if (off < 0) continue;
    float inv = 1.f / l_run[i];
    if (MODE == MODE_DECODE) {
      int64_t prow = (((int64_t)(b * p.Hkv + kvh) * p.n_splits + split) * p.rows_pad + row0 + r);
#pragma unroll
      for (int c = 0; c < NV; ++c) {
        float x[4] = {acc[i][c * 4] * inv, acc[i][c * 4 + 1] * inv, acc[i][c * 4 + 2] * inv, acc[i][c * 4 + 3] * inv};
        Elem<float>::store4(p.part_o + prow * D + c * 64 + tx * 4, x);
      }
      if (tx == 0) p.part_lse[prow] = m_run[i] + log2f(l_run[i]);
    } else {
      T* og = reinterpret_cast<T*>(p.o);
#pragma unroll
      for (int c = 0; c < NV; ++c) {
        float x[4] = {acc[i][c * 4] * inv, acc[i][c * 4 + 1] * inv, acc[i][c * 4 + 2] * inv, acc[i][c * 4 + 3] * inv};
        Elem<T>::store4(og + off + c * 64 + tx * 4, x);
      }
      if (MODE == MODE_PREFILL && p.lse != nullptr && tx == 0) {
        int64_t tok = (int64_t)p.cu_seqlens[b] + row0 + r;
        int64_t total = p.cu_seqlens[gridDim.z];
        p.lse[(int64_t)q_head * total + tok] = (m_run[i] + log2f(l_run[i])) * kLn2;
      }
    }
  }
}

template <typename T, int D, int BM, int MODE>
cudaError_t launch_one(const SimtParams& p, dim3 grid, cudaStream_t st) {
  constexpr size_t smem = simt_smem_bytes<D, BM>();
  auto kern = attn_simt_kernel<T, D, BM, MODE>;
  cudaError_t e = ensure_dynamic_smem<attn_simt_kernel<T, D, BM, MODE>>((int)smem);
  if (e != cudaSuccess) return e;
  kern<<<grid, 256, smem, st>>>(p);
  note_launch();
  return cudaGetLastError();
}

template <int BM, int MODE>
cudaError_t dispatch(const SimtParams& p, dim3 grid, int dtype, int D, cudaStream_t st) {
  if (dtype == EARN_F32) {
    return D == 64 ? launch_one<float, 64, BM, MODE>(p, grid, st) : launch_one<float, 128, BM, MODE>(p, grid, st);
  }
  return D == 64 ? launch_one<__nv_bfloat16, 64, BM, MODE>(p, grid, st)
                 : launch_one<__nv_bfloat16, 128, BM, MODE>(p, grid, st);
}

// ------------------------------------------------------------------------------------------------
// Decode merge: one warp per (beam, query head).  Appends the new K/V row to the private segment,
// attends over the generated tokens of the beam's lineage, and folds in the split partials of the
// shared segment by their LSE weights.
// ------------------------------------------------------------------------------------------------
template <typename T, int D>
__global__ void __launch_bounds__(128) decode_merge_kernel(DecodeArgs a) {
  constexpr int E = D / 32;   // elements per lane
  const int lane = threadIdx.x & 31;
  const int h = blockIdx.x * 4 + (threadIdx.x >> 5);
  const int j = blockIdx.y;
  if (h >= a.Hq) return;
  const int g = a.Hq / a.Hkv, kvh = h / g, gi = h % g;
  const int b = j / a.beams, w = j % a.beams;
  const float scale_log2 = a.scale * kLog2e;

  const T* q = reinterpret_cast<const T*>(a.q) + ((int64_t)j * a.Hq + h) * D + lane * E;
  float qv[E];
#pragma unroll
  for (int e = 0; e < E; ++e) qv[e] = (float)q[e] * scale_log2;

  T* kp = reinterpret_cast<T*>(a.k_priv);
  T* vp = reinterpret_cast<T*>(a.v_priv);
  const int t_new = a.step - 1;
  {  // Eq. 4: append first.  Only this beam reads row (j, t_new) during this step.
    const T* kn = reinterpret_cast<const T*>(a.k_new) + ((int64_t)j * a.Hkv + kvh) * D + lane * E;
    const T* vn = reinterpret_cast<const T*>(a.v_new) + ((int64_t)j * a.Hkv + kvh) * D + lane * E;
    if (gi == 0) {
      int64_t dst = (priv_row(a, j, t_new) * a.Hkv + kvh) * D + lane * E;
#pragma unroll
      for (int e = 0; e < E; ++e) { kp[dst + e] = kn[e]; vp[dst + e] = vn[e]; }
    }
  }

  float m = -INFINITY, l = 0.f, acc[E];
#pragma unroll
  for (int e = 0; e < E; ++e) acc[e] = 0.f;
  for (int t = 0; t <= t_new; ++t) {
    const T *kr, *vr;
    if (t == t_new) {
      kr = reinterpret_cast<const T*>(a.k_new) + ((int64_t)j * a.Hkv + kvh) * D + lane * E;
      vr = reinterpret_cast<const T*>(a.v_new) + ((int64_t)j * a.Hkv + kvh) * D + lane * E;
    } else {
      int slab = a.lineage ? min(max(a.lineage[(int64_t)j * a.max_new + t], 0), a.batch * a.beams - 1) : j;
      int64_t off = (priv_row(a, slab, t) * a.Hkv + kvh) * D + lane * E;
      kr = kp + off;
      vr = vp + off;
    }
    float s = 0.f;
#pragma unroll
    for (int e = 0; e < E; ++e) s += qv[e] * (float)kr[e];
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    float m_new = fmaxf(m, s);
    float alpha = exp2f(m - m_new), pe = exp2f(s - m_new);
    l = l * alpha + pe;
#pragma unroll
    for (int e = 0; e < E; ++e) acc[e] = acc[e] * alpha + pe * (float)vr[e];
    m = m_new;
  }

  // fold in the shared-segment partials
  const int seq_len = a.src.paged ? a.src.n_regs : (a.cu_seqlens[b + 1] - a.cu_seqlens[b]);
  const int row = w * g + gi;
  float big = m;
  for (int s = 0; s < a.plan.n_splits && s * a.plan.chunk < seq_len; ++s) {
    int64_t prow = ((int64_t)(b * a.Hkv + kvh) * a.plan.n_splits + s) * a.plan.rows_pad + row;
    big = fmaxf(big, a.part_lse[prow]);
  }
  float wp = exp2f(m - big);
  float den = l * wp, out[E];
#pragma unroll
  for (int e = 0; e < E; ++e) out[e] = acc[e] * wp;
  for (int s = 0; s < a.plan.n_splits && s * a.plan.chunk < seq_len; ++s) {
    int64_t prow = ((int64_t)(b * a.Hkv + kvh) * a.plan.n_splits + s) * a.plan.rows_pad + row;
    float ws = exp2f(a.part_lse[prow] - big);
    den += ws;
    const float* po = a.part_o + prow * D + lane * E;
#pragma unroll
    for (int e = 0; e < E; ++e) out[e] += ws * po[e];
  }
  T* o = reinterpret_cast<T*>(a.o) + ((int64_t)j * a.Hq + h) * D + lane * E;
  float inv = 1.f / den;
#pragma unroll
  for (int e = 0; e < E; ++e) o[e] = (T)(out[e] * inv);
}

}  // namespace

cudaError_t launch_prefill_simt(const PrefillArgs& a, cudaStream_t st) {
  SimtParams p{};
  p.q = a.q; p.o = a.o; p.lse = a.lse;
  p.src.k = a.k; p.src.v = a.v; p.src.cu_seqlens = a.cu_seqlens; p.src.paged = 0;
  p.cu_seqlens = a.cu_seqlens;
  p.Hq = a.Hq; p.Hkv = a.Hkv; p.g = a.Hq / a.Hkv;
  p.scale_log2 = a.scale * kLog2e;
  dim3 grid((a.max_seqlen + 63) / 64, a.Hq, a.batch);
  return dispatch<64, MODE_PREFILL>(p, grid, a.dtype, a.D, st);
}

cudaError_t launch_register_simt(const RegisterArgs& a, cudaStream_t st) {
  SimtParams p{};
  p.q = a.q_reg; p.o = a.o_reg;
  p.src = a.src;
  p.Hq = a.Hq; p.Hkv = a.Hkv; p.g = a.Hq / a.Hkv; p.R = a.R;
  p.scale_log2 = a.scale * kLog2e;
  dim3 grid((a.R + 31) / 32, a.Hq, a.batch);
  return dispatch<32, MODE_REGISTER>(p, grid, a.dtype, a.D, st);
}

cudaError_t launch_decode_simt(const DecodeArgs& a, cudaStream_t st) {
  if (a.plan.n_splits > 0) {
    SimtParams p{};
    p.q = a.q;
    p.src = a.src;
    p.cu_seqlens = a.cu_seqlens;
    p.part_o = a.part_o; p.part_lse = a.part_lse;
    p.Hq = a.Hq; p.Hkv = a.Hkv; p.g = a.Hq / a.Hkv; p.R = a.src.n_regs; p.W = a.beams;
    p.n_splits = a.plan.n_splits; p.chunk = a.plan.chunk; p.rows_pad = a.plan.rows_pad; p.row_tiles = a.plan.row_tiles;
    p.scale_log2 = a.scale * kLog2e;
    dim3 grid(a.plan.n_splits * a.plan.row_tiles, a.Hkv, a.batch);
    cudaError_t e = dispatch<kDecodeRows, MODE_DECODE>(p, grid, a.dtype, a.D, st);
    if (e != cudaSuccess) return e;
  }
  dim3 grid((a.Hq + 3) / 4, a.batch * a.beams);
  note_launch();
  if (a.dtype == EARN_F32) {
    if (a.D == 64) decode_merge_kernel<float, 64><<<grid, 128, 0, st>>>(a);
    else decode_merge_kernel<float, 128><<<grid, 128, 0, st>>>(a);
  } else {
    if (a.D == 64) decode_merge_kernel<__nv_bfloat16, 64><<<grid, 128, 0, st>>>(a);
    else decode_merge_kernel<__nv_bfloat16, 128><<<grid, 128, 0, st>>>(a);
  }
  return cudaGetLastError();
}

}  // namespace earn
