// Decode attention (Eq. 4: append K_t, V_t, then attend over K_{1:t}) for bf16 caches.
//
// HBM-bound: every byte of the cache is read once per step, so the kernel is built around keeping
// enough loads in flight, not around the tensor cores; warp-level mma.sync (m16n8k16) only keeps the
// few query rows per key (g heads x W beams, padded to 16) off the FMA pipe.
//
// One CTA = (sequence b, kv head, split of the shared segment, tile of 16 query rows); 2 warps.  The key
// list of a CTA is its chunk of the shared segment (the prompt K/V of a layer l < k read in place, or
// the compact register pages of a layer l >= k) followed -- in split 0 only -- by the generated tokens
// of the beams its rows belong to (masked per row to the row's own beam; the newest token comes
// straight from k_new / v_new, which split 0 also appends to the private segment).  Tiles of 16 keys are
// dealt round-robin to the warps; each warp runs its own 3-stage cp.async ring (no block-wide barrier
// in the main loop) and an online softmax in the log2 domain.  The per-warp partial results are merged
// through shared memory.  With a single split the CTA writes O itself; otherwise it writes a normalised
// partial + log2-domain LSE and decode_combine_kernel folds the splits.
#include "earn_common.cuh"

namespace earn {
namespace {

constexpr int KT = 16;       // keys per tile
constexpr int STAGES = 3;    // cp.async ring depth per warp
constexpr int NWARPS = 2;    // 48 KB of rings per CTA at head_dim 128: four CTAs share an SM

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&t);
}

template <int D>
constexpr int decode_smem_bytes() {
  // the cp.async rings; reused for the cross-warp merge (NWARPS x 16 x D fp32 + statistics)
  constexpr int ring = NWARPS * STAGES * 2 * KT * D * 2;
  constexpr int merge = NWARPS * 16 * D * 4 + NWARPS * 16 * 2 * 4;
  return ring > merge ? ring : merge;
}

template <int D>
__global__ void __launch_bounds__(NWARPS * 32) decode_mma_kernel(DecodeArgs a) {
  using bf16 = __nv_bfloat16;
  constexpr int ROWB = D * 2;          // bytes per key row
  constexpr int CH = ROWB / 16;        // 16-byte chunks per row
  constexpr int TILE_B = KT * ROWB;    // bytes of one K (or V) tile
  constexpr int KSTEPS = D / 16, NTILES = D / 8;
  extern __shared__ __align__(128) uint8_t smem[];

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int b = blockIdx.z, kvh = blockIdx.y;
  const int row_tiles = a.plan.row_tiles;
  const int split = blockIdx.x / row_tiles, row0 = (blockIdx.x % row_tiles) * 16;
  const int g = a.Hq / a.Hkv, W = a.beams, n_rows = W * g, step = a.step;
  const int shared_len = a.src.paged ? a.src.n_regs : (a.cu_seqlens[b + 1] - a.cu_seqlens[b]);
  const int key_begin = split * a.plan.chunk;
  const int key_end = min(key_begin + a.plan.chunk, shared_len);
  const int n_shared = max(key_end - key_begin, 0);
  const int w_lo = row0 / g, w_hi = min((row0 + 15) / g, W - 1);
  const int n_priv = (split == 0) ? (w_hi - w_lo + 1) * step : 0;
  if (n_shared == 0 && n_priv == 0) return;
  const int tiles_sh = (n_shared + KT - 1) / KT, n_tiles = tiles_sh + (n_priv + KT - 1) / KT;
  const float scale_log2 = a.scale * kLog2e;

  const bf16* kg = reinterpret_cast<const bf16*>(a.src.k);
  const bf16* vg = reinterpret_cast<const bf16*>(a.src.v);
  bf16* kp = reinterpret_cast<bf16*>(a.k_priv);
  bf16* vp = reinterpret_cast<bf16*>(a.v_priv);
  const bf16* kn = reinterpret_cast<const bf16*>(a.k_new);
  const bf16* vn = reinterpret_cast<const bf16*>(a.v_new);

  // ---- Eq. 4: append.  Split 0 stores the new K/V row of every beam whose first query row is in this tile.
  if (split == 0) {
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

  const int c2 = (lane & 3) * 2;
  const int rr0 = row0 + (lane >> 2), rr1 = rr0 + 8;
  const int beam0 = rr0 / g, beam1 = rr1 / g;

  // ---- per-warp cp.async ring
  uint8_t* ring = smem + warp * (STAGES * 2 * TILE_B);
  const uint32_t ring_s = smem_addr(ring);

  auto issue_tile = [&](int tile, int stage) {
    const uint32_t kdst = ring_s + stage * 2 * TILE_B, vdst = kdst + TILE_B;
#pragma unroll
    for (int i = 0; i < KT * CH / 32; ++i) {
      const int idx = lane + 32 * i, r = idx / CH, ch = idx % CH;
      const bf16 *ks = kg, *vs = vg;
      int bytes = 0;
      if (tile < tiles_sh) {
        const int key = key_begin + tile * KT + r;
        if (key < key_end) {
          const int64_t off = (key_row(a.src, b, key) * a.Hkv + kvh) * D + ch * 8;
          ks = kg + off; vs = vg + off; bytes = 16;
        }
      } else {
        const int pk = (tile - tiles_sh) * KT + r;
        if (pk < n_priv) {
          const int w = w_lo + pk / step, t = pk % step;
          const int64_t j = (int64_t)b * W + w;
          if (t == step - 1) {
            const int64_t off = (j * a.Hkv + kvh) * D + ch * 8;
            ks = kn + off; vs = vn + off;
          } else {
            int64_t slab = j;
            if (a.lineage) slab = min(max(a.lineage[j * a.max_new + t], 0), a.batch * W - 1);
            const int64_t off = ((slab * a.max_new + t) * a.Hkv + kvh) * D + ch * 8;
            ks = kp + off; vs = vp + off;
          }
          bytes = 16;
        }
      }
      const uint32_t so = r * ROWB + ((ch ^ (r & 7)) << 4);
      cp_async16(kdst + so, ks, bytes);   // bytes == 0: the 16 destination bytes are zero-filled
      cp_async16(vdst + so, vs, bytes);
    }
  };

  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
  float o[NTILES][4];
#pragma unroll
  for (int n = 0; n < NTILES; ++n) { o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f; }

  const int n_my = (n_tiles - warp + NWARPS - 1) / NWARPS;   // tiles warp, warp + NWARPS, ...
#pragma unroll
  for (int s = 0; s < STAGES - 1; ++s) {
    if (s < n_my) issue_tile(warp + s * NWARPS, s);
    cp_async_commit();
  }

  // ---- Q fragments (A operand, 16 rows x D), loaded while the first tiles are in flight;
  //      rows beyond W*g are zero
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

  for (int it = 0; it < n_my; ++it) {
    const int nxt = it + STAGES - 1;
    if (nxt < n_my) issue_tile(warp + nxt * NWARPS, nxt % STAGES);
    cp_async_commit();
    cp_async_wait<STAGES - 1>();
    __syncwarp();
    const int tile = warp + it * NWARPS;
    const uint32_t ks = ring_s + (it % STAGES) * 2 * TILE_B, vs = ks + TILE_B;

    // S = Q K^T for 16 keys: two n-tiles of 8 keys
    float s[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
    {
      const int mat = lane >> 3, r = ((mat >> 1) << 3) + (lane & 7);
#pragma unroll
      for (int kk = 0; kk < KSTEPS; ++kk) {
        const int ch = kk * 2 + (mat & 1);
        uint32_t b0, b1, b2, b3;
        ldsm_x4(ks + r * ROWB + ((ch ^ (r & 7)) << 4), b0, b1, b2, b3);
        mma_bf16(s[0], qf[kk], b0, b1);
        mma_bf16(s[1], qf[kk], b2, b3);
      }
    }
    // mask + scale
    const bool priv = tile >= tiles_sh;
    const int kbase = priv ? (tile - tiles_sh) * KT : key_begin + tile * KT;
#pragma unroll
    for (int n = 0; n < 2; ++n)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int key = kbase + n * 8 + c2 + (e & 1);
        bool vis;
        if (priv) vis = key < n_priv && (w_lo + key / step) == ((e < 2) ? beam0 : beam1);
        else vis = key < key_end;
        s[n][e] = vis ? s[n][e] * scale_log2 : -INFINITY;
      }
    float mx0 = fmaxf(fmaxf(s[0][0], s[0][1]), fmaxf(s[1][0], s[1][1]));
    float mx1 = fmaxf(fmaxf(s[0][2], s[0][3]), fmaxf(s[1][2], s[1][3]));
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
    const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);
    const float mu0 = (mn0 == -INFINITY) ? 0.f : mn0, mu1 = (mn1 == -INFINITY) ? 0.f : mn1;
    const float al0 = exp2f(m0 - mu0), al1 = exp2f(m1 - mu1);
    m0 = mn0; m1 = mn1;
    uint32_t pf[4];
    {
      const float p00 = exp2f(s[0][0] - mu0), p01 = exp2f(s[0][1] - mu0), p02 = exp2f(s[0][2] - mu1), p03 = exp2f(s[0][3] - mu1);
      const float p10 = exp2f(s[1][0] - mu0), p11 = exp2f(s[1][1] - mu0), p12 = exp2f(s[1][2] - mu1), p13 = exp2f(s[1][3] - mu1);
      l0 = l0 * al0 + (p00 + p01 + p10 + p11);   // per-lane partial sums; reduced over the quad at the end
      l1 = l1 * al1 + (p02 + p03 + p12 + p13);
      pf[0] = pack2(p00, p01); pf[1] = pack2(p02, p03); pf[2] = pack2(p10, p11); pf[3] = pack2(p12, p13);
    }
    // O = O * alpha + P V
    {
      const int mat = lane >> 3, r = ((mat & 1) << 3) + (lane & 7);
#pragma unroll
      for (int nn = 0; nn < NTILES / 2; ++nn) {
        const int ch = nn * 2 + (mat >> 1);
        uint32_t b0, b1, b2, b3;
        ldsm_x4_t(vs + r * ROWB + ((ch ^ (r & 7)) << 4), b0, b1, b2, b3);
        float* oa = o[2 * nn];
        float* ob = o[2 * nn + 1];
        oa[0] *= al0; oa[1] *= al0; oa[2] *= al1; oa[3] *= al1;
        ob[0] *= al0; ob[1] *= al0; ob[2] *= al1; ob[3] *= al1;
        mma_bf16(o[2 * nn], pf, b0, b1);
        mma_bf16(o[2 * nn + 1], pf, b2, b3);
      }
    }
    __syncwarp();   // every lane is done with this stage before a later iteration refills it
  }
  cp_async_wait<0>();
  l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
  l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
  __syncthreads();   // all rings are idle: reuse the shared memory for the merge

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
  }
}

// Folds the split partials: one warp per (query row, kv head, sequence).
template <int D>
__global__ void __launch_bounds__(128) decode_combine_kernel(DecodeArgs a) {
  constexpr int E = D / 32;
  const int lane = threadIdx.x & 31;
  const int rr = blockIdx.x * 4 + (threadIdx.x >> 5), kvh = blockIdx.y, b = blockIdx.z;
  const int g = a.Hq / a.Hkv, W = a.beams;
  if (rr >= W * g) return;
  const int shared_len = a.src.paged ? a.src.n_regs : (a.cu_seqlens[b + 1] - a.cu_seqlens[b]);
  const int64_t prow0 = (int64_t)(b * a.Hkv + kvh) * a.plan.n_splits * a.plan.rows_pad + rr;
  float big = -INFINITY;
  for (int s = 0; s < a.plan.n_splits; ++s)
    if (s == 0 || s * a.plan.chunk < shared_len) big = fmaxf(big, a.part_lse[prow0 + (int64_t)s * a.plan.rows_pad]);
  float den = 0.f, out[E];
#pragma unroll
  for (int e = 0; e < E; ++e) out[e] = 0.f;
  for (int s = 0; s < a.plan.n_splits; ++s) {
    if (!(s == 0 || s * a.plan.chunk < shared_len)) continue;
    const int64_t prow = prow0 + (int64_t)s * a.plan.rows_pad;
    const float wt = exp2f(a.part_lse[prow] - big);
    den += wt;
    const float* po = a.part_o + prow * D + lane * E;
#pragma unroll
    for (int e = 0; e < E; ++e) out[e] += wt * po[e];
  }
  __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(a.o) + (((int64_t)b * W + rr / g) * a.Hq + kvh * g + rr % g) * D + lane * E;
  const float inv = 1.f / den;
#pragma unroll
  for (int e = 0; e < E; e += 2) *reinterpret_cast<uint32_t*>(dst + e) = pack2(out[e] * inv, out[e + 1] * inv);
}

template <int D>
cudaError_t launch_d(const DecodeArgs& a, cudaStream_t st) {
  constexpr int smem = decode_smem_bytes<D>();
  cudaError_t e = ensure_dynamic_smem<decode_mma_kernel<D>>(smem);
  if (e != cudaSuccess) return e;
  const int splits = a.plan.n_splits > 0 ? a.plan.n_splits : 1;
  dim3 grid(splits * a.plan.row_tiles, a.Hkv, a.batch);
  decode_mma_kernel<D><<<grid, NWARPS * 32, smem, st>>>(a);
  note_launch();
  e = cudaGetLastError();
  if (e != cudaSuccess || a.plan.n_splits <= 1) return e;
  dim3 cgrid((a.plan.rows + 3) / 4, a.Hkv, a.batch);
  decode_combine_kernel<D><<<cgrid, 128, 0, st>>>(a);
  note_launch();
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_decode_mma(const DecodeArgs& a, cudaStream_t st) {
  return a.D == 64 ? launch_d<64>(a, st) : launch_d<128>(a, st);
}

}  // namespace earn
