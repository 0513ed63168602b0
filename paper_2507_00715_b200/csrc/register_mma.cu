// Register-only attention of a layer l >= k during prefill (Section 3.2, register-focused process):
// causal attention among the R compact register rows of each sequence, order [prefix; suffix].
//
// The work per sequence is tiny (R <= 128 keys), so the kernel is shaped for HBM traffic and latency:
// one CTA per (sequence, kv head) brings that head's compact K and V rows into shared memory once
// (through the page table) and all g query heads of the group use them.  The g*R query rows
// (row = head-in-group * R + register index) are cut into tiles of 16; each of the warps takes
// tiles round-robin, copies its 16 query rows into a private shared-memory tile with 16-byte
// asynchronous copies (in flight together with the K/V copies), reads them back as ldmatrix
// fragments, runs mma.sync m16n8k16 over 16-key tiles up to the causal limit with an online softmax
// in the log2 domain, and writes its 16 output rows through the same private tile as 16-byte stores.
#include <type_traits>

#include "earn_common.cuh"
#include "mma_sync.cuh"
#include "sm100_ptx.cuh"

namespace earn {
namespace {
using namespace mma;

// Warps per CTA (template parameter NW): four, so that several CTAs share an SM and one's loads overlap another's math,
// when the grid covers the GPU; eight on a small grid, where a CTA's chain of row tiles is what the launch waits for
// (measured on B200, compaction fused: 32 sequences x 2 kv heads 5.7 -> 3.6 us per layer with eight warps, but
// 128 sequences x 8 kv heads 29.4 -> 34.8 us).
constexpr int MAX_R = 128;

template <int D>
struct RGeo {
  static constexpr int ROWB = D * 2;
  static constexpr int PITCH = ROWB + 16;
};

// Four CTAs of four warps per SM (MINB = 4: 128 registers, 16 bytes of spills): the 512 CTAs of the 7B shapes are then
// resident at once instead of 1.15 waves of three per SM (18.4 -> 14.7 us per fused register layer; 28.8 -> 27.4
// ragged).  The eight-warp form, which runs on small grids, keeps all the registers it wants when every CTA has an SM to
// itself (capped, it lost 0.7 us at the 1.5B shapes) and is held to two CTAs per SM when there are more CTAs than SMs
// (192 CTAs: 6.1 -> 4.4 us, one wave instead of two).
template <int D, int NW, int MINB>
__global__ void __launch_bounds__(NW * 32, MINB) register_mma_kernel(RegisterArgs a, int r_pad) {
  using bf16 = __nv_bfloat16;
  using G = RGeo<D>;
  constexpr int KSTEPS = D / 16, NTILES = D / 8, CH = G::ROWB / 16;
  extern __shared__ __align__(128) uint8_t smem[];
  pdl_wait();   // everything below reads or writes global memory
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int kvh = blockIdx.x, b = blockIdx.y;
  const int R = a.R, g = a.Hq / a.Hkv, n_rows = g * R;
  const uint32_t sK = ptx::smem_u32(smem), sV = sK + r_pad * G::PITCH;
  uint8_t* gO = smem + 2 * r_pad * G::PITCH + warp * 16 * G::PITCH;   // this warp's tile: Q rows in, O rows out
  const uint32_t sQ = ptx::smem_u32(gO);
  const bool fused = a.k_full != nullptr;
  const bf16* qg = reinterpret_cast<const bf16*>(fused ? a.q_full : a.q_reg);
  // fused with the compaction: register m of the sequence is prompt row idx_b[m] (Eq. 5 layout: the first r_head rows,
  // then the last r_tail rows)
  const int seq_lo = fused ? a.cu_seqlens[b] : 0, seq_len = fused ? a.cu_seqlens[b + 1] - seq_lo : 0;
  auto src_pos = [&](int m) { return m < a.r_head ? m : seq_len - a.r_tail + (m - a.r_head); };
  // Row r of a tile is query row (head in group, register index) = (rr / R, rr % R), rr = 16 * tile + r, and sits
  // at the same element offset in q_reg and o_reg.  Lane r (and r + 16) works the offset out once per tile; the
  // copy loops fetch it by shuffle (-1: the row does not exist).
  constexpr int RPI = 32 / CH;   // rows covered by one 16-byte access of the whole warp
  auto row_offset = [&](int tile) -> int64_t {
    const int rr = tile * 16 + (lane & 15);
    if (rr >= n_rows) return -1;
    const int gi = rr / R, m = rr - gi * R;
    return (((int64_t)b * R + m) * a.Hq + kvh * g + gi) * D;
  };
  // the same row in the tensor the queries are read from: q_reg has the layout of o_reg, the packed prompt tensor not
  auto q_row_offset = [&](int tile, int64_t o_off) -> int64_t {
    if (!fused || o_off < 0) return o_off;
    const int rr = tile * 16 + (lane & 15);
    const int gi = rr / R, m = rr - gi * R;
    return (((int64_t)seq_lo + src_pos(m)) * a.Hq + kvh * g + gi) * D;
  };
  // 16 query rows of a tile -> the warp's tile (rows past g*R become zero)
  auto load_q_tile = [&](int64_t my_off) {
#pragma unroll
    for (int it = 0; it < 16 / RPI; ++it) {
      const int r = it * RPI + lane / CH, ch = lane % CH;
      const int64_t off = __shfl_sync(0xffffffffu, my_off, r);
      cp_async16(sQ + r * G::PITCH + ch * 16, qg + (off < 0 ? 0 : off) + ch * 8, off < 0 ? 0 : 16);
    }
  };
  int64_t tile_off = row_offset(warp);
  if (warp * 16 < n_rows) load_q_tile(q_row_offset(warp, tile_off));

  // ---- compact K/V rows of this (sequence, kv head) -> shared memory; rows R..r_pad-1 are zero
  {
    const bf16* kg = reinterpret_cast<const bf16*>(fused ? a.k_full : a.src.k);
    const bf16* vg = reinterpret_cast<const bf16*>(fused ? a.v_full : a.src.v);
    for (int i = threadIdx.x; i < r_pad * CH; i += NW * 32) {
      const int r = i / CH, ch = i % CH;
      const int64_t src_row = r >= R ? 0 : fused ? (int64_t)seq_lo + src_pos(r) : key_row(a.src, b, r);
      const int64_t off = r < R ? (src_row * a.Hkv + kvh) * D + ch * 8 : 0;
      const int bytes = r < R ? 16 : 0;
      cp_async16(sK + r * G::PITCH + ch * 16, kg + off, bytes);
      cp_async16(sV + r * G::PITCH + ch * 16, vg + off, bytes);
    }
    cp_async_commit();
  }

  const float scale_log2 = a.scale * kLog2e;
  const int c2 = (lane & 3) * 2;
  const int mat = lane >> 3;
  const uint32_t k_lane = (uint32_t)(((mat >> 1) << 3) + (lane & 7)) * G::PITCH + (uint32_t)(mat & 1) * 16;
  const uint32_t v_lane = (uint32_t)(((mat & 1) << 3) + (lane & 7)) * G::PITCH + (uint32_t)(mat >> 1) * 16;
  bf16* og = reinterpret_cast<bf16*>(a.o_reg);
  cp_async_wait<0>();
  __syncthreads();   // every warp's copies have landed (warps without a tile take part too)
  pdl_launch_dependents();
  if (fused) {
    // the compaction itself (Section 3.2, X -> X'): this kv head's slice of every register row goes from the tile in
    // shared memory to its cache page, bit for bit; the CTA of kv head 0 also records the source positions
    bf16* kc = reinterpret_cast<bf16*>(const_cast<void*>(a.src.k));
    bf16* vc = reinterpret_cast<bf16*>(const_cast<void*>(a.src.v));
    for (int i = threadIdx.x; i < R * CH; i += NW * 32) {
      const int r = i / CH, ch = i % CH;
      const int64_t dst = (key_row(a.src, b, r) * a.Hkv + kvh) * D + ch * 8;
      *reinterpret_cast<uint4*>(kc + dst) = *reinterpret_cast<const uint4*>(smem + r * G::PITCH + ch * 16);
      *reinterpret_cast<uint4*>(vc + dst) = *reinterpret_cast<const uint4*>(smem + (r_pad + r) * G::PITCH + ch * 16);
    }
    if (kvh == 0 && a.reg_idx != nullptr)
      for (int m = threadIdx.x; m < R; m += NW * 32) a.reg_idx[b * R + m] = src_pos(m);
  }

  for (int tile = warp; tile * 16 < n_rows; tile += NW) {
    const int rr0 = tile * 16 + (lane >> 2), rr1 = rr0 + 8;
    // row -> (head in group, register index); rows past g*R read nothing and write nothing
    const int m0r = rr0 % R, m1r = rr1 % R;
    if (tile != warp) {   // later tiles of this warp: the first one came in with the K/V rows
      tile_off = row_offset(tile);
      load_q_tile(q_row_offset(tile, tile_off));
      cp_async_commit();
      cp_async_wait<0>();
      __syncwarp();
    }
    uint32_t qf[KSTEPS][4];
#pragma unroll
    for (int kk = 0; kk < KSTEPS; ++kk)
      ldsm_x4(sQ + (lane & 15) * G::PITCH + (lane >> 4) * 16 + kk * 32, qf[kk][0], qf[kk][1], qf[kk][2], qf[kk][3]);
    // causal limit of the tile: the largest register index among its rows
    const int first = tile * 16, last = min(first + 15, n_rows - 1);
    const int m_hi = (first / R == last / R) ? last % R : R - 1;
    const int key_tiles = m_hi / 16 + 1;

    float mx0 = -INFINITY, mx1 = -INFINITY, l0 = 0.f, l1 = 0.f;
    float o[NTILES][4];
#pragma unroll
    for (int n = 0; n < NTILES; ++n) { o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f; }

    // At most 32 registers (one or two key tiles, the usual case): all scores first, one maximum, one round of
    // exponentials, then P V with nothing to rescale -- compiled for the tile count, so that the whole tile is one block
    // of straight-line code.  Longer register lists take the running-maximum loop below.
    auto short_list = [&](auto tiles_tag) {
      constexpr int KTS = decltype(tiles_tag)::value;
      float s[KTS][2][4];
#pragma unroll
      for (int kt = 0; kt < KTS; ++kt) {
#pragma unroll
        for (int n = 0; n < 2; ++n) s[kt][n][0] = s[kt][n][1] = s[kt][n][2] = s[kt][n][3] = 0.f;
        const uint32_t ks = sK + kt * 16 * G::PITCH;
#pragma unroll
        for (int kk = 0; kk < KSTEPS; ++kk) {
          uint32_t b0, b1, b2, b3;
          ldsm_x4(ks + k_lane + kk * 32, b0, b1, b2, b3);
          mma_bf16(s[kt][0], qf[kk], b0, b1);
          mma_bf16(s[kt][1], qf[kk], b2, b3);
        }
      }
      float t0 = -INFINITY, t1 = -INFINITY;
#pragma unroll
      for (int kt = 0; kt < KTS; ++kt)
#pragma unroll
        for (int n = 0; n < 2; ++n)
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int j = kt * 16 + n * 8 + c2 + (e & 1);
            s[kt][n][e] = j > ((e < 2) ? m0r : m1r) ? -INFINITY : s[kt][n][e];   // key after the row's own register (also j >= R)
            if (e < 2) t0 = fmaxf(t0, s[kt][n][e]); else t1 = fmaxf(t1, s[kt][n][e]);
          }
      t0 = fmaxf(t0, __shfl_xor_sync(0xffffffffu, t0, 1));
      t0 = fmaxf(t0, __shfl_xor_sync(0xffffffffu, t0, 2));
      t1 = fmaxf(t1, __shfl_xor_sync(0xffffffffu, t1, 1));
      t1 = fmaxf(t1, __shfl_xor_sync(0xffffffffu, t1, 2));
      const float mu0 = t0 * scale_log2, mu1 = t1 * scale_log2;   // every row sees at least key 0: finite
      uint32_t pf[KTS][4];
#pragma unroll
      for (int kt = 0; kt < KTS; ++kt) {
        const float p00 = ex2(fmaf(s[kt][0][0], scale_log2, -mu0)), p01 = ex2(fmaf(s[kt][0][1], scale_log2, -mu0));
        const float p02 = ex2(fmaf(s[kt][0][2], scale_log2, -mu1)), p03 = ex2(fmaf(s[kt][0][3], scale_log2, -mu1));
        const float p10 = ex2(fmaf(s[kt][1][0], scale_log2, -mu0)), p11 = ex2(fmaf(s[kt][1][1], scale_log2, -mu0));
        const float p12 = ex2(fmaf(s[kt][1][2], scale_log2, -mu1)), p13 = ex2(fmaf(s[kt][1][3], scale_log2, -mu1));
        l0 += p00 + p01 + p10 + p11;
        l1 += p02 + p03 + p12 + p13;
        pf[kt][0] = pack2(p00, p01); pf[kt][1] = pack2(p02, p03); pf[kt][2] = pack2(p10, p11); pf[kt][3] = pack2(p12, p13);
      }
#pragma unroll
      for (int kt = 0; kt < KTS; ++kt) {
        const uint32_t vs = sV + kt * 16 * G::PITCH;
#pragma unroll
        for (int nn = 0; nn < NTILES / 2; ++nn) {
          uint32_t b0, b1, b2, b3;
          ldsm_x4_t(vs + v_lane + nn * 32, b0, b1, b2, b3);
          mma_bf16(o[2 * nn], pf[kt], b0, b1);
          mma_bf16(o[2 * nn + 1], pf[kt], b2, b3);
        }
      }
    };
    if (key_tiles == 1) short_list(std::integral_constant<int, 1>{});
    else if (key_tiles == 2) short_list(std::integral_constant<int, 2>{});
    else
    for (int kt = 0; kt < key_tiles; ++kt) {
      const uint32_t ks = sK + kt * 16 * G::PITCH, vs = sV + kt * 16 * G::PITCH;
      float s[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
      for (int kk = 0; kk < KSTEPS; ++kk) {
        uint32_t b0, b1, b2, b3;
        ldsm_x4(ks + k_lane + kk * 32, b0, b1, b2, b3);
        mma_bf16(s[0], qf[kk], b0, b1);
        mma_bf16(s[1], qf[kk], b2, b3);
      }
#pragma unroll
      for (int n = 0; n < 2; ++n)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int j = kt * 16 + n * 8 + c2 + (e & 1);
          if (j > ((e < 2) ? m0r : m1r)) s[n][e] = -INFINITY;   // key after the row's own register (also j >= R)
        }
      float t0 = fmaxf(fmaxf(s[0][0], s[0][1]), fmaxf(s[1][0], s[1][1]));
      float t1 = fmaxf(fmaxf(s[0][2], s[0][3]), fmaxf(s[1][2], s[1][3]));
      t0 = fmaxf(t0, __shfl_xor_sync(0xffffffffu, t0, 1));
      t0 = fmaxf(t0, __shfl_xor_sync(0xffffffffu, t0, 2));
      t1 = fmaxf(t1, __shfl_xor_sync(0xffffffffu, t1, 1));
      t1 = fmaxf(t1, __shfl_xor_sync(0xffffffffu, t1, 2));
      const float mn0 = fmaxf(mx0, t0 * scale_log2), mn1 = fmaxf(mx1, t1 * scale_log2);
      const float mu0 = (mn0 == -INFINITY) ? 0.f : mn0, mu1 = (mn1 == -INFINITY) ? 0.f : mn1;
      const float al0 = ex2(mx0 - mu0), al1 = ex2(mx1 - mu1);
      mx0 = mn0; mx1 = mn1;
      uint32_t pf[4];
      {
        const float p00 = ex2(fmaf(s[0][0], scale_log2, -mu0)), p01 = ex2(fmaf(s[0][1], scale_log2, -mu0));
        const float p02 = ex2(fmaf(s[0][2], scale_log2, -mu1)), p03 = ex2(fmaf(s[0][3], scale_log2, -mu1));
        const float p10 = ex2(fmaf(s[1][0], scale_log2, -mu0)), p11 = ex2(fmaf(s[1][1], scale_log2, -mu0));
        const float p12 = ex2(fmaf(s[1][2], scale_log2, -mu1)), p13 = ex2(fmaf(s[1][3], scale_log2, -mu1));
        l0 = l0 * al0 + (p00 + p01 + p10 + p11);
        l1 = l1 * al1 + (p02 + p03 + p12 + p13);
        pf[0] = pack2(p00, p01); pf[1] = pack2(p02, p03); pf[2] = pack2(p10, p11); pf[3] = pack2(p12, p13);
      }
#pragma unroll
      for (int nn = 0; nn < NTILES / 2; ++nn) {
        uint32_t b0, b1, b2, b3;
        ldsm_x4_t(vs + v_lane + nn * 32, b0, b1, b2, b3);
        float* oa = o[2 * nn];
        float* ob = o[2 * nn + 1];
        oa[0] *= al0; oa[1] *= al0; oa[2] *= al1; oa[3] *= al1;
        ob[0] *= al0; ob[1] *= al0; ob[2] *= al1; ob[3] *= al1;
        mma_bf16(o[2 * nn], pf, b0, b1);
        mma_bf16(o[2 * nn + 1], pf, b2, b3);
      }
    }
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
    l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
    const float i0 = 1.f / l0, i1 = 1.f / l1;   // every row sees at least its own key
    // ---- stage the 16 x D bf16 tile, then 16-byte stores (a row = D*2 contiguous bytes of o_reg)
    __syncwarp();
    {
      const int r0 = lane >> 2, r1 = r0 + 8;
#pragma unroll
      for (int n = 0; n < NTILES; ++n) {
        *reinterpret_cast<uint32_t*>(gO + r0 * G::PITCH + (n * 8 + c2) * 2) = pack2(o[n][0] * i0, o[n][1] * i0);
        *reinterpret_cast<uint32_t*>(gO + r1 * G::PITCH + (n * 8 + c2) * 2) = pack2(o[n][2] * i1, o[n][3] * i1);
      }
    }
    __syncwarp();
#pragma unroll
    for (int it = 0; it < 16 / RPI; ++it) {
      const int r = it * RPI + lane / CH, ch = lane % CH;
      const int64_t off = __shfl_sync(0xffffffffu, tile_off, r);
      if (off >= 0) {
        const uint4 v = *reinterpret_cast<const uint4*>(gO + r * G::PITCH + ch * 16);
        *reinterpret_cast<uint4*>(og + off + ch * 8) = v;
      }
    }
    __syncwarp();   // the tile is free for the next Q rows
  }
}

template <int D, int NW, int MINB>
cudaError_t launch_r(const RegisterArgs& a, cudaStream_t st) {
  const int r_pad = (a.R + 15) / 16 * 16;
  const int smem = 2 * r_pad * RGeo<D>::PITCH + NW * 16 * RGeo<D>::PITCH;
  cudaError_t e = ensure_dynamic_smem<register_mma_kernel<D, NW, MINB>>(2 * MAX_R * RGeo<D>::PITCH + NW * 16 * RGeo<D>::PITCH);
  if (e != cudaSuccess) return e;
  dim3 grid(a.Hkv, a.batch);
  e = launch_pdl(register_mma_kernel<D, NW, MINB>, grid, dim3(NW * 32), smem, st, a, r_pad);
  note_launch();
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace

bool register_mma_supported(const RegisterArgs& a) { return a.dtype == EARN_BF16 && a.R <= MAX_R; }

cudaError_t launch_register_mma(const RegisterArgs& a, cudaStream_t st) {
  const long ctas = (long)a.Hkv * a.batch;
  const bool small_grid = ctas <= 2L * sm_count(), one_each = ctas <= sm_count();
  if (a.D == 64)
    return !small_grid ? launch_r<64, 4, 4>(a, st) : one_each ? launch_r<64, 8, 1>(a, st) : launch_r<64, 8, 2>(a, st);
  return !small_grid ? launch_r<128, 4, 4>(a, st) : one_each ? launch_r<128, 8, 1>(a, st) : launch_r<128, 8, 2>(a, st);
}

}  // namespace earn
