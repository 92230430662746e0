// bf16 GEMM for sm_100a: C = epilogue(A W^T), A [M, K] and W [N, K] both K-major.
//
// Persistent, warp-specialised CTAs of 192 threads:
//   warp 0      one lane issues TMA loads (A 128 x 64 and W BN x 64 boxes, 128-byte swizzle)
//               into a ring of shared-memory stages guarded by full/empty mbarriers;
//   warp 1      allocates tensor memory, one lane issues tcgen05.mma (128 x BN x 16, f32
//               accumulation in TMEM) and commits stage releases / accumulator readiness;
//   warps 2..5  read the accumulator with tcgen05.ld (one row per thread), apply the fused
//               epilogue, stage 32-row x 128-byte pieces in swizzled shared memory and hand them
//               to TMA for the store.  The residual update fetches the old values of the residual
//               stream by TMA one piece ahead, adds in place in shared memory and stores from
//               there, leaving per-row partial sums for the LayerNorm that the next GEMM folds
//               into its own epilogue.  All this runs while the MMA warp already fills the other
//               accumulator buffer.
// Every mbarrier wait is bounded; on a timeout the CTA sets an error word, drains its own
// TMA copies, frees its tensor memory and returns.
#include <algorithm>

#include "wf_internal.h"
#include "wf_epilogue.cuh"
#include "wf_ptx.cuh"

namespace wf {

using namespace ptx;

constexpr int kBM = 128;
constexpr int kBK = 64;
constexpr int kGemmThreads = 192;
// Residual epilogue (kEpiResidSplit): every epilogue warp owns kXSets staging sets of 8 KB (a
// 32-row x 64-column piece of x_hi and of x_lo); the old values of piece p + kXLook are fetched
// by TMA while piece p is processed, and a set is stored from in place.
constexpr int kXSets = 2;
constexpr int kXLook = 1;
constexpr int kSmemBudget = 224 * 1024;  // operand stages + epilogue staging

// Shared-memory plan of a CTA that stages 128 x 64 of A and BROWS x 64 of W per stage.
template <int BROWS, int EPI, int XS = kXSets>
struct SmemPlan {
  static constexpr int kABytes = kBM * kBK * 2;
  static constexpr int kBBytes = BROWS * kBK * 2;
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kStagingPerWarp = EPI == kEpiResidSplit ? XS * 8192 : 2 * 4096;
  static constexpr int kStages = (kSmemBudget - 4 * kStagingPerWarp) / kStageBytes;
  static constexpr int kStagingOffset = kStages * kStageBytes;
  static constexpr int kBarOffset = kStagingOffset + 4 * kStagingPerWarp;
  // barriers: full[kStages], empty[kStages], tfull[2], tempty[2], xld[4][kXSets] (XS <= kXSets of them
  // used per warp); then the tensor memory slot and the abort flag
  static constexpr int kNumBars = 2 * kStages + 4 + 4 * kXSets;
  static constexpr int kSmemBytes = kBarOffset + 8 * kNumBars + 16 + 1024;  // + alignment slack
  static_assert(kStages >= 3 && 8 * kNumBars + 16 <= 256, "shared-memory plan");
};

__host__ __device__ constexpr bool epi_is_ln(int epi) { return epi == kEpiLnBias || epi == kEpiLnBiasGelu; }

// Mean and reciprocal standard deviation of one row of x (K columns) from the partial sums its
// producer left: returns (rstd, -rstd * mean).
__device__ __forceinline__ float2 row_norm(const EpiParams& ep, long row, long M, int K) {
  float s1 = 0.f, s2 = 0.f;
  if (row < M) {
    for (int p = 0; p < K / 128; ++p) {
      const float2 t = __ldg(ep.stats_in + (long)p * ep.stats_pitch + row);
      s1 += t.x;
      s2 += t.y;
    }
  }
  const float inv = 1.0f / (float)K;
  const float mean = s1 * inv;
  const float var = fmaxf(fmaf(s2, inv, -mean * mean), 0.f);
  const float rstd = rsqrtf(var + 1e-5f);
  return make_float2(rstd, -rstd * mean);
}

// Partial accumulators of a tile whose K range was split over the CTAs of a cluster (the single-CTA
// kernel's small-M variant): CTAs 1 .. n of the cluster leave their 128 x 128 float32 accumulators
// in the shared memory of CTA 0 (its operand stages, idle by then), which adds them to its own in
// rank order before the epilogue arithmetic.  Layout of one partial (64 KB): row r at r * 512
// bytes, its 16-byte chunk c at position (c & ~7) | ((c & 7) ^ (r & 7)).
struct Partials {
  uint32_t base;  // shared-memory address of the first partial (in the CTA that reads them)
  int n;          // how many (0: none)
};
__device__ __forceinline__ uint32_t partial_addr(uint32_t base, int p, int row, int chunk) {
  return base + (uint32_t)p * 65536u + (uint32_t)row * 512u + (uint32_t)(((chunk & ~7) | ((chunk & 7) ^ (row & 7))) << 4);
}
// acc (32 columns starting at tile column c0, accumulator row `row`) += the partials, in rank order
__device__ __forceinline__ void add_partials(const Partials& ps, int row, int c0, uint32_t (&acc)[32]) {
  for (int p = 0; p < ps.n; ++p) {
#pragma unroll
    for (int g = 0; g < 8; ++g) {
      uint32_t q[4];
      ld_shared_v4(partial_addr(ps.base, p, row, (c0 >> 2) + g), q[0], q[1], q[2], q[3]);
#pragma unroll
      for (int i = 0; i < 4; ++i) acc[4 * g + i] = __float_as_uint(__uint_as_float(acc[4 * g + i]) + __uint_as_float(q[i]));
    }
  }
}

// Epilogue arithmetic of 32 accumulator columns starting at col0 (col0 + 32 <= padded N is not
// required: columns at or beyond N are computed from zeros and never stored).  nrm = row_norm()
// for the LayerNorm-folded epilogues.
template <int EPI>
__device__ __forceinline__ void bias_act32(const EpiParams& ep, int col0, int N, const uint32_t (&acc)[32],
                                           float (&v)[32], float2 nrm) {
  const uint64_t rs = pack_f32x2(nrm.x, nrm.x), nm = pack_f32x2(nrm.y, nrm.y);
#pragma unroll
  for (int g = 0; g < 8; ++g) {
    const int col = col0 + 4 * g;
    const float4 b = col < N ? __ldg(reinterpret_cast<const float4*>(ep.bias + col)) : make_float4(0.f, 0.f, 0.f, 0.f);
    const uint64_t a01 = pack_f32x2(__uint_as_float(acc[4 * g + 0]), __uint_as_float(acc[4 * g + 1]));
    const uint64_t a23 = pack_f32x2(__uint_as_float(acc[4 * g + 2]), __uint_as_float(acc[4 * g + 3]));
    if (epi_is_ln(EPI)) {
      const float4 cs = col < N ? __ldg(reinterpret_cast<const float4*>(ep.colsum + col)) : make_float4(0.f, 0.f, 0.f, 0.f);
      unpack_f32x2(fma_f32x2(rs, a01, fma_f32x2(nm, pack_f32x2(cs.x, cs.y), pack_f32x2(b.x, b.y))), v[4 * g + 0], v[4 * g + 1]);
      unpack_f32x2(fma_f32x2(rs, a23, fma_f32x2(nm, pack_f32x2(cs.z, cs.w), pack_f32x2(b.z, b.w))), v[4 * g + 2], v[4 * g + 3]);
    } else {
      unpack_f32x2(add_f32x2(a01, pack_f32x2(b.x, b.y)), v[4 * g + 0], v[4 * g + 1]);
      unpack_f32x2(add_f32x2(a23, pack_f32x2(b.z, b.w)), v[4 * g + 2], v[4 * g + 3]);
    }
  }
  if (EPI == kEpiBiasGelu || EPI == kEpiLnBiasGelu || EPI == kEpiConv1 || EPI == kEpiConv2) {
#pragma unroll
    for (int i = 0; i < 32; i += 2) gelu_sigmoid_poly2(v[i], v[i + 1]);
  }
}

// x = hi + lo with hi = bf16(x), lo = bf16(x - hi): two values per call, packed as bf16 pairs
// (first value in the low half).
__device__ __forceinline__ void split_bf16x2(float x0, float x1, uint32_t& hi, uint32_t& lo) {
  __nv_bfloat162 h = __floats2bfloat162_rn(x0, x1);
  hi = *reinterpret_cast<uint32_t*>(&h);
  __nv_bfloat162 l = __floats2bfloat162_rn(x0 - __uint_as_float(hi << 16), x1 - __uint_as_float(hi & 0xffff0000u));
  lo = *reinterpret_cast<uint32_t*>(&l);
}

// Stride-2 conv epilogue, whose output rows are remapped per sequence (plain stores, no TMA):
// x[dst] = gelu(acc + bias) + pe[pos], written as the two planes of the residual stream; s1 / s2
// gather the row's sum and sum of squares.
__device__ __forceinline__ void conv2_store32(const EpiParams& ep, int2 d, int col0, int N, const float (&v)[32],
                                              float& s1, float& s2) {
  if (d.x < 0 || col0 >= N) return;
#pragma unroll
  for (int g = 0; g < 4; ++g) {
    const int col = col0 + 8 * g;
    if (col >= N) break;
    const float4 e0 = __ldg(reinterpret_cast<const float4*>(ep.pe + (long)d.y * ep.ldc + col));
    const float4 e1 = __ldg(reinterpret_cast<const float4*>(ep.pe + (long)d.y * ep.ldc + col + 4));
    const float x[8] = {v[8 * g] + e0.x,     v[8 * g + 1] + e0.y, v[8 * g + 2] + e0.z, v[8 * g + 3] + e0.w,
                        v[8 * g + 4] + e1.x, v[8 * g + 5] + e1.y, v[8 * g + 6] + e1.z, v[8 * g + 7] + e1.w};
    uint4 h, l;
    split_bf16x2(x[0], x[1], h.x, l.x);
    split_bf16x2(x[2], x[3], h.y, l.y);
    split_bf16x2(x[4], x[5], h.z, l.z);
    split_bf16x2(x[6], x[7], h.w, l.w);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      s1 += x[i];
      s2 = fmaf(x[i], x[i], s2);
    }
    *reinterpret_cast<uint4*>(ep.x_hi + (long)d.x * ep.ldc + col) = h;
    *reinterpret_cast<uint4*>(ep.x_lo + (long)d.x * ep.ldc + col) = l;
  }
}

// Epilogue of one 128 x BN accumulator tile for the warp that owns TMEM lanes 32 * quarter ..:
// t_row is the tensor-memory address of that lane group's first column of the tile, m0 / n0 the
// tile origin in the output, stage_base this warp's staging buffers (bf16 outputs: two of 4 KB).
template <int BN, int EPI>
__device__ __forceinline__ void epilogue_tile(const EpiParams& ep, const CUtensorMap* tmap_c, uint32_t t_row, int m0,
                                              int n0, long M, int N, int K, int quarter, int lane, uint32_t stage_base,
                                              uint32_t& piece, const Partials ps = Partials{0u, 0}) {
  const long row = (long)m0 + quarter * 32 + lane;
  if (EPI == kEpiConv2) {
    const int2 d = row < M ? ep.row_dst[row] : make_int2(-1, 0);
    float s1 = 0.f, s2 = 0.f;
#pragma unroll 1
    for (int c = 0; c < BN / 32; ++c) {
      uint32_t a32[32];
      float v[32];
      tmem_ld_32x32(t_row + c * 32, a32);
      tmem_ld_wait();
      bias_act32<EPI>(ep, n0 + c * 32, N, a32, v, make_float2(0.f, 0.f));
      conv2_store32(ep, d, n0 + c * 32, N, v, s1, s2);
      if ((c & 3) == 3) {  // 128 columns done: one partial of the row statistics
        if (d.x >= 0 && n0 + c * 32 < N) ep.stats_out[(long)((n0 + c * 32) >> 7) * ep.stats_pitch + d.x] = make_float2(s1, s2);
        s1 = s2 = 0.f;
      }
    }
  } else {
    // bf16: 64 columns = 128 bytes per row and piece
    // Rows at or beyond M that the last tile still stores (outputs are capacity-sized) are written as
    // zeros, never as whatever the accumulator holds for them: the attention kernel multiplies the
    // value rows behind a sequence's end by probabilities that are exactly zero, which only gives
    // zero if those rows are finite.
    bool valid = row < M;
    if (EPI == kEpiConv1) valid = valid && ep.row_valid[row] != 0;
    float2 nrm = make_float2(0.f, 0.f);
    if (epi_is_ln(EPI)) nrm = row_norm(ep, row, M, K);
#pragma unroll 1
    for (int c = 0; c < BN / 64; ++c) {
      const uint32_t buf = stage_base + (uint32_t)((piece & 1u) * 4096);
      if (lane == 0) bulk_wait_read<1>();   // the copy that last read this buffer is done with it
      __syncwarp();
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
        uint32_t a32[32];
        float v[32];
        tmem_ld_32x32(t_row + c * 64 + hf * 32, a32);
        tmem_ld_wait();
        if (ps.n > 0) add_partials(ps, quarter * 32 + lane, c * 64 + hf * 32, a32);
        bias_act32<EPI>(ep, n0 + c * 64 + hf * 32, N, a32, v, nrm);
        if (!valid) {
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] = 0.f;
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          __nv_bfloat162 p0 = __floats2bfloat162_rn(v[8 * j + 0], v[8 * j + 1]);
          __nv_bfloat162 p1 = __floats2bfloat162_rn(v[8 * j + 2], v[8 * j + 3]);
          __nv_bfloat162 p2 = __floats2bfloat162_rn(v[8 * j + 4], v[8 * j + 5]);
          __nv_bfloat162 p3 = __floats2bfloat162_rn(v[8 * j + 6], v[8 * j + 7]);
          st_shared_v4(buf + lane * 128 + (((hf * 4 + j) ^ (lane & 7)) << 4), *reinterpret_cast<uint32_t*>(&p0),
                       *reinterpret_cast<uint32_t*>(&p1), *reinterpret_cast<uint32_t*>(&p2),
                       *reinterpret_cast<uint32_t*>(&p3));
        }
      }
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) {
        if (n0 + c * 64 < N && (long)m0 + quarter * 32 < M) tma_store_2d(tmap_c, buf, n0 + c * 64, m0 + quarter * 32);
        // One bulk group per piece, empty when the piece lies outside the matrix: wait_read<1> above
        // counts groups to know that the copy two pieces back has let go of its buffer.
        bulk_commit();
      }
      ++piece;
    }
  }
}

// ---- residual epilogue on the split residual stream --------------------------------------------
// The pieces (32 rows x 64 columns) an epilogue warp handles, in order: tile `first + i * stride`
// (while below `count`), columns 64 c .. of it, c = 0 .. ppt - 1.
struct XWalk {
  int first, stride, count, num_n;
  int tile_rows, row_off;  // rows per tile step; this warp's row offset inside the tile
  int bn, ppt;             // tile width; pieces per tile = bn / 64
};
// Coordinates of piece p; false if there is no such piece or it lies outside the M x N matrix.
__device__ __forceinline__ bool piece_xy(const XWalk& w, uint32_t p, long M, int N, int& x, int& y) {
  const long t = (long)w.first + (long)(p / (uint32_t)w.ppt) * w.stride;
  if (t >= w.count) return false;
  x = (int)(t % w.num_n) * w.bn + (int)(p % (uint32_t)w.ppt) * 64;
  y = (int)(t / w.num_n) * w.tile_rows + w.row_off;
  return x < N && y < M;
}
// One lane: fetch the old x_hi / x_lo values of piece p into its staging set (XS sets per warp, the
// fetch running XL pieces ahead of the piece being processed).
template <int XS = kXSets, int XL = kXLook>
__device__ __forceinline__ void x_fetch(const XWalk& w, uint32_t p, long M, int N, const CUtensorMap* t_hi,
                                        const CUtensorMap* t_lo, uint32_t stage_base, uint32_t xbar0, uint32_t& armed) {
  int x, y;
  if (!piece_xy(w, p, M, N, x, y)) return;
  const uint32_t set = p % XS;
  // The set was last used by piece p - XS.  This runs while piece p - XL is current, after the
  // groups of all earlier pieces were committed: at most XS - XL - 1 of them may still be reading
  // shared memory.
  static_assert(XS - XL - 1 >= 0, "the fetch may not run further ahead than there are sets");
  bulk_wait_read<XS - XL - 1>();
  mbar_arrive_expect_tx(xbar0 + 8u * set, 8192);
  tma_load_2d(stage_base + set * 8192u, t_hi, x, y, xbar0 + 8u * set);
  tma_load_2d(stage_base + set * 8192u + 4096u, t_lo, x, y, xbar0 + 8u * set);
  armed |= 1u << set;
}
struct XState {
  uint32_t piece;   // pieces handled so far
  uint32_t phase;   // bit s: parity of staging set s's barrier to wait for next
  uint32_t armed;   // lane 0: sets with a fetch in flight
};
// One tile: x <- x + acc + bias in place in shared memory, pieces stored back by TMA, the row's
// (sum, sum of squares) over each 128 columns written to stats_out.  False after a timed-out wait.
template <int BN, int XS = kXSets, int XL = kXLook>
__device__ __forceinline__ bool epilogue_tile_split(const EpiParams& ep, const CUtensorMap* t_hi, const CUtensorMap* t_lo,
                                                    uint32_t t_row, int m0, int n0, long M, int N, int quarter, int lane,
                                                    uint32_t stage_base, uint32_t xbar0, const XWalk& w, XState& st,
                                                    volatile int* abort_flag, const Partials ps = Partials{0u, 0}) {
  const long row = (long)m0 + quarter * 32 + lane;
  float s1 = 0.f, s2 = 0.f;
#pragma unroll 1
  for (int c = 0; c < BN / 64; ++c) {
    const uint32_t p = st.piece;
    if (lane == 0) x_fetch<XS, XL>(w, p + XL, M, N, t_hi, t_lo, stage_base, xbar0, st.armed);
    const bool valid = n0 + c * 64 < N && (long)m0 + quarter * 32 < M;
    if (valid) {
      const uint32_t set = p % XS;
      const uint32_t buf = stage_base + set * 8192u;
      bool ok = mbar_wait(xbar0 + 8u * set, (st.phase >> set) & 1u, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) return false;
      st.phase ^= 1u << set;
      st.armed &= ~(1u << set);
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
        uint32_t a32[32];
        float v[32];
        tmem_ld_32x32(t_row + c * 64 + hf * 32, a32);
        tmem_ld_wait();
        if (ps.n > 0) add_partials(ps, quarter * 32 + lane, c * 64 + hf * 32, a32);
        bias_act32<kEpiResidSplit>(ep, n0 + c * 64 + hf * 32, N, a32, v, make_float2(0.f, 0.f));
        if (row >= M) {  // a row beyond the matrix inside a stored piece keeps its old value
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] = 0.f;
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const uint32_t a = buf + lane * 128 + (((hf * 4 + j) ^ (lane & 7)) << 4);
          uint32_t h[4], l[4];
          ld_shared_v4(a, h[0], h[1], h[2], h[3]);
          ld_shared_v4(a + 4096u, l[0], l[1], l[2], l[3]);
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            // hi + lo is exact in float32 (16 significant bits)
            const float x0 = (__uint_as_float(h[q] << 16) + __uint_as_float(l[q] << 16)) + v[8 * j + 2 * q];
            const float x1 = (__uint_as_float(h[q] & 0xffff0000u) + __uint_as_float(l[q] & 0xffff0000u)) + v[8 * j + 2 * q + 1];
            s1 += x0 + x1;
            s2 = fmaf(x0, x0, fmaf(x1, x1, s2));
            split_bf16x2(x0, x1, h[q], l[q]);
          }
          st_shared_v4(a, h[0], h[1], h[2], h[3]);
          st_shared_v4(a + 4096u, l[0], l[1], l[2], l[3]);
        }
      }
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) {
        tma_store_2d(t_hi, buf, n0 + c * 64, m0 + quarter * 32);
        tma_store_2d(t_lo, buf + 4096u, n0 + c * 64, m0 + quarter * 32);
      }
    }
    if (lane == 0) bulk_commit();  // one group per piece, empty for a piece outside the matrix (x_fetch counts groups)
    ++st.piece;
    if (c & 1) {  // 128 columns done
      if (valid && row < M) ep.stats_out[(long)((n0 + c * 64) >> 7) * ep.stats_pitch + row] = make_float2(s1, s2);
      s1 = s2 = 0.f;
    }
  }
  return true;
}
// After a timed-out wait: let the fetches this lane issued land before the CTA's shared memory is released.
__device__ __forceinline__ void x_drain(uint32_t xbar0, const XState& st) {
  for (uint32_t s = 0; s < (uint32_t)kXSets; ++s) {
    if (!(st.armed & (1u << s))) continue;
    for (uint32_t it = 0; it < (1u << 20); ++it)
      if (mbar_try_wait(xbar0 + 8u * s, (st.phase >> s) & 1u)) break;
  }
}

// Bounded wait (after a timed-out wait elsewhere in the CTA) for the operand copies a producer
// thread has in flight: bit s of `armed` = stage s has a copy whose barrier phase has parity bit s
// of `parity`.
__device__ __forceinline__ void drain_stages(uint32_t full_bar0, int stages, uint32_t armed, uint32_t parity) {
  for (int s = 0; s < stages; ++s) {
    if (!(armed & (1u << s))) continue;
    for (uint32_t it = 0; it < (1u << 20); ++it)
      if (mbar_try_wait(full_bar0 + 8u * s, (parity >> s) & 1u)) break;
  }
}

// Single-CTA kernel, 128 x 128 or 128 x 256 tiles: the small-M regime, where 256 x 256 tiles would
// leave most CTA pairs idle.  tmap_c is the bf16 output map, or x_hi's (with tmap_c2 = x_lo's) for kEpiResidSplit.
template <int BN, int EPI>
__global__ void __launch_bounds__(kGemmThreads, 1) gemm_bf16_kernel(
    const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
    const __grid_constant__ CUtensorMap tmap_c, const __grid_constant__ CUtensorMap tmap_c2, long M, int N, int K,
    int a_cols, EpiParams ep, int* err_flag) {
  using Cfg = SmemPlan<BN, EPI>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t bar_base = smem_base + Cfg::kBarOffset;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (Cfg::kStages + s); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * Cfg::kStages + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * Cfg::kStages + 2 + a); };
  const uint32_t xbar_base = bar_base + 8u * (2 * Cfg::kStages + 4);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_gen + Cfg::kBarOffset + 8 * Cfg::kNumBars);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_gen + Cfg::kBarOffset + 8 * Cfg::kNumBars + 8);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < Cfg::kStages; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(tfull_bar(a), 1);
      mbar_init(tempty_bar(a), 4);
    }
    for (int i = 0; i < 4 * kXSets; ++i) mbar_init(xbar_base + 8u * i, 1);
    *abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), 2 * BN);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  griddep_wait();  // everything above overlapped the previous kernel's tail; its output is needed from here on
  griddep_launch_dependents();

  const int num_m = (int)((M + kBM - 1) / kBM);
  const int num_n = (N + BN - 1) / BN;
  const int num_k = (K + kBK - 1) / kBK;
  const int num_tiles = num_m * num_n;

  if (warp == 0) {
    if (lane == 0) {
      prefetch_tmap(&tmap_a);
      prefetch_tmap(&tmap_b);
      int stage = 0;
      uint32_t phase = 0;
      uint32_t armed = 0, armed_parity = 0;  // bit s: stage s has had a load issued / its parity
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
        const int m0 = (tile / num_n) * kBM, n0 = (tile % num_n) * BN;
        for (int kb = 0; kb < num_k; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) { ok = false; break; }
          mbar_arrive_expect_tx(full_bar(stage), Cfg::kStageBytes);
          const uint32_t sa = smem_base + stage * Cfg::kStageBytes;
          // A row of the GEMM may wrap over consecutive rows of the stored matrix (conv stem:
          // three time rows laid end to end); a_cols is the stored row length, K for a plain GEMM.
          const int e = kb * kBK;
          tma_load_2d(sa, &tmap_a, e % a_cols, m0 + e / a_cols, full_bar(stage));
          tma_load_2d(sa + Cfg::kABytes, &tmap_b, kb * kBK, n0, full_bar(stage));
          if (BN == 256)  // the W map's box has 128 rows: the second half of a 256-wide tile
            tma_load_2d(sa + Cfg::kABytes + 128 * kBK * 2, &tmap_b, kb * kBK, n0 + 128, full_bar(stage));
          armed |= 1u << stage;
          armed_parity = (armed_parity & ~(1u << stage)) | (phase << stage);
          if (++stage == Cfg::kStages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        atomicExch(err_flag, 1);
        drain_stages(full_bar(0), Cfg::kStages, armed, armed_parity);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(kBM, BN, 0, 0);
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; ok && tile < num_tiles; tile += gridDim.x) {
        if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
        for (int kb = 0; kb < num_k; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = smem_base + stage * Cfg::kStageBytes;
          const uint64_t adesc = umma_desc_k_sw128(sa);
          const uint64_t bdesc = umma_desc_k_sw128(sa + Cfg::kABytes);
#pragma unroll
          for (int k = 0; k < kBK / 16; ++k) {
            // 16 bf16 = 32 bytes further along K inside the swizzled row: +2 in 16-byte units
            umma_bf16(d_tmem, adesc + 2 * k, bdesc + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
          }
          umma_commit(empty_bar(stage));
          if (++stage == Cfg::kStages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        umma_commit(tfull_bar(acc));
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
      if (!ok) atomicExch(err_flag, 2);
    }
  } else {
    const int quarter = warp & 3;  // TMEM lanes this warp may read: 32 * quarter .. + 31
    const uint32_t stage_base = smem_base + Cfg::kStagingOffset + (uint32_t)((warp - 2) * Cfg::kStagingPerWarp);
    const uint32_t xbar0 = xbar_base + 8u * (uint32_t)((warp - 2) * kXSets);
    const XWalk walk{(int)blockIdx.x, (int)gridDim.x, num_tiles, num_n, kBM, quarter * 32, BN, BN / 64};
    XState xs{0u, 0u, 0u};
    if (EPI == kEpiResidSplit && lane == 0) {
      prefetch_tmap(&tmap_c);
      prefetch_tmap(&tmap_c2);
      for (uint32_t p = 0; p < (uint32_t)kXLook; ++p) x_fetch(walk, p, M, N, &tmap_c, &tmap_c2, stage_base, xbar0, xs.armed);
    }
    uint32_t piece = 0;
    int acc = 0;
    uint32_t acc_phase = 0;
    for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x) {
      const int m0 = (tile / num_n) * kBM, n0 = (tile % num_n) * BN;
      bool ok = mbar_wait(tfull_bar(acc), acc_phase, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (ok) {
        tc_fence_after();
        const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BN);
        if constexpr (EPI == kEpiResidSplit)
          ok = epilogue_tile_split<BN>(ep, &tmap_c, &tmap_c2, t_row, m0, n0, M, N, quarter, lane, stage_base, xbar0, walk, xs,
                                       abort_flag);
        else
          epilogue_tile<BN, EPI>(ep, &tmap_c, t_row, m0, n0, M, N, K, quarter, lane, stage_base, piece);
      }
      if (!ok) {
        if (lane == 0) {
          atomicExch(err_flag, 3);
          x_drain(xbar0, xs);
        }
        break;
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty_bar(acc));
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
    if (lane == 0) bulk_wait_all();  // every store this lane issued has completed
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 2 * BN);
  }
}

// ---------------------------------------------------------------------------------------------
// Small-M variant of the single-CTA kernel: one 128 x 128 tile per CLUSTER of `split` CTAs, each
// CTA accumulating its share of the K range (so that a few tiles still draw their weights through
// many SMs: one SM takes in about 100 GB/s, and ten tiles of K = 5120 would otherwise stream a
// 13 MB weight matrix through ten SMs).  The partial accumulators meet in CTA 0's shared memory
// through distributed shared memory (see Partials) and are added in rank order: the result does
// not depend on timing.  Two cluster barriers separate the phases; every thread reaches both,
// also after a timed-out wait.  The hand-over costs several microseconds per launch, so the
// launcher only splits GEMMs with a long K range (64 K blocks = K >= 4096 by default: FC2).
template <int EPI>
__global__ void __launch_bounds__(kGemmThreads, 1) gemm_bf16_splitk_kernel(
    const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
    const __grid_constant__ CUtensorMap tmap_c, const __grid_constant__ CUtensorMap tmap_c2, long M, int N, int K,
    EpiParams ep, int* err_flag, int split) {
  constexpr int BN = 128;
  // one staging set per warp for the residual epilogue (a warp has only two pieces to update): that
  // leaves six operand stages, 192 KB, for up to three partial accumulators
  using Cfg = SmemPlan<BN, EPI, 1>;
  static_assert(Cfg::kStagingOffset >= 3 * 65536, "three partial accumulators fit in the operand stages");
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t bar_base = smem_base + Cfg::kBarOffset;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (Cfg::kStages + s); };
  const uint32_t tfull_bar = bar_base + 8u * (2 * Cfg::kStages);
  const uint32_t xbar_base = bar_base + 8u * (2 * Cfg::kStages + 4);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_gen + Cfg::kBarOffset + 8 * Cfg::kNumBars);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_gen + Cfg::kBarOffset + 8 * Cfg::kNumBars + 8);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = (int)cluster_ctarank();
  const int tile = (int)blockIdx.x / split;

  if (threadIdx.x == 0) {
    for (int s = 0; s < Cfg::kStages; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    mbar_init(tfull_bar, 1);
    for (int i = 0; i < 4 * kXSets; ++i) mbar_init(xbar_base + 8u * i, 1);
    *abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), BN);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();  // nothing of another CTA is touched before the first cluster barrier below
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  griddep_wait();  // everything above overlapped the previous kernel's tail; its output is needed from here on
  griddep_launch_dependents();

  const int num_n = (N + BN - 1) / BN;
  const int num_k = (K + kBK - 1) / kBK;
  const int m0 = (tile / num_n) * kBM, n0 = (tile % num_n) * BN;
  const int kb0 = rank * num_k / split, kb1 = (rank + 1) * num_k / split;  // split <= num_k: never empty
  const int quarter = warp & 3;
  const uint32_t stage_base = smem_base + Cfg::kStagingOffset + (uint32_t)((warp - 2) * Cfg::kStagingPerWarp);
  const uint32_t xbar0 = xbar_base + 8u * (uint32_t)((warp - 2) * kXSets);
  const XWalk walk{tile, 1 << 30, tile + 1, num_n, kBM, quarter * 32, BN, BN / 64};
  XState xs{0u, 0u, 0u};
  bool acc_ok = true;  // epilogue warps: this CTA's accumulator is complete

  // ---- phase 1: this CTA's share of the K range
  if (warp == 0) {
    if (lane == 0) {
      prefetch_tmap(&tmap_a);
      prefetch_tmap(&tmap_b);
      int stage = 0;
      uint32_t phase = 0, armed = 0, armed_parity = 0;
      bool ok = true;
      for (int kb = kb0; kb < kb1; ++kb) {
        if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) { ok = false; break; }
        mbar_arrive_expect_tx(full_bar(stage), Cfg::kStageBytes);
        const uint32_t sa = smem_base + stage * Cfg::kStageBytes;
        tma_load_2d(sa, &tmap_a, kb * kBK, m0, full_bar(stage));
        tma_load_2d(sa + Cfg::kABytes, &tmap_b, kb * kBK, n0, full_bar(stage));
        armed |= 1u << stage;
        armed_parity = (armed_parity & ~(1u << stage)) | (phase << stage);
        if (++stage == Cfg::kStages) { stage = 0; phase ^= 1u; }
      }
      if (!ok) {
        atomicExch(err_flag, 7);
        drain_stages(full_bar(0), Cfg::kStages, armed, armed_parity);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(kBM, BN, 0, 0);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int kb = kb0; kb < kb1; ++kb) {
        if (!mbar_wait(full_bar(stage), phase, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t sa = smem_base + stage * Cfg::kStageBytes;
        const uint64_t adesc = umma_desc_k_sw128(sa);
        const uint64_t bdesc = umma_desc_k_sw128(sa + Cfg::kABytes);
#pragma unroll
        for (int k = 0; k < kBK / 16; ++k) umma_bf16(tmem_base, adesc + 2 * k, bdesc + 2 * k, idesc, (kb > kb0 || k != 0) ? 1u : 0u);
        umma_commit(empty_bar(stage));
        if (++stage == Cfg::kStages) { stage = 0; phase ^= 1u; }
      }
      if (ok) umma_commit(tfull_bar);
      else atomicExch(err_flag, 8);
    }
  } else {
    if (EPI == kEpiResidSplit && rank == 0 && lane == 0) {
      prefetch_tmap(&tmap_c);
      prefetch_tmap(&tmap_c2);
    }
    acc_ok = __all_sync(0xffffffffu, mbar_wait(tfull_bar, 0, abort_flag));
    if (!acc_ok && lane == 0) atomicExch(err_flag, 9);
    tc_fence_after();
  }
  // every CTA's accumulator is complete and its operand stages are idle (all its MMAs have completed)
  tc_fence_before();
  cluster_sync_all();

  // ---- phase 2: CTAs 1 .. split - 1 hand their accumulators to CTA 0
  if (warp >= 2 && rank > 0) {
    tc_fence_after();
    const int row = quarter * 32 + lane;
    const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16);
#pragma unroll 1
    for (int c = 0; c < BN / 32; ++c) {
      uint32_t a32[32];
      tmem_ld_32x32(t_row + c * 32, a32);
      tmem_ld_wait();
#pragma unroll
      for (int g = 0; g < 8; ++g)
        st_cluster_v4(map_to_cta(partial_addr(smem_base, rank - 1, row, 8 * c + g), 0), a32[4 * g], a32[4 * g + 1],
                      a32[4 * g + 2], a32[4 * g + 3]);
    }
  }
  cluster_sync_all();  // release / acquire: the partials are visible in CTA 0

  // ---- phase 3: CTA 0 adds them up and runs the epilogue
  if (warp >= 2 && rank == 0) {
    tc_fence_after();
    const Partials ps{smem_base, split - 1};
    const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16);
    uint32_t piece = 0;
    bool ok = true;
    if constexpr (EPI == kEpiResidSplit)
      ok = epilogue_tile_split<BN, 1, 0>(ep, &tmap_c, &tmap_c2, t_row, m0, n0, M, N, quarter, lane, stage_base, xbar0, walk, xs,
                                         abort_flag, ps);
    else
      epilogue_tile<BN, EPI>(ep, &tmap_c, t_row, m0, n0, M, N, K, quarter, lane, stage_base, piece, ps);
    if (!ok && lane == 0) {
      atomicExch(err_flag, 9);
      x_drain(xbar0, xs);
    }
    if (lane == 0) bulk_wait_all();  // every store this lane issued has completed
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, BN);
  }
}

// ---------------------------------------------------------------------------------------------
// The same GEMM on CTA pairs (thread-block clusters of two, tcgen05 cta_group::2): one MMA
// covers a 256 x 256 tile, 128 rows per CTA, and each CTA stages only half of the W tile
// (128 of the 256 output columns), which cuts the shared-memory traffic per flop by a third.
//   - both CTAs run a TMA producer for their own halves; every copy signals the full barrier
//     of the pair's first CTA (the leader), which alone issues the MMAs;
//   - tcgen05.commit multicasts "stage free" and "accumulator ready" to both CTAs;
//   - the epilogue warps of both CTAs arrive on the leader's "accumulator drained" barrier.
// Tiles are dealt round-robin to the pairs.
template <int EPI>
__global__ void __launch_bounds__(kGemmThreads, 1) gemm_bf16_pair_kernel(
    const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
    const __grid_constant__ CUtensorMap tmap_c, const __grid_constant__ CUtensorMap tmap_c2, long M, int N, int K,
    int a_cols, EpiParams ep, int* err_flag) {
  constexpr int BN = 256;
  using Cfg = SmemPlan<BN / 2, EPI>;  // this CTA's 128 rows of A and 128 of the 256 W rows per stage: 32 KB
  constexpr int kStages = Cfg::kStages;
  constexpr int kABytes = Cfg::kABytes;
  constexpr int kStageBytes = Cfg::kStageBytes;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t bar_base = smem_base + Cfg::kBarOffset;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (kStages + s); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * kStages + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * kStages + 2 + a); };
  const uint32_t xbar_base = bar_base + 8u * (2 * kStages + 4);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_gen + Cfg::kBarOffset + 8 * Cfg::kNumBars);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_gen + Cfg::kBarOffset + 8 * Cfg::kNumBars + 8);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();  // 0 = leader
  const int pair_id = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(full_bar(s), 1);    // used in the leader only: its producer's arrive + both CTAs' bytes
      mbar_init(empty_bar(s), 1);   // one multicast commit
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(tfull_bar(a), 1);   // one multicast commit
      mbar_init(tempty_bar(a), 8);  // used in the leader only: 4 epilogue warps of each CTA
    }
    for (int i = 0; i < 4 * kXSets; ++i) mbar_init(xbar_base + 8u * i, 1);
    *abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc_pair(smem_u32(const_cast<uint32_t*>(tmem_slot)), 512);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  cluster_sync_all();  // barriers of both CTAs are initialised before anyone signals them
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  griddep_wait();  // everything above overlapped the previous kernel's tail; its output is needed from here on
  griddep_launch_dependents();

  const int num_m = (int)((M + 2 * kBM - 1) / (2 * kBM));
  const int num_n = (N + BN - 1) / BN;
  const int num_k = (K + kBK - 1) / kBK;
  const int num_tiles = num_m * num_n;

  if (warp == 0) {
    if (lane == 0) {
      prefetch_tmap(&tmap_a);
      prefetch_tmap(&tmap_b);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int tile = pair_id; ok && tile < num_tiles; tile += n_pairs) {
        const int m0 = (tile / num_n) * (2 * kBM) + (int)rank * kBM;
        const int n0 = (tile % num_n) * BN + (int)rank * (BN / 2);
        for (int kb = 0; kb < num_k; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag)) { ok = false; break; }
          const uint32_t leader_full = map_to_cta(full_bar(stage), 0);  // the leader CTA's barrier
          if (rank == 0) mbar_arrive_expect_tx(full_bar(stage), 2 * kStageBytes);
          const uint32_t sa = smem_base + stage * kStageBytes;
          const int e = kb * kBK;
          tma_load_2d_pair(sa, &tmap_a, e % a_cols, m0 + e / a_cols, leader_full);
          tma_load_2d_pair(sa + kABytes, &tmap_b, kb * kBK, n0, leader_full);
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        atomicExch(err_flag, 4);
        // This thread's copies signal the leader's barriers, which only the leader's MMA thread
        // follows; what can be waited for here is that the stages it filled were consumed, i.e. one
        // more lap of the "stage free" barriers, each wait bounded.
        for (int s = 0; s < kStages; ++s)
          for (uint32_t it = 0; it < (1u << 16); ++it)
            if (mbar_try_wait(empty_bar(s), (s < stage ? phase : phase ^ 1u))) break;
      }
    }
  } else if (warp == 1) {
    if (rank == 0 && lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(2 * kBM, BN, 0, 0);
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int tile = pair_id; ok && tile < num_tiles; tile += n_pairs) {
        if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
        for (int kb = 0; kb < num_k; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = smem_base + stage * kStageBytes;
          const uint64_t adesc = umma_desc_k_sw128(sa);
          const uint64_t bdesc = umma_desc_k_sw128(sa + kABytes);
#pragma unroll
          for (int k = 0; k < kBK / 16; ++k)
            umma_bf16_pair(d_tmem, adesc + 2 * k, bdesc + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
          umma_commit_pair(empty_bar(stage), 3);
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        umma_commit_pair(tfull_bar(acc), 3);
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
      if (!ok) atomicExch(err_flag, 5);
    }
  } else {
    const int quarter = warp & 3;
    const uint32_t stage_base = smem_base + Cfg::kStagingOffset + (uint32_t)((warp - 2) * Cfg::kStagingPerWarp);
    const uint32_t xbar0 = xbar_base + 8u * (uint32_t)((warp - 2) * kXSets);
    const XWalk walk{pair_id, n_pairs, num_tiles, num_n, 2 * kBM, (int)rank * kBM + quarter * 32, BN, BN / 64};
    XState xs{0u, 0u, 0u};
    if (EPI == kEpiResidSplit && lane == 0) {
      prefetch_tmap(&tmap_c);
      prefetch_tmap(&tmap_c2);
      for (uint32_t p = 0; p < (uint32_t)kXLook; ++p) x_fetch(walk, p, M, N, &tmap_c, &tmap_c2, stage_base, xbar0, xs.armed);
    }
    uint32_t piece = 0;
    int acc = 0;
    uint32_t acc_phase = 0;
    for (int tile = pair_id; tile < num_tiles; tile += n_pairs) {
      const int m0 = (tile / num_n) * (2 * kBM) + (int)rank * kBM;
      const int n0 = (tile % num_n) * BN;
      bool ok = mbar_wait(tfull_bar(acc), acc_phase, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (ok) {
        tc_fence_after();
        const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BN);
        if constexpr (EPI == kEpiResidSplit)
          ok = epilogue_tile_split<BN>(ep, &tmap_c, &tmap_c2, t_row, m0, n0, M, N, quarter, lane, stage_base, xbar0, walk, xs,
                                       abort_flag);
        else
          epilogue_tile<BN, EPI>(ep, &tmap_c, t_row, m0, n0, M, N, K, quarter, lane, stage_base, piece);
      }
      if (!ok) {
        if (lane == 0) {
          atomicExch(err_flag, 6);
          x_drain(xbar0, xs);
        }
        break;
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(map_to_cta(tempty_bar(acc), 0));
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
    if (lane == 0) bulk_wait_all();
  }

  tc_fence_before();
  cluster_sync_all();  // neither CTA leaves while the other may still touch its memory or barriers
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, 512);
  }
}

// ---------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

bool tma_api_init(TmaApi* api) {
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
  if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || fn == nullptr) return false;
  api->encode_tiled = fn;
  return true;
}

bool make_tmap_2d(const TmaApi& api, CUtensorMap* m, const void* base, int elem_bytes, uint64_t cols,
                  uint64_t rows, uint64_t pitch_elems, uint32_t box_cols, uint32_t box_rows) {
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {pitch_elems * (uint64_t)elem_bytes};
  cuuint32_t box[2] = {box_cols, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = reinterpret_cast<EncodeTiledFn>(api.encode_tiled)(
      m, elem_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2,
      const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
      CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

bool make_tmap_bf16(const TmaApi& api, CUtensorMap* m, const void* base, uint64_t cols, uint64_t rows,
                    uint64_t pitch_elems, uint32_t box_rows) {
  return make_tmap_2d(api, m, base, 2, cols, rows, pitch_elems, (uint32_t)kBK, box_rows);
}

bool make_tmap_out(const TmaApi& api, CUtensorMap* m, const void* base, int elem_bytes, uint64_t cols,
                   uint64_t rows) {
  return make_tmap_2d(api, m, base, elem_bytes, cols, rows, cols, elem_bytes == 2 ? 64 : 32, 32);
}

template <int EPI>
static cudaError_t configure_one() {
  cudaError_t e = cudaFuncSetAttribute(gemm_bf16_kernel<128, EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       SmemPlan<128, EPI>::kSmemBytes);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(gemm_bf16_kernel<256, EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              SmemPlan<256, EPI>::kSmemBytes);
}

template <int EPI>
static cudaError_t configure_splitk() {
  return cudaFuncSetAttribute(gemm_bf16_splitk_kernel<EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              SmemPlan<128, EPI, 1>::kSmemBytes);
}

template <int EPI>
static cudaError_t configure_pair() {
  cudaError_t e = cudaFuncSetAttribute(gemm_bf16_pair_kernel<EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       SmemPlan<128, EPI>::kSmemBytes);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(gemm_bf16_pair_kernel<EPI>, cudaFuncAttributeNonPortableClusterSizeAllowed, 0);
}

// Function attributes are per device: called by every create, on the device that is current then.
cudaError_t gemm_bf16_configure() {
  cudaError_t e;
  if ((e = configure_pair<kEpiBias>()) != cudaSuccess) return e;
  if ((e = configure_pair<kEpiBiasGelu>()) != cudaSuccess) return e;
  if ((e = configure_pair<kEpiConv1>()) != cudaSuccess) return e;
  if ((e = configure_pair<kEpiConv2>()) != cudaSuccess) return e;
  if ((e = configure_pair<kEpiLnBias>()) != cudaSuccess) return e;
  if ((e = configure_pair<kEpiLnBiasGelu>()) != cudaSuccess) return e;
  if ((e = configure_pair<kEpiResidSplit>()) != cudaSuccess) return e;
  if ((e = configure_one<kEpiBias>()) != cudaSuccess) return e;
  if ((e = configure_one<kEpiBiasGelu>()) != cudaSuccess) return e;
  if ((e = configure_one<kEpiLnBias>()) != cudaSuccess) return e;
  if ((e = configure_one<kEpiLnBiasGelu>()) != cudaSuccess) return e;
  if ((e = configure_one<kEpiResidSplit>()) != cudaSuccess) return e;
  if ((e = configure_splitk<kEpiBias>()) != cudaSuccess) return e;
  if ((e = configure_splitk<kEpiBiasGelu>()) != cudaSuccess) return e;
  if ((e = configure_splitk<kEpiLnBias>()) != cudaSuccess) return e;
  if ((e = configure_splitk<kEpiLnBiasGelu>()) != cudaSuccess) return e;
  if ((e = configure_splitk<kEpiResidSplit>()) != cudaSuccess) return e;
  return cudaSuccess;
}

template <int EPI, int BN = 128>
static void launch_one(const CUtensorMap& ta, const CUtensorMap& tb, const CUtensorMap& tc, const CUtensorMap& tc2,
                       long M, int N, int K, int a_cols, const EpiParams& ep, int* err_flag, int num_sms, bool pdl,
                       cudaStream_t s) {
  const long tiles = ((M + kBM - 1) / kBM) * ((N + BN - 1) / BN);
  const int grid = (int)(tiles < num_sms ? tiles : num_sms);
  launch_dependent(gemm_bf16_kernel<BN, EPI>, dim3(grid), dim3(kGemmThreads), SmemPlan<BN, EPI>::kSmemBytes, s, 1, pdl,
                   ta, tb, tc, tc2, M, N, K, a_cols, ep, err_flag);
}

template <int EPI>
static void launch_splitk(const CUtensorMap& ta, const CUtensorMap& tb, const CUtensorMap& tc, const CUtensorMap& tc2,
                          long M, int N, int K, const EpiParams& ep, int* err_flag, int split, bool pdl, cudaStream_t s) {
  const long tiles = ((M + kBM - 1) / kBM) * ((N + 127) / 128);
  launch_dependent(gemm_bf16_splitk_kernel<EPI>, dim3((unsigned)(tiles * split)), dim3(kGemmThreads),
                   SmemPlan<128, EPI, 1>::kSmemBytes, s, split, pdl, ta, tb, tc, tc2, M, N, K, ep, err_flag, split);
}

template <int EPI>
static void launch_pair(const CUtensorMap& ta, const CUtensorMap& tb, const CUtensorMap& tc, const CUtensorMap& tc2,
                        long M, int N, int K, int a_cols, const EpiParams& ep, int* err_flag, int num_sms, bool pdl,
                        cudaStream_t s) {
  const long tiles = ((M + 2 * kBM - 1) / (2 * kBM)) * ((N + 255) / 256);
  const long max_pairs = num_sms / 2;
  const long pairs = tiles < max_pairs ? tiles : max_pairs;
  launch_dependent(gemm_bf16_pair_kernel<EPI>, dim3((unsigned)(2 * pairs)), dim3(kGemmThreads),
                   SmemPlan<128, EPI>::kSmemBytes, s, 2, pdl, ta, tb, tc, tc2, M, N, K, a_cols, ep, err_flag);
}

void launch_gemm_bf16(const CUtensorMap& ta, const CUtensorMap& tb, const CUtensorMap& tc, const CUtensorMap& tc2,
                      long M, int N, int K, int a_cols, int epi, const EpiParams& ep, int* err_flag, int num_sms,
                      const LaunchOpts& opt, cudaStream_t s) {
  if (M <= 0 || N <= 0 || K <= 0) return;
  const bool pdl = opt.pdl != 0;
  // Small problems leave most CTA pairs idle or waste most of a last round of 256 x 256 tiles:
  // 128 x 128 tiles on single CTAs (same tensor maps: both use 128-row boxes) quarter the
  // granularity.  Estimated rounds, a 128 x 128 tile counted as half a pair tile's time times
  // kSmallTilePenalty for its lower efficiency (it reads shared memory at the full 128 B/clk;
  // measured: a round of small tiles takes ~0.8 of a round of pair tiles).
  if (opt.small_tiles && epi != kEpiConv1 && epi != kEpiConv2 && a_cols == K) {
    // Estimated time in rounds of tiles, in units of one round of 256 x 256 pair tiles (measured on
    // the FC1 shape at M = 775: a round of 128 x 128 tiles takes ~0.8 of that, a round of 128 x 256
    // tiles ~1.25: per K block a CTA takes in 32 / 32 / 48 KB)
    constexpr double kRound128 = 0.8, kRound256 = 1.25;
    const long t_pair = ((M + 2 * kBM - 1) / (2 * kBM)) * ((N + 255) / 256);
    const long t_small = ((M + kBM - 1) / kBM) * ((N + 127) / 128);
    const long t_wide = ((M + kBM - 1) / kBM) * ((N + 255) / 256);
    const long n_pairs = num_sms / 2;
    double r_pair = (double)((t_pair + n_pairs - 1) / n_pairs);
    double r_small = (double)((t_small + num_sms - 1) / num_sms) * kRound128;
    double r_wide = (double)((t_wide + num_sms - 1) / num_sms) * kRound256;
    if (opt.tile == 1) r_small = r_wide = 1e30;
    if (opt.tile == 2) r_pair = r_wide = 1e30;
    if (opt.tile == 3) r_pair = r_small = 1e30;
    if (r_wide < r_pair && r_wide < r_small) {
      switch (epi) {
        case kEpiBias: launch_one<kEpiBias, 256>(ta, tb, tc, tc2, M, N, K, a_cols, ep, err_flag, num_sms, pdl, s); break;
        case kEpiBiasGelu: launch_one<kEpiBiasGelu, 256>(ta, tb, tc, tc2, M, N, K, a_cols, ep, err_flag, num_sms, pdl, s); break;
        case kEpiLnBias: launch_one<kEpiLnBias, 256>(ta, tb, tc, tc2, M, N, K, a_cols, ep, err_flag, num_sms, pdl, s); break;
        case kEpiLnBiasGelu: launch_one<kEpiLnBiasGelu, 256>(ta, tb, tc, tc2, M, N, K, a_cols, ep, err_flag, num_sms, pdl, s); break;
        default: launch_one<kEpiResidSplit, 256>(ta, tb, tc, tc2, M, N, K, a_cols, ep, err_flag, num_sms, pdl, s); break;
      }
      return;
    }
    if (r_small < r_pair) {
      // so few tiles that half of the SMs or more would idle, and a K range long enough for the
      // hand-over between the CTAs to pay: split every tile's K range over a cluster of 2 or 4 CTAs
      const long num_k = (K + kBK - 1) / kBK;
      const bool may = opt.split_k > 0 && num_k >= opt.split_k;
      const int split = (may && t_small * 4 <= num_sms && num_k >= 16) ? 4 : (may && t_small * 2 <= num_sms && num_k >= 8) ? 2 : 1;
      if (split > 1) {
        switch (epi) {
          case kEpiBias: launch_splitk<kEpiBias>(ta, tb, tc, tc2, M, N, K, ep, err_flag, split, pdl, s); break;
          case kEpiBiasGelu: launch_splitk<kEpiBiasGelu>(ta, tb, tc, tc2, M, N, K, ep, err_flag, split, pdl, s); break;
          case kEpiLnBias: launch_splitk<kEpiLnBias>(ta, tb, tc, tc2, M, N, K, ep, err_flag, split, pdl, s); break;
          case kEpiLnBiasGelu: launch_splitk<kEpiLnBiasGelu>(ta, tb, tc, tc2, M, N, K, ep, err_flag, split, pdl, s); break;
          default: launch_splitk<kEpiResidSplit>(ta, tb, tc, tc2, M, N, K, ep, err_flag, split, pdl, s); break;
        }
        return;
      }
      switch (epi) {
        case kEpiBias: launch_one<kEpiBias>(ta, tb, tc, tc2, M, N, K, a_cols, ep, err_flag, num_sms, pdl, s); break;
        case kEpiBiasGelu: launch_one<kEpiBiasGelu>(ta, tb, tc, tc2, M, N, K, a_cols, ep, err_flag, num_sms, pdl, s); break;
        case kEpiLnBias: launch_one<kEpiLnBias>(ta, tb, tc, tc2, M, N, K, a_cols, ep, err_flag, num_sms, pdl, s); break;
        case kEpiLnBiasGelu: launch_one<kEpiLnBiasGelu>(ta, tb, tc, tc2, M, N, K, a_cols, ep, err_flag, num_sms, pdl, s); break;
        default: launch_one<kEpiResidSplit>(ta, tb, tc, tc2, M, N, K, a_cols, ep, err_flag, num_sms, pdl, s); break;
      }
      return;
    }
  }
  switch (epi) {
    case kEpiBias: launch_pair<kEpiBias>(ta, tb, tc, tc2, M, N, K, a_cols, ep, err_flag, num_sms, pdl, s); break;
    case kEpiBiasGelu: launch_pair<kEpiBiasGelu>(ta, tb, tc, tc2, M, N, K, a_cols, ep, err_flag, num_sms, pdl, s); break;
    case kEpiConv1: launch_pair<kEpiConv1>(ta, tb, tc, tc2, M, N, K, a_cols, ep, err_flag, num_sms, pdl, s); break;
    case kEpiConv2: launch_pair<kEpiConv2>(ta, tb, tc, tc2, M, N, K, a_cols, ep, err_flag, num_sms, pdl, s); break;
    case kEpiLnBias: launch_pair<kEpiLnBias>(ta, tb, tc, tc2, M, N, K, a_cols, ep, err_flag, num_sms, pdl, s); break;
    case kEpiLnBiasGelu: launch_pair<kEpiLnBiasGelu>(ta, tb, tc, tc2, M, N, K, a_cols, ep, err_flag, num_sms, pdl, s); break;
    default: launch_pair<kEpiResidSplit>(ta, tb, tc, tc2, M, N, K, a_cols, ep, err_flag, num_sms, pdl, s); break;
  }
}

}  // namespace wf
