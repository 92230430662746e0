// bf16 GEMM for sm_100a: C = epilogue(A W^T), A [M, K] and W [N, K] both K-major.
//
// Persistent, warp-specialised CTAs of 192 threads:
//   warp 0      one lane issues TMA loads (A 128 x 64 and W BN x 64 boxes, 128-byte swizzle)
//               into a ring of shared-memory stages guarded by full/empty mbarriers;
//   warp 1      allocates tensor memory, one lane issues tcgen05.mma (128 x BN x 16, f32
//               accumulation in TMEM) and commits stage releases / accumulator readiness;
//   warps 2..5  read the accumulator with tcgen05.ld (one row per thread), apply the fused
//               epilogue, stage 32-row x 128-byte pieces in swizzled shared memory and hand them
//               to TMA: a tile store for bf16 outputs, a float32 add-reduction (performed at the
//               L2) for the residual update, so the residual is never read by the SM.  This runs
//               while the MMA warp already fills the other accumulator buffer.
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

template <int BN>
struct GemmCfg {
  static constexpr int kStages = BN == 256 ? 4 : 6;
  static constexpr int kABytes = kBM * kBK * 2;
  static constexpr int kBBytes = BN * kBK * 2;
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kStagingOffset = kStages * kStageBytes;       // 4 warps x 2 buffers x 4 KB
  static constexpr int kStagingBytes = 4 * 2 * 4096;
  static constexpr int kBarOffset = kStagingOffset + kStagingBytes;
  static constexpr int kSmemBytes = kBarOffset + 256 + 1024;  // barriers + alignment slack
  static constexpr int kTmemCols = 2 * BN;
};

// bias add (+ GELU) of 32 accumulator columns starting at col0 (col0 + 32 <= padded N is not
// required: columns at or beyond N are computed from a clamped bias index and never stored).
template <int EPI>
__device__ __forceinline__ void bias_act32(const EpiParams& ep, int col0, int N, const uint32_t (&acc)[32],
                                           float (&v)[32], bool with_bias = true) {
#pragma unroll
  for (int g = 0; g < 8; ++g) {
    int col = col0 + 4 * g;
    float4 b = (col < N && with_bias) ? __ldg(reinterpret_cast<const float4*>(ep.bias + col)) : make_float4(0.f, 0.f, 0.f, 0.f);
    unpack_f32x2(add_f32x2(pack_f32x2(__uint_as_float(acc[4 * g + 0]), __uint_as_float(acc[4 * g + 1])),
                           pack_f32x2(b.x, b.y)), v[4 * g + 0], v[4 * g + 1]);
    unpack_f32x2(add_f32x2(pack_f32x2(__uint_as_float(acc[4 * g + 2]), __uint_as_float(acc[4 * g + 3])),
                           pack_f32x2(b.z, b.w)), v[4 * g + 2], v[4 * g + 3]);
  }
  if (EPI == kEpiBiasGelu || EPI == kEpiConv1 || EPI == kEpiConv2) {
#pragma unroll
    for (int i = 0; i < 32; i += 2) gelu_sigmoid_poly2(v[i], v[i + 1]);
  }
}

// Direct (non-TMA) store of one row segment for the stride-2 conv epilogue, whose output rows
// are remapped per sequence: resid[dst] = gelu(acc + bias) + pe[pos].
__device__ __forceinline__ void conv2_store32(const EpiParams& ep, long row, long M, int col0, int N,
                                              const float (&v)[32]) {
  if (row >= M || col0 >= N) return;
  int2 d = ep.row_dst[row];
  if (d.x < 0) return;
#pragma unroll
  for (int g = 0; g < 8; ++g) {
    int col = col0 + 4 * g;
    if (col >= N) break;
    float4 e = __ldg(reinterpret_cast<const float4*>(ep.pe + (long)d.y * ep.ldc + col));
    *reinterpret_cast<float4*>(ep.resid + (long)d.x * ep.ldc + col) =
        make_float4(v[4 * g] + e.x, v[4 * g + 1] + e.y, v[4 * g + 2] + e.z, v[4 * g + 3] + e.w);
  }
}

// Epilogue of one 128 x BN accumulator tile for the warp that owns TMEM lanes 32 * quarter ..:
// t_row is the tensor-memory address of that lane group's first column of the tile, m0 / n0 the
// tile origin in the output, stage_base this warp's two 4 KB staging buffers.
template <int BN, int EPI, int NBUF = 2>
__device__ __forceinline__ void epilogue_tile(const EpiParams& ep, const CUtensorMap* tmap_c, uint32_t t_row, int m0,
                                              int n0, long M, int N, int quarter, int lane, uint32_t stage_base,
                                              uint32_t& piece, bool with_bias = true) {
  const long row = (long)m0 + quarter * 32 + lane;
  if (EPI == kEpiConv2) {
#pragma unroll 1
    for (int c = 0; c < BN / 32; ++c) {
      uint32_t a32[32];
      float v[32];
      tmem_ld_32x32(t_row + c * 32, a32);
      tmem_ld_wait();
      bias_act32<EPI>(ep, n0 + c * 32, N, a32, v);
      conv2_store32(ep, row, M, n0 + c * 32, N, v);
    }
  } else if (EPI == kEpiBiasResid) {
    // float32: 32 columns = 128 bytes per row and piece
#pragma unroll 1
    for (int c = 0; c < BN / 32; ++c) {
      const uint32_t buf = stage_base + (uint32_t)((piece % NBUF) * 4096);
      if (lane == 0) bulk_wait_read<NBUF - 1>();   // the copy that last read this buffer is done with it
      __syncwarp();
      uint32_t a32[32];
      float v[32];
      tmem_ld_32x32(t_row + c * 32, a32);
      tmem_ld_wait();
      bias_act32<EPI>(ep, n0 + c * 32, N, a32, v, with_bias);
#pragma unroll
      for (int j = 0; j < 8; ++j)
        st_shared_v4(buf + lane * 128 + ((j ^ (lane & 7)) << 4), __float_as_uint(v[4 * j]),
                     __float_as_uint(v[4 * j + 1]), __float_as_uint(v[4 * j + 2]), __float_as_uint(v[4 * j + 3]));
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) {
        if (n0 + c * 32 < N && (long)m0 + quarter * 32 < M) tma_reduce_add_2d(tmap_c, buf, n0 + c * 32, m0 + quarter * 32);
        bulk_commit();  // one group per piece, empty when the piece lies outside the matrix: wait_read<1>
                        // above counts groups to know that the copy two pieces back has let go of its buffer
      }
      ++piece;
    }
  } else {
    // bf16: 64 columns = 128 bytes per row and piece
    bool valid = true;
    if (EPI == kEpiConv1) valid = row < M && ep.row_valid[row] != 0;
#pragma unroll 1
    for (int c = 0; c < BN / 64; ++c) {
      const uint32_t buf = stage_base + (uint32_t)((piece % NBUF) * 4096);
      if (lane == 0) bulk_wait_read<NBUF - 1>();
      __syncwarp();
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
        uint32_t a32[32];
        float v[32];
        tmem_ld_32x32(t_row + c * 64 + hf * 32, a32);
        tmem_ld_wait();
        bias_act32<EPI>(ep, n0 + c * 64 + hf * 32, N, a32, v);
        if (EPI == kEpiConv1 && !valid) {
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
        bulk_commit();  // one group per piece, also when nothing was stored (see above)
      }
      ++piece;
    }
  }
}

template <int BN, int EPI>
__global__ void __launch_bounds__(kGemmThreads, 1) gemm_bf16_kernel(
    const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
    const __grid_constant__ CUtensorMap tmap_c, long M, int N, int K, int a_cols, EpiParams ep, int* err_flag) {
  using Cfg = GemmCfg<BN>;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t bar_base = smem_base + Cfg::kBarOffset;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (Cfg::kStages + s); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * Cfg::kStages + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * Cfg::kStages + 2 + a); };
  volatile uint32_t* tmem_slot =
      reinterpret_cast<volatile uint32_t*>(smem_gen + Cfg::kBarOffset + 8 * (2 * Cfg::kStages + 4));
  volatile int* abort_flag =
      reinterpret_cast<volatile int*>(smem_gen + Cfg::kBarOffset + 8 * (2 * Cfg::kStages + 4) + 8);

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
    *abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), Cfg::kTmemCols);
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
          armed |= 1u << stage;
          armed_parity = (armed_parity & ~(1u << stage)) | (phase << stage);
          if (++stage == Cfg::kStages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        atomicExch(err_flag, 1);
        // Let the copies this thread issued land before the CTA's shared memory is released.
        for (int s = 0; s < Cfg::kStages; ++s) {
          if (!(armed & (1u << s))) continue;
          for (uint32_t it = 0; it < (1u << 20); ++it)
            if (mbar_try_wait(full_bar(s), (armed_parity >> s) & 1u)) break;
        }
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
    const uint32_t stage_base = smem_base + Cfg::kStagingOffset + (uint32_t)((warp - 2) * 8192);
    uint32_t piece = 0;
    int acc = 0;
    uint32_t acc_phase = 0;
    for (int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x) {
      const int m0 = (tile / num_n) * kBM, n0 = (tile % num_n) * BN;
      bool ok = mbar_wait(tfull_bar(acc), acc_phase, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) {
        if (lane == 0) atomicExch(err_flag, 3);
        break;
      }
      tc_fence_after();
      epilogue_tile<BN, EPI>(ep, &tmap_c, tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BN), m0, n0,
                             M, N, quarter, lane, stage_base, piece);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty_bar(acc));
      if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
    }
    if (lane == 0) bulk_wait_all();  // every store / reduction this lane issued has completed
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, Cfg::kTmemCols);
  }
}

// Work units of the CTA-pair kernel.  Tiles are dealt round-robin to the pairs; the tiles of the
// last, partial round are cut along K into `split` parts (only for the residual epilogue, whose
// float32 add-reduction makes partial sums free to combine), so that every pair has work in
// that round too.  Unit u < full is the whole tile u; the others are (tile, K part) pairs, with
// the bias added by part 0 alone.
struct GemmUnit {
  int tile, kb0, kb1;
  bool first;
};
__device__ __forceinline__ GemmUnit gemm_unit(int u, int full, int rem, int split, int num_k) {
  if (u < full) return GemmUnit{u, 0, num_k, true};
  const int v = u - full, part = v / rem;
  return GemmUnit{full + v % rem, part * num_k / split, (part + 1) * num_k / split, part == 0};
}

// ---------------------------------------------------------------------------------------------
// The same GEMM on CTA pairs (thread-block clusters of two, tcgen05 cta_group::2): one MMA
// covers a 256 x 256 tile, 128 rows per CTA, and each CTA stages only half of the W tile
// (128 of the 256 output columns), which cuts the shared-memory traffic per flop by a third.
//   - both CTAs run a TMA producer for their own halves; every copy signals the full barrier
//     of the pair's first CTA (the leader), which alone issues the MMAs;
//   - tcgen05.commit multicasts "stage free" and "accumulator ready" to both CTAs;
//   - the epilogue warps of both CTAs arrive on the leader's "accumulator drained" barrier.
template <int EPI>
__global__ void __launch_bounds__(kGemmThreads, 1) gemm_bf16_pair_kernel(
    const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
    const __grid_constant__ CUtensorMap tmap_c, long M, int N, int K, int a_cols, EpiParams ep, int* err_flag,
    int tail_split) {
  constexpr int BN = 256;
  // The float32 add-reduction holds its staging buffer for ~2 us (the L2 performs the additions), so
  // with two buffers per warp the residual epilogue is latency-bound at ~13 GB/s per CTA and the
  // K = 1280 out-projection waits for it: that epilogue gets four buffers per warp, paid for with
  // one operand stage.
  constexpr int kStages = EPI == kEpiBiasResid ? 5 : 6;
  constexpr int kBufs = EPI == kEpiBiasResid ? 4 : 2;
  constexpr int kABytes = kBM * kBK * 2;          // this CTA's 128 rows of A
  constexpr int kBBytes = (BN / 2) * kBK * 2;     // this CTA's 128 of the 256 W rows
  constexpr int kStageBytes = kABytes + kBBytes;  // 32 KB
  constexpr int kStagingOffset = kStages * kStageBytes;
  constexpr int kBarOffset = kStagingOffset + 4 * kBufs * 4096;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t bar_base = smem_base + kBarOffset;
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (kStages + s); };
  auto tfull_bar = [&](int a) { return bar_base + 8u * (2 * kStages + a); };
  auto tempty_bar = [&](int a) { return bar_base + 8u * (2 * kStages + 2 + a); };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem_gen + kBarOffset + 8 * (2 * kStages + 4));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem_gen + kBarOffset + 8 * (2 * kStages + 4) + 8);

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
  const int full_tiles = (num_tiles / n_pairs) * n_pairs, rem_tiles = num_tiles - full_tiles;
  const int num_units = full_tiles + rem_tiles * tail_split;

  if (warp == 0) {
    if (lane == 0) {
      prefetch_tmap(&tmap_a);
      prefetch_tmap(&tmap_b);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int u = pair_id; ok && u < num_units; u += n_pairs) {
        const GemmUnit w = gemm_unit(u, full_tiles, rem_tiles, tail_split, num_k);
        const int m0 = (w.tile / num_n) * (2 * kBM) + (int)rank * kBM;
        const int n0 = (w.tile % num_n) * BN + (int)rank * (BN / 2);
        for (int kb = w.kb0; kb < w.kb1; ++kb) {
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
      if (!ok) atomicExch(err_flag, 4);
    }
  } else if (warp == 1) {
    if (rank == 0 && lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16(2 * kBM, BN, 0, 0);
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      bool ok = true;
      for (int u = pair_id; ok && u < num_units; u += n_pairs) {
        const GemmUnit w = gemm_unit(u, full_tiles, rem_tiles, tail_split, num_k);
        if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(acc * BN);
        for (int kb = w.kb0; kb < w.kb1; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = smem_base + stage * kStageBytes;
          const uint64_t adesc = umma_desc_k_sw128(sa);
          const uint64_t bdesc = umma_desc_k_sw128(sa + kABytes);
#pragma unroll
          for (int k = 0; k < kBK / 16; ++k)
            umma_bf16_pair(d_tmem, adesc + 2 * k, bdesc + 2 * k, idesc, (kb > w.kb0 || k != 0) ? 1u : 0u);
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
    const uint32_t stage_base = smem_base + kStagingOffset + (uint32_t)((warp - 2) * kBufs * 4096);
    uint32_t piece = 0;
    int acc = 0;
    uint32_t acc_phase = 0;
    for (int u = pair_id; u < num_units; u += n_pairs) {
      const GemmUnit w = gemm_unit(u, full_tiles, rem_tiles, tail_split, num_k);
      const int m0 = (w.tile / num_n) * (2 * kBM) + (int)rank * kBM;
      const int n0 = (w.tile % num_n) * BN;
      bool ok = mbar_wait(tfull_bar(acc), acc_phase, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) {
        if (lane == 0) atomicExch(err_flag, 6);
        break;
      }
      tc_fence_after();
      epilogue_tile<BN, EPI, kBufs>(ep, &tmap_c, tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * BN), m0, n0,
                             M, N, quarter, lane, stage_base, piece, w.first);
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

template <int BN, int EPI>
static cudaError_t configure_one() {
  return cudaFuncSetAttribute(gemm_bf16_kernel<BN, EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              GemmCfg<BN>::kSmemBytes);
}

constexpr int kPairSmemBytes = 6 * 32768 + 4 * 2 * 4096 + 256 + 1024;

template <int EPI>
static cudaError_t configure_pair() {
  cudaError_t e = cudaFuncSetAttribute(gemm_bf16_pair_kernel<EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       kPairSmemBytes);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(gemm_bf16_pair_kernel<EPI>, cudaFuncAttributeNonPortableClusterSizeAllowed, 0);
}

cudaError_t gemm_bf16_configure() {
  cudaError_t e;
  if ((e = configure_pair<kEpiBias>()) != cudaSuccess) return e;
  if ((e = configure_pair<kEpiBiasGelu>()) != cudaSuccess) return e;
  if ((e = configure_pair<kEpiBiasResid>()) != cudaSuccess) return e;
  if ((e = configure_pair<kEpiConv1>()) != cudaSuccess) return e;
  if ((e = configure_pair<kEpiConv2>()) != cudaSuccess) return e;
  if ((e = configure_one<256, kEpiBias>()) != cudaSuccess) return e;
  if ((e = configure_one<256, kEpiBiasGelu>()) != cudaSuccess) return e;
  if ((e = configure_one<256, kEpiBiasResid>()) != cudaSuccess) return e;
  if ((e = configure_one<256, kEpiConv1>()) != cudaSuccess) return e;
  if ((e = configure_one<256, kEpiConv2>()) != cudaSuccess) return e;
  if ((e = configure_one<128, kEpiBias>()) != cudaSuccess) return e;
  if ((e = configure_one<128, kEpiBiasGelu>()) != cudaSuccess) return e;
  if ((e = configure_one<128, kEpiBiasResid>()) != cudaSuccess) return e;
  return cudaSuccess;
}

template <int BN, int EPI>
static void launch_one(const CUtensorMap& ta, const CUtensorMap& tb, const CUtensorMap& tc, long M, int N, int K,
                       int a_cols, const EpiParams& ep, int* err_flag, int num_sms, cudaStream_t s) {
  const long tiles = ((M + kBM - 1) / kBM) * ((N + BN - 1) / BN);
  const int grid = (int)(tiles < num_sms ? tiles : num_sms);
  launch_dependent(gemm_bf16_kernel<BN, EPI>, dim3(grid), dim3(kGemmThreads), GemmCfg<BN>::kSmemBytes, s, 1, ta, tb, tc,
                   M, N, K, a_cols, ep, err_flag);
}

// pair = 1: CTA-pair kernel (W maps must then use 128-row boxes); 0: single-CTA kernel
static int g_gemm_use_pair = 1;
static int g_gemm_tail_split = 0;
static int g_gemm_small_tiles = 1;
void gemm_bf16_set_pair(int on) { g_gemm_use_pair = on; }
int gemm_bf16_uses_pair() { return g_gemm_use_pair; }
void gemm_bf16_set_tail_split(int on) { g_gemm_tail_split = on; }
void gemm_bf16_set_small_tiles(int on) { g_gemm_small_tiles = on; }

template <int EPI>
static void launch_pair(const CUtensorMap& ta, const CUtensorMap& tb, const CUtensorMap& tc, long M, int N, int K,
                        int a_cols, const EpiParams& ep, int* err_flag, int num_sms, cudaStream_t s) {
  const long tiles = ((M + 2 * kBM - 1) / (2 * kBM)) * ((N + 255) / 256);
  const long max_pairs = num_sms / 2;
  long pairs = tiles < max_pairs ? tiles : max_pairs;
  // the residual epilogue lets the tiles of the last, partial round be cut along K (see GemmUnit);
  // with fewer tiles than pairs that round is the only one, and more pairs are launched for it
  int tail_split = 1;
  if (EPI == kEpiBiasResid && g_gemm_tail_split) {
    const long num_k = (K + kBK - 1) / kBK;
    if (tiles < max_pairs) pairs = std::min(max_pairs, tiles * num_k);
    const long rem = tiles % pairs;
    if (rem > 0) tail_split = (int)std::max(1L, std::min(pairs / rem, num_k));
    if (tiles < max_pairs) pairs = tiles * tail_split;
  }
  launch_dependent(gemm_bf16_pair_kernel<EPI>, dim3((unsigned)(2 * pairs)), dim3(kGemmThreads), kPairSmemBytes, s, 2,
                   ta, tb, tc, M, N, K, a_cols, ep, err_flag, tail_split);
}

void launch_gemm_bf16(const CUtensorMap& ta, const CUtensorMap& tb, const CUtensorMap& tc, long M, int N, int K,
                      int a_cols, int epi, const EpiParams& ep, int* err_flag, int num_sms, cudaStream_t s) {
  if (M <= 0 || N <= 0 || K <= 0) return;
  if (g_gemm_use_pair) {
    // Small problems leave most CTA pairs idle or waste most of a last round of 256 x 256 tiles:
    // 128 x 128 tiles on single CTAs (same tensor maps: both use 128-row boxes) quarter the
    // granularity.  Estimated rounds, a 128 x 128 tile counted as half a pair tile's time times
    // kSmallTilePenalty for its lower efficiency (it reads shared memory at the full 128 B/clk;
    // measured: a round of small tiles takes ~0.8 of a round of pair tiles).
    if (g_gemm_small_tiles && epi <= kEpiBiasResid && a_cols == K) {
      constexpr double kSmallTilePenalty = 1.6;
      const long t_pair = ((M + 2 * kBM - 1) / (2 * kBM)) * ((N + 255) / 256);
      const long t_small = ((M + kBM - 1) / kBM) * ((N + 127) / 128);
      const long n_pairs = num_sms / 2;
      const double r_pair = (double)((t_pair + n_pairs - 1) / n_pairs);
      const double r_small = (double)((t_small + num_sms - 1) / num_sms) * 0.5 * kSmallTilePenalty;
      if (r_small < r_pair) {
        switch (epi) {
          case kEpiBias: launch_one<128, kEpiBias>(ta, tb, tc, M, N, K, a_cols, ep, err_flag, num_sms, s); break;
          case kEpiBiasGelu: launch_one<128, kEpiBiasGelu>(ta, tb, tc, M, N, K, a_cols, ep, err_flag, num_sms, s); break;
          default: launch_one<128, kEpiBiasResid>(ta, tb, tc, M, N, K, a_cols, ep, err_flag, num_sms, s); break;
        }
        return;
      }
    }
    switch (epi) {
      case kEpiBias: launch_pair<kEpiBias>(ta, tb, tc, M, N, K, a_cols, ep, err_flag, num_sms, s); break;
      case kEpiBiasGelu: launch_pair<kEpiBiasGelu>(ta, tb, tc, M, N, K, a_cols, ep, err_flag, num_sms, s); break;
      case kEpiBiasResid: launch_pair<kEpiBiasResid>(ta, tb, tc, M, N, K, a_cols, ep, err_flag, num_sms, s); break;
      case kEpiConv1: launch_pair<kEpiConv1>(ta, tb, tc, M, N, K, a_cols, ep, err_flag, num_sms, s); break;
      default: launch_pair<kEpiConv2>(ta, tb, tc, M, N, K, a_cols, ep, err_flag, num_sms, s); break;
    }
    return;
  }
  switch (epi) {
    case kEpiBias: launch_one<256, kEpiBias>(ta, tb, tc, M, N, K, a_cols, ep, err_flag, num_sms, s); break;
    case kEpiBiasGelu: launch_one<256, kEpiBiasGelu>(ta, tb, tc, M, N, K, a_cols, ep, err_flag, num_sms, s); break;
    case kEpiBiasResid: launch_one<256, kEpiBiasResid>(ta, tb, tc, M, N, K, a_cols, ep, err_flag, num_sms, s); break;
    case kEpiConv1: launch_one<256, kEpiConv1>(ta, tb, tc, M, N, K, a_cols, ep, err_flag, num_sms, s); break;
    default: launch_one<256, kEpiConv2>(ta, tb, tc, M, N, K, a_cols, ep, err_flag, num_sms, s); break;
  }
}

}  // namespace wf
