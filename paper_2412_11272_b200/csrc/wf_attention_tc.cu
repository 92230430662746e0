// Non-causal variable-length attention on the 5th-generation tensor cores (bf16, head dim 64).
//
// A persistent CTA (352 threads) walks a list of work items.  An item is two tiles of 128 query
// rows that run side by side: either 256 consecutive rows of one (sequence, head), which share
// every K / V stage, or -- for the odd last tile of a sequence -- the same 128 rows of two
// neighbouring heads, each tile with K / V stages of its own.  Keys are consumed 96 at a time.
// Roles:
//   warps 0-3 / 4-7  softmax for query tile 0 / 1, one thread per query row.  A step loads the
//                    96 scores of its row from tensor memory once, releases the score buffer,
//                    takes the row maximum, exponentiates and writes the probabilities back to
//                    tensor memory as packed bf16 (double-buffered).  The output row is
//                    accumulated by the tensor core in tensor memory across steps; probabilities
//                    are taken relative to a reference maximum that is only raised (and the
//                    accumulator rescaled, read-modify-write in tensor memory) when the true
//                    maximum exceeds it by more than 2^8 -- the final O / l does not depend on
//                    that choice.  After an item's first step the row maximum is not even
//                    computed unless the step's sum of probabilities shows that it is needed.
//                    In steady state the softmax never waits for the tensor pipe.
//   warp 8           one lane issues the TMA loads: Q tiles once per item, K and V tiles of 96
//                    keys through two rings of kKvStages stages.
//   warps 9, 10      MMA issue for query tile 0 / 1 (warp 9 also owns the tensor-memory
//                    allocation).  The whole warp runs the loop so that descriptors stay in
//                    uniform registers; one elected lane issues S = Q K^T (128x96x64, operands in
//                    shared memory) as soon as the softmax has read the previous scores, and
//                    O += P V (128x64x96, P from tensor memory, V from shared memory as an
//                    MN-major operand) when the probabilities are in place.  A K / V stage is
//                    released by two arrivals: one per tile when the tiles share it, both from
//                    the one tile that uses it otherwise.
// Keys are addressed through the token prefix sums: a key tile that runs past the end of its
// sequence is masked in the softmax, so no padded token ever contributes.
// Tensor-memory columns per query tile t (base 256 t): S [0,96) f32; P0 [96,144), P1 [144,192)
// packed bf16; O [192,256) f32.  Every mbarrier wait is bounded (wf_ptx.cuh).
#include <type_traits>

#include "wf_internal.h"
#include "wf_ptx.cuh"

namespace wf {

using namespace ptx;

namespace {

constexpr int kTQ = 128;          // query rows per tile
constexpr int kTK = 96;           // keys per step
constexpr int kPolyEvery = 4;  // every 4th pair of exponentials is evaluated on the FMA pipe (0: none)
constexpr int kKvStages = 4;
// When the two tiles of an item belong to different heads their stages alternate, tile t owning
// every second stage; with an even count each tile's stages are its own, so neither tile ever
// waits for the other (an odd count made them share stages and deadlock; three was tried).
// Same-pod A/B: four stages are 0.3-1.3 % faster than six, eight are 2-3 % slower.
static_assert(kKvStages >= 4 && kKvStages % 2 == 0, "K/V ring: even, at least four stages");
constexpr int kQBytes = kTQ * 64 * 2;      // 16 KB
constexpr int kKvBytes = kTK * 64 * 2;     // 12 KB
constexpr int kAttnThreads = 352;

// shared-memory map (offsets from a 1024-byte aligned base)
constexpr int kOffQ = 0;                                   // 2 tiles
constexpr int kOffK = kOffQ + 2 * kQBytes;
constexpr int kOffV = kOffK + kKvStages * kKvBytes;
constexpr int kOffBar = kOffV + kKvStages * kKvBytes;
// q_full, q_free | k_full, k_free, v_full, v_free per stage | per tile: s_full, s_free, p_full[2], o_full[2]
constexpr int kNumBars = 2 + 4 * kKvStages + 2 * 6;
constexpr int kAttnSmem = kOffBar + 8 * kNumBars + 16 + 1024;

__device__ __forceinline__ uint64_t umma_desc_mn_sw128(uint32_t smem_addr) {
  // rows are the K index (a key), the 64 contiguous elements of a row are the N index:
  // 8-row groups are 1024 B apart (stride byte offset); there is a single 64-wide N block.
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr >> 4) & 0x3FFF);
  d |= (uint64_t)1 << 16;
  d |= (uint64_t)(1024 >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

struct Item {
  int tok0, n, q0, q1, head, head1, n_kv;  // tile 1 covers rows q1.. of head1
  bool two;    // tile 1 has work
  bool split;  // the tiles belong to different heads: K / V stages alternate between them
};

// The work list holds (sequence, first query row | kind << 30, first item) triples in launch order;
// kind 0: 256 consecutive rows (both tiles non-empty), one item per head; kind 1: the odd last
// tile of a sequence, one item per pair of heads (a last unpaired head runs as a single tile);
// kind 2: one 128-row tile of one head (the planner's choice when that still gives no more items
// than there are SMs: half the work per CTA, and a lone tile's exponentials run faster).
// An entry of kind 1 directly follows the other entries of its sequence, so that its K / V tiles
// are still in the L2 when it runs.  Behind the triples sits one int per item: its entry.
__device__ __forceinline__ Item load_item(const int* __restrict__ meta, const MetaLayout& ml, int it, int n_head,
                                          int n_entries) {
  const int* wl = meta + ml.attn_work;
  const int lo = wl[3 * n_entries + it];  // the entry of every item follows the triples
  const int local = it - wl[3 * lo + 2];
  const int seq = wl[3 * lo], q0k = wl[3 * lo + 1];
  Item w;
  w.q0 = q0k & 0x3FFFFFFF;
  const unsigned kind = (unsigned)q0k >> 30;
  if (kind == 0 || kind == 2) {
    w.head = w.head1 = local;
    w.two = kind == 0;
    w.split = false;
  } else {
    w.head = 2 * local;
    w.two = w.split = w.head + 1 < n_head;
    w.head1 = w.two ? w.head + 1 : w.head;
  }
  w.q1 = w.split ? w.q0 : w.q0 + kTQ;
  w.tok0 = meta[ml.tok_off + seq];
  w.n = meta[ml.tok_off + seq + 1] - w.tok0;
  w.n_kv = (w.n + kTK - 1) / kTK;
  return w;
}

}  // namespace

__global__ void __launch_bounds__(kAttnThreads, 1) attention_tc_kernel(
    const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_kv,
    __nv_bfloat16* __restrict__ out, const int* __restrict__ meta, MetaLayout ml, int n_items, int n_entries,
    int n_head, int d_model, int* err_flag) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* sgen = smem_raw + (sbase - smem_u32(smem_raw));
  const uint32_t bars = sbase + kOffBar;
  const uint32_t q_full = bars, q_free = bars + 8;
  auto k_full = [&](int s) { return bars + 8u * (2 + s); };
  auto k_free = [&](int s) { return bars + 8u * (2 + kKvStages + s); };
  auto v_full = [&](int s) { return bars + 8u * (2 + 2 * kKvStages + s); };
  auto v_free = [&](int s) { return bars + 8u * (2 + 3 * kKvStages + s); };
  const uint32_t tile_bars = bars + 8u * (2 + 4 * kKvStages);
  auto s_full = [&](int t) { return tile_bars + 8u * (6 * t); };
  auto s_free = [&](int t) { return tile_bars + 8u * (6 * t + 1); };
  auto p_full = [&](int t, int b) { return tile_bars + 8u * (6 * t + 2 + b); };
  auto o_full = [&](int t, int b) { return tile_bars + 8u * (6 * t + 4 + b); };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(sgen + kOffBar + 8 * kNumBars);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(sgen + kOffBar + 8 * kNumBars + 8);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    mbar_init(q_full, 1);
    mbar_init(q_free, 2);
    for (int s = 0; s < kKvStages; ++s) {
      mbar_init(k_full(s), 1);
      mbar_init(k_free(s), 2);
      mbar_init(v_full(s), 1);
      mbar_init(v_free(s), 2);
    }
    for (int t = 0; t < 2; ++t) {
      mbar_init(s_full(t), 1);
      mbar_init(s_free(t), 128);
      for (int b = 0; b < 2; ++b) {
        mbar_init(p_full(t, b), 128);
        mbar_init(o_full(t, b), 1);
      }
    }
    *abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 9) {
    tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  griddep_wait();  // the set-up above overlapped the previous kernel's tail; qkv is read from here on
  griddep_launch_dependents();

  if (warp == 8) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      prefetch_tmap(&tmap_q);
      prefetch_tmap(&tmap_kv);
      uint32_t kc = 0, vc = 0, items = 0;
      bool ok = true;
      for (int it = blockIdx.x; ok && it < n_items; it += gridDim.x) {
        const Item w = load_item(meta, ml, it, n_head, n_entries);
        if (!mbar_wait(q_free, (items & 1u) ^ 1u, abort_flag)) { ok = false; break; }
        mbar_arrive_expect_tx(q_full, w.two ? 2 * kQBytes : kQBytes);
        tma_load_2d(sbase + kOffQ, &tmap_q, w.head * kHeadDim, w.tok0 + w.q0, q_full);
        if (w.two) tma_load_2d(sbase + kOffQ + kQBytes, &tmap_q, w.head1 * kHeadDim, w.tok0 + w.q1, q_full);
        const int n_h = w.split ? 2 : 1;  // K / V stages per key step
        for (int j = 0; ok && j < w.n_kv; ++j) {
          for (int h = 0; h < n_h; ++h) {
            const int s = kc % kKvStages;
            if (!mbar_wait(k_free(s), ((kc / kKvStages) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
            mbar_arrive_expect_tx(k_full(s), kKvBytes);
            tma_load_2d(sbase + kOffK + s * kKvBytes, &tmap_kv, d_model + (h ? w.head1 : w.head) * kHeadDim,
                        w.tok0 + j * kTK, k_full(s));
            ++kc;
          }
          for (int h = 0; ok && h < n_h; ++h) {
            const int s = vc % kKvStages;
            if (!mbar_wait(v_free(s), ((vc / kKvStages) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
            mbar_arrive_expect_tx(v_full(s), kKvBytes);
            tma_load_2d(sbase + kOffV + s * kKvBytes, &tmap_kv, 2 * d_model + (h ? w.head1 : w.head) * kHeadDim,
                        w.tok0 + j * kTK, v_full(s));
            ++vc;
          }
        }
        if (!ok) break;
        ++items;
      }
      if (!ok) {
        atomicExch(err_flag, 11);
        // bounded drain: give the copies already issued time to land
        for (uint32_t it2 = 0; it2 < (1u << 16); ++it2) {
          bool all = mbar_try_wait(q_full, (items & 1u));
          for (int s = 0; s < kKvStages; ++s) all = all && mbar_try_wait(k_full(s), 0) && mbar_try_wait(v_full(s), 0);
          if (all) break;
        }
      }
    }
  } else if (warp == 9 || warp == 10) {
    // ------------------------------------------------------------------ MMA issue for tile t
    const int t = warp - 9;
    constexpr uint32_t idesc_s = umma_idesc_bf16(kTQ, kTK, 0, 0);
    constexpr uint32_t idesc_o = umma_idesc_bf16(kTQ, kHeadDim, 0, 1);
    const bool leader = elect_one();
    const uint64_t qd = umma_desc_k_sw128(sbase + kOffQ + t * kQBytes);
    const uint64_t kd0 = umma_desc_k_sw128(sbase + kOffK);
    const uint64_t vd0 = umma_desc_mn_sw128(sbase + kOffV);
    const uint32_t tm_s = tmem_base + t * 256;
    uint32_t kc = 0, vc = 0, items = 0, g = 0;  // g: steps done; buffer = g & 1, parity = (g >> 1) & 1
    bool ok = true;
    // every lane waits; the verdict is made warp-uniform so that the warp never splits
    auto wait_all = [&](uint32_t bar, uint32_t parity) -> bool {
      return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag));
    };
    auto issue_s = [&](int ks) {
      if (leader) {
        const uint64_t kd = kd0 + (uint64_t)(ks * (kKvBytes >> 4));
        umma_bf16(tm_s, qd, kd, idesc_s, 0u);
        umma_bf16(tm_s, qd + 2, kd + 2, idesc_s, 1u);
        umma_bf16(tm_s, qd + 4, kd + 4, idesc_s, 1u);
        umma_bf16(tm_s, qd + 6, kd + 6, idesc_s, 1u);
        umma_commit(s_full(t));
      }
      __syncwarp();
    };
    for (int it = blockIdx.x; ok && it < n_items; it += gridDim.x) {
      const Item w = load_item(meta, ml, it, n_head, n_entries);
      if (t == 1 && !w.two) {
        // nothing to compute for this tile: release the stages in step with the other tile
        for (int j = 0; ok && j < w.n_kv; ++j) {
          int ks = kc % kKvStages;
          if (!wait_all(k_full(ks), (kc / kKvStages) & 1u)) { ok = false; break; }
          if (leader) mbar_arrive(k_free(ks));
          ++kc;
          int vs = vc % kKvStages;
          if (!wait_all(v_full(vs), (vc / kKvStages) & 1u)) { ok = false; break; }
          if (leader) mbar_arrive(v_free(vs));
          ++vc;
        }
        if (!ok) break;
        if (!wait_all(q_full, items & 1u)) { ok = false; break; }
        if (leader) mbar_arrive(q_free);
        ++items;
        continue;
      }
      if (!wait_all(q_full, items & 1u)) { ok = false; break; }
      // with split tiles the stages alternate: this tile's are the t-th of every pair, and it alone
      // gives both arrivals that release them
      const uint32_t own = w.split ? (uint32_t)t : 0u, adv = w.split ? 2u : 1u;
      auto release = [&](uint32_t bar) {
        if (leader) {
          umma_commit(bar);
          if (w.split) umma_commit(bar);
        }
      };
      int ks = (kc + own) % kKvStages;
      if (!wait_all(k_full(ks), ((kc + own) / kKvStages) & 1u)) { ok = false; break; }
      tc_fence_after();
      issue_s(ks);  // the score buffer is free: its last reader arrived on s_free (waited below)
      release(k_free(ks));
      kc += adv;
      for (int j = 0; j < w.n_kv; ++j) {
        if (!wait_all(s_free(t), g & 1u)) { ok = false; break; }
        if (j + 1 < w.n_kv) {
          ks = (kc + own) % kKvStages;
          if (!wait_all(k_full(ks), ((kc + own) / kKvStages) & 1u)) { ok = false; break; }
          tc_fence_after();
          issue_s(ks);
          release(k_free(ks));
          kc += adv;
        }
        const int vs = (vc + own) % kKvStages;
        if (!wait_all(v_full(vs), ((vc + own) / kKvStages) & 1u)) { ok = false; break; }
        const int k_steps = (min(kTK, w.n - j * kTK) + 15) >> 4;
        const uint32_t b = g & 1u;
        if (!wait_all(p_full(t, b), (g >> 1) & 1u)) { ok = false; break; }
        tc_fence_after();
        if (leader) {
          const uint64_t vd = vd0 + (uint64_t)(vs * (kKvBytes >> 4));
          const uint32_t tm_o = tm_s + 192, tm_p = tm_s + 96 + 48 * b;
          // 16 keys per instruction: 8 packed columns of P, 2048 B of V; the first instruction of
          // an item overwrites the accumulator, everything after adds to it
          umma_bf16_ts(tm_o, tm_p, vd, idesc_o, j > 0 ? 1u : 0u);
          if (k_steps > 1) umma_bf16_ts(tm_o, tm_p + 8, vd + 128, idesc_o, 1u);
          if (k_steps > 2) umma_bf16_ts(tm_o, tm_p + 16, vd + 256, idesc_o, 1u);
          if (k_steps > 3) umma_bf16_ts(tm_o, tm_p + 24, vd + 384, idesc_o, 1u);
          if (k_steps > 4) umma_bf16_ts(tm_o, tm_p + 32, vd + 512, idesc_o, 1u);
          if (k_steps > 5) umma_bf16_ts(tm_o, tm_p + 40, vd + 640, idesc_o, 1u);
          umma_commit(o_full(t, b));
        }
        release(v_free(vs));
        __syncwarp();
        vc += adv;
        ++g;
      }
      if (!ok) break;
      if (leader) umma_commit(q_free);
      ++items;
    }
    if (!ok && leader) atomicExch(err_flag, 12);
  } else if (warp < 8) {
    // ------------------------------------------------------------------ softmax, one row per thread
    const int t = warp >> 2;
    const int r = (warp & 3) * 32 + lane;
    const uint32_t lane_field = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t ta_s = tmem_base + lane_field + t * 256;
    const float scale = 0.125f * 1.4426950408889634f;  // 1/sqrt(64), base-2 exponent
    uint32_t g = 0;  // steps done by this tile (same counter as the MMA issuer's)
    bool ok = true;

    const uint32_t ta_o = ta_s + 192;
    constexpr float kRaise = 8.0f;  // the reference maximum is raised when exceeded by 2^8
    constexpr float kRaiseSum = 256.0f;  // a probability above 2^kRaise makes the step's sum exceed this
    auto wait_warp = [&](uint32_t bar, uint32_t parity) -> bool {
      return __all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag));
    };

    for (int it = blockIdx.x; ok && it < n_items; it += gridDim.x) {
      const Item w = load_item(meta, ml, it, n_head, n_entries);
      if (t == 1 && !w.two) continue;
      // a warp whose 32 rows all lie beyond the sequence keeps pace with the barriers only
      const int row0 = t ? w.q1 : w.q0;  // first query row of this tile
      const bool active = row0 + (warp & 3) * 32 < w.n;
      float m_ref = -INFINITY, l_run = 0.f;

      for (int j = 0; j < w.n_kv; ++j) {
        if (!wait_warp(s_full(t), g & 1u)) { ok = false; break; }
        tc_fence_after();
        const int kv_valid = min(kTK, w.n - j * kTK);
        uint32_t sv[kTK];
        if (active) {
          tmem_ld_32x32(ta_s, *reinterpret_cast<uint32_t(*)[32]>(&sv[0]));
          tmem_ld_32x32(ta_s + 32, *reinterpret_cast<uint32_t(*)[32]>(&sv[32]));
          tmem_ld_32x32(ta_s + 64, *reinterpret_cast<uint32_t(*)[32]>(&sv[64]));
          tmem_ld_wait();
        }
        tc_fence_before();
        mbar_arrive(s_free(t));  // the scores are in registers: the next S may overwrite them
        if (active) {
          auto row_max = [&]() -> float {
            float mx = -INFINITY;
            if (kv_valid == kTK) {
              // four independent chains: a single running maximum would serialise 48 dependent ops
              float m0 = -INFINITY, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;
#pragma unroll
              for (int i = 0; i < kTK; i += 8) {
                m0 = fmaxf(m0, fmaxf(__uint_as_float(sv[i]), __uint_as_float(sv[i + 1])));
                m1 = fmaxf(m1, fmaxf(__uint_as_float(sv[i + 2]), __uint_as_float(sv[i + 3])));
                m2 = fmaxf(m2, fmaxf(__uint_as_float(sv[i + 4]), __uint_as_float(sv[i + 5])));
                m3 = fmaxf(m3, fmaxf(__uint_as_float(sv[i + 6]), __uint_as_float(sv[i + 7])));
              }
              mx = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
            } else {
#pragma unroll
              for (int i = 0; i < kTK; ++i)
                if (i < kv_valid) mx = fmaxf(mx, __uint_as_float(sv[i]));
            }
            return mx * scale;  // finite: the first key of a step is always valid
          };
          if (j == 0) m_ref = row_max();
          // The probability buffer of this step was last read by the P V of two steps ago.  That
          // product was issued, by the same thread, before the S of this step, and the commit
          // behind S tracks every earlier MMA of that thread: having seen s_full, it has landed.
          float rs = 0.f, rs1 = 0.f;
          uint64_t acc2 = 0, acc2b = 0;  // two-wide running sums of the step's probabilities
          const uint32_t ta_p = ta_s + 96 + 48 * (g & 1u);
          const uint64_t scale2 = pack_f32x2(scale, scale);
          uint64_t nref2 = 0;  // (-m_ref, -m_ref), set at the start of exp_step
          // 32 keys: exponentials, row-sum contribution, packed bf16 probabilities to tensor memory
          // (the scaling and the sums go through two-wide float32 instructions: the loop is bound by
          // instruction issue next to the special-function unit)
          auto exp_chunk = [&](int h, auto masked_tag) {
            constexpr bool masked = decltype(masked_tag)::value;
            uint32_t pk[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              float a0, a1;
              unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(sv[32 * h + 2 * i]), __uint_as_float(sv[32 * h + 2 * i + 1])),
                                     scale2, nref2), a0, a1);
              float p0, p1;
              if (kPolyEvery > 0 && (i % kPolyEvery) == kPolyEvery - 1) {
                // 2^a on the FMA pipe for every kPolyEvery-th pair (the special-function unit is the
                // loop's limit): a = j + f with j the nearest integer (magic-number rounding) and
                // |f| <= 0.5, 2^f by a cubic (relative error 8e-5, far below bf16 rounding of the
                // probability), j added to the exponent bits.  -120 <= a <= 127 keeps the exponent in
                // range: a score far above the reference then gives 2^127 (not a wrapped exponent), which
                // drives the step's sum over the raise threshold exactly as the ex2 lanes' +inf does.
                const uint64_t ax = pack_f32x2(fminf(fmaxf(a0, -120.0f), 127.0f), fminf(fmaxf(a1, -120.0f), 127.0f));
                const uint64_t tt = add_f32x2(ax, pack_f32x2(12582912.0f, 12582912.0f));
                const uint64_t jj = add_f32x2(tt, pack_f32x2(-12582912.0f, -12582912.0f));
                const uint64_t ff = fma_f32x2(jj, pack_f32x2(-1.0f, -1.0f), ax);
                uint64_t pp = fma_f32x2(ff, pack_f32x2(0.05508868396282196f, 0.05508868396282196f),
                                        pack_f32x2(0.24260404706001282f, 0.24260404706001282f));
                pp = fma_f32x2(ff, pp, pack_f32x2(0.6932762265205383f, 0.6932762265205383f));
                pp = fma_f32x2(ff, pp, pack_f32x2(0.9999289512634277f, 0.9999289512634277f));
                float t0, t1, q0, q1;
                unpack_f32x2(tt, t0, t1);
                unpack_f32x2(pp, q0, q1);
                p0 = __uint_as_float(__float_as_uint(q0) + (__float_as_uint(t0) << 23));
                p1 = __uint_as_float(__float_as_uint(q1) + (__float_as_uint(t1) << 23));
              } else {
                p0 = ex2_approx(a0);
                p1 = ex2_approx(a1);
              }
              if (masked) {
                if (32 * h + 2 * i >= kv_valid) p0 = 0.f;
                if (32 * h + 2 * i + 1 >= kv_valid) p1 = 0.f;
              }
              if (i & 1) acc2b = add_f32x2(acc2b, pack_f32x2(p0, p1)); else acc2 = add_f32x2(acc2, pack_f32x2(p0, p1));
              __nv_bfloat162 v = __floats2bfloat162_rn(p0, p1);
              pk[i] = *reinterpret_cast<uint32_t*>(&v);
            }
            tmem_st_32x16(ta_p + 16 * h, pk);
          };
          auto exp_step = [&]() {
            acc2 = 0;
            acc2b = 0;
            nref2 = pack_f32x2(-m_ref, -m_ref);
            if (kv_valid == kTK) {
              exp_chunk(0, std::false_type{});
              exp_chunk(1, std::false_type{});
              exp_chunk(2, std::false_type{});
            } else {
              // ragged last step of a sequence: only the 32-key chunks that hold a valid key (the
              // P V product reads no probability column beyond them)
              exp_chunk(0, std::true_type{});
              if (kv_valid > 32) exp_chunk(1, std::true_type{});
              if (kv_valid > 64) exp_chunk(2, std::true_type{});
            }
            float s0, s1, s2, s3;
            unpack_f32x2(acc2, s0, s1);
            unpack_f32x2(acc2b, s2, s3);
            rs = s0 + s1;
            rs1 = s2 + s3;
          };
          // After the first step the probabilities are taken against the reference maximum as it
          // stands, without looking for the step's own maximum first.  A score more than 2^8 above
          // the reference shows in the step's sum of probabilities (> 2^8, while a step whose
          // maximum stays below the reference sums to at most 96): only then is the maximum taken,
          // the reference raised, the accumulator rescaled and the step's probabilities redone.
          exp_step();
          if (j > 0 && __any_sync(0xffffffffu, !(rs + rs1 <= kRaiseSum))) {
            const float m_tile = row_max();
            const bool raise = m_tile > m_ref + kRaise;
            if (__any_sync(0xffffffffu, raise)) {
              // rescale this warp's accumulator rows; needs the previous P V to have landed
              if (!wait_warp(o_full(t, (g - 1) & 1u), ((g - 1) >> 1) & 1u)) { ok = false; break; }
              tc_fence_after();
              const float corr = raise ? ex2_approx(m_ref - m_tile) : 1.0f;
              if (raise) { m_ref = m_tile; l_run *= corr; }
#pragma unroll
              for (int c = 0; c < 4; ++c) {
                uint32_t a[16];
                tmem_ld_32x16(ta_o + 16 * c, a);
                tmem_ld_wait();
#pragma unroll
                for (int i = 0; i < 16; ++i) a[i] = __float_as_uint(__uint_as_float(a[i]) * corr);
                tmem_st_32x16(ta_o + 16 * c, a);
              }
              tmem_st_wait();
              exp_step();  // lanes that did not raise reproduce what they had
            }
          }
          l_run += rs + rs1;
          tmem_st_wait();
        }
        tc_fence_before();
        mbar_arrive(p_full(t, g & 1u));
        ++g;
      }
      if (!ok) break;
      // drain the last two products (earlier phases of these barriers completed before the
      // s_full waits above returned, so the parities below are unambiguous)
      if (w.n_kv >= 2) {
        if (!wait_warp(o_full(t, (g - 2) & 1u), ((g - 2) >> 1) & 1u)) { ok = false; break; }
      }
      if (!wait_warp(o_full(t, (g - 1) & 1u), ((g - 1) >> 1) & 1u)) { ok = false; break; }
      tc_fence_after();
      const int q = row0 + r;
      if (active) {
        const float inv = 1.0f / l_run;
        __nv_bfloat16* dst = out + (long)(w.tok0 + q) * d_model + (t ? w.head1 : w.head) * kHeadDim;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint32_t a[16];
          tmem_ld_32x16(ta_o + 16 * c, a);
          tmem_ld_wait();
          if (q < w.n) {
#pragma unroll
            for (int gi = 0; gi < 2; ++gi) {
              __nv_bfloat162 p0 = __floats2bfloat162_rn(__uint_as_float(a[8 * gi + 0]) * inv, __uint_as_float(a[8 * gi + 1]) * inv);
              __nv_bfloat162 p1 = __floats2bfloat162_rn(__uint_as_float(a[8 * gi + 2]) * inv, __uint_as_float(a[8 * gi + 3]) * inv);
              __nv_bfloat162 p2 = __floats2bfloat162_rn(__uint_as_float(a[8 * gi + 4]) * inv, __uint_as_float(a[8 * gi + 5]) * inv);
              __nv_bfloat162 p3 = __floats2bfloat162_rn(__uint_as_float(a[8 * gi + 6]) * inv, __uint_as_float(a[8 * gi + 7]) * inv);
              uint4 u;
              u.x = *reinterpret_cast<uint32_t*>(&p0);
              u.y = *reinterpret_cast<uint32_t*>(&p1);
              u.z = *reinterpret_cast<uint32_t*>(&p2);
              u.w = *reinterpret_cast<uint32_t*>(&p3);
              *reinterpret_cast<uint4*>(dst + 16 * c + 8 * gi) = u;
            }
          }
        }
      }
      // the accumulator has been read: the next item's first P V may overwrite it
      tc_fence_before();
    }
    if (!ok && lane == 0) atomicExch(err_flag, 13);
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 9) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

cudaError_t attention_bf16_configure() {
  return cudaFuncSetAttribute(attention_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kAttnSmem);
}

void launch_attention_bf16(const CUtensorMap& tmap_q, const CUtensorMap& tmap_kv, __nv_bfloat16* out,
                           const int* meta, MetaLayout ml, int n_entries, int n_items, int d_model, int* err_flag,
                           int num_sms, bool pdl, cudaStream_t s) {
  if (n_items <= 0) return;
  const int n_head = d_model / kHeadDim;
  const int grid = n_items < num_sms ? n_items : num_sms;
  launch_dependent(attention_tc_kernel, dim3(grid), dim3(kAttnThreads), kAttnSmem, s, 1, pdl, tmap_q, tmap_kv, out, meta, ml,
                   n_items, n_entries, n_head, d_model, err_flag);
}

}  // namespace wf
