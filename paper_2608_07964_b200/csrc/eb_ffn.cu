// eb_expert_ffn_grouped: expert_i of Eq. 1 (bias-free SwiGLU MLP) for every (layer, expert) group
// of a step in one grouped pass on the 5th-generation tensor cores.
//
// Two persistent launches over a device-built tile list (ragged groups, no padding rows in memory):
//   gate/up : act[r, i] = silu(sum_h xp[r,h] Wg[i,h]) * (sum_h xp[r,h] Wu[i,h])      (bf16 out)
//   down    : yp[r, h]  = sum_i act[r,i] Wd[h,i]                                      (bf16 out)
//
// Both run ffn_kernel on CTA pairs (2-CTA clusters, one CTA per SM).  The WEIGHTS are the M operand of
// tcgen05.mma cta_group::2 (M = 256 weight rows, 128 per CTA) and the TOKEN rows of the tile are the N
// operand: N = the tile's rows rounded up to 16, at most 256.  Tensor-core work, shared-memory fill and
// TMEM columns of a tile therefore follow the rows it really holds - a group of 45 rows costs a 48-column
// tile, not a 128- or 256-row one - and a group is cut into ceil(rows / 256) tiles of nearly equal size.
// Every k-step issues two MMAs that share the token operand:
//   gate/up: W0 = 256 rows of W_gate, W1 = the same 256 rows of W_up.  The TMEM lane that holds gate
//            output i of a token holds up output i of that token, so SiLU * up fuses in registers
//            (256 outputs per tile);
//   down   : W0, W1 = two consecutive 256-row blocks of W_down (512 outputs per tile).
// Per CTA: warp 0 = TMA producer (its own 128 rows of W0 and W1 and its half of the token rows), warp 1 =
// MMA issuer (leader CTA only) and TMEM owner, warps 2..9 = epilogue.  A stage is 48 KB per CTA (W0 | W1 |
// up to 128 token rows of one 64-wide k-block, bf16, 128-byte swizzled K-major) for up to 1024 tensor-core
// cycles; four stages.  TMA completions of both CTAs count on the leader's barrier; the tcgen05.commit
// that frees a stage is delivered to both CTAs; no load is multicast.  The two accumulators fill TMEM
// (2 x 256 fp32 columns), so the epilogue of a tile does not overlap the next tile's MMAs; eight epilogue
// warps (two per TMEM lane quadrant, alternating 16-column chunks) keep that gap short and the producer
// keeps prefetching through it.  The accumulator holds outputs in lanes and tokens in columns: an
// epilogue warp transposes each 16-token chunk through 1 KB of shared memory and stores 16-byte vectors.
//
// Tiles: a device-built list (plan_kernel, fill_kernel).  Tiles of one group are weight-tile-major and
// token-tile-minor, so pairs working side by side share the weight tile in L2 and every weight byte leaves
// HBM once per group.  The D replicas of a shared expert (one group per virtual device, all reading the
// same matrix) are merged when all are small: their rows are packed into common tiles in slots of 16
// rows, so the matrix is streamed once per step instead of D times.  Groups are listed widest tiles
// first and the list is dealt out in rounds of alternating direction, which gives every pair nearly the
// same total cost without a dynamic scheduler.
//
// Every wait on an mbarrier is bounded: on expiry the kernel records EB_ERR_TIMEOUT in the
// context status word, lets copies in flight land, frees its TMEM and returns.
#include "eb_internal.cuh"

namespace {

constexpr int BK = 64;                                         // bf16 elements of one k-block (128 bytes)
constexpr int kStages = 4;
constexpr int kWBytes = 128 * BK * 2;                          // 128 weight rows of one k-block
constexpr int kTBytes = 128 * BK * 2;                          // up to 128 token rows of one k-block
constexpr int kStageBytes = 2 * kWBytes + kTBytes;             // W0 | W1 | token rows
constexpr int kRingBytes = kStages * kStageBytes;
constexpr int kEpiWarps = 8;
constexpr int kThreads = 64 + 32 * kEpiWarps;
constexpr size_t kSmemBytes = (size_t)kRingBytes + 1024 /*alignment slack*/ + 256 /*barriers*/ + kEpiWarps * 2048 /*transposes*/;
static_assert(kSmemBytes <= 232448, "shared memory of one CTA");
constexpr int kTmemCols = 512;
constexpr int kTileRows = 256;                                 // token rows of a tile at most
constexpr int kFeat1 = 256;                                    // outputs of a gate/up tile
constexpr int kFeat2 = 512;                                    // outputs of a down tile
constexpr int kSlotRows = 16;                                  // rows of one slot of a merged tile
constexpr int kMergeSlots = kTileRows / kSlotRows;             // slots of a merged tile at most
constexpr int kMergeMaxRows = 64;                              // replicas of a shared expert are merged when none has more rows
constexpr long long kSpinLimitCycles = 4000000000LL;

// ---- PTX wrappers ----------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: false if the limit expired or another thread of the CTA already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* s_abort, int* status,
                                          long long limit = kSpinLimitCycles) {
  if (mbar_try(bar, parity)) return true;
  const long long t0 = clock64();
  for (uint32_t spin = 1;; ++spin) {
    if (mbar_try(bar, parity)) return true;
    if ((spin & 63u) == 0u) {
      if (*s_abort) return false;
      if (clock64() - t0 > limit) {
        *s_abort = 1;
        atomicExch(status, (int)EB_ERR_TIMEOUT);
        return false;
      }
    }
  }
}

__device__ __forceinline__ void prefetch_tmap(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// shared::cluster address of the same offset in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA loads whose completion is counted on a barrier that may live in the peer CTA (the data goes to the
// issuing CTA only)
__device__ __forceinline__ void tma_pair_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void tma_pair_load_3d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t dst_smem, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t addr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(addr), "r"(cols) : "memory");
}
// D[tmem of both CTAs] (+)= A * B^T with M = 256 (128 rows of A per CTA), N from the descriptor (half of B per CTA), K = 16
__device__ __forceinline__ void umma_pair_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5, %5, %5, %5, %5}, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u)
      : "memory");
}
// arrives on the barrier at this offset in both CTAs of the pair once the MMAs issued so far are done
__device__ __forceinline__ void umma_pair_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar), "h"((uint16_t)3)
               : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }



__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory operand descriptor: K-major, 128-byte swizzle, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr) {
  return (uint64_t)((addr & 0x3FFFFu) >> 4) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor without its N field: fp32 accumulate, bf16 A and B, both K-major, M = 256.
constexpr uint32_t kIdescBase = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(256 >> 4) << 24);

// silu(g) * u with one special-function instruction: silu(g) = g / (1 + exp(-g)) = h + h tanh(h), h = g / 2.
// tanh.approx.f32 is good to about 2^-11 relative, well inside the bf16 rounding of the result.
__device__ __forceinline__ float silu_mul(uint32_t g_bits, uint32_t u_bits) {
  const float h = 0.5f * __uint_as_float(g_bits), u = __uint_as_float(u_bits);
  float t;
  asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(h));
  return fmaf(h, t, h) * u;
}

// Accumulator columns of a tile of `valid_rows` token rows: rounded up to 16 (each CTA of the pair supplies half
// of them, whole 8-row groups of the swizzled layout).
__device__ __forceinline__ int tile_cols(int valid_rows) {
  const int n = (valid_rows + 15) & ~15;
  return n > kTileRows ? kTileRows : n;
}
// Columns of a merged tile of n 16-row slots: an even number of slots, so that neither CTA's half cuts a slot.
__device__ __forceinline__ int merged_cols(int n_slots) { return ((n_slots + 1) & ~1) * kSlotRows; }
// Columns of a tile from its list entry (y = rows, or minus the slot count of a merged tile).
__device__ __forceinline__ int entry_cols(int y) { return y < 0 ? merged_cols(-y) : tile_cols(y); }

// ---- the grouped GEMM kernel -----------------------------------------------------------------
// PHASE 1: gate/up + SwiGLU (256 outputs per tile);  PHASE 2: down (512 outputs per tile).
// A tile is an int4 of the list: x = first row, y = rows (1..256), z = weight matrix, w = output tile.
// y < 0 marks a merged tile of -y slots of 16 rows each, described by slots[x ..): (first row, rows).
template <int PHASE>
__global__ void __launch_bounds__(kThreads, 1)
ffn_kernel(const __grid_constant__ CUtensorMap tmT128, const __grid_constant__ CUtensorMap tmT64,
           const __grid_constant__ CUtensorMap tmT32, const __grid_constant__ CUtensorMap tmT16,
           const __grid_constant__ CUtensorMap tmT8, const __grid_constant__ CUtensorMap tmW0, const __grid_constant__ CUtensorMap tmW1,
           const int4* __restrict__ work, const int2* __restrict__ slots, const int32_t* __restrict__ work_count,
           bf16* __restrict__ out, int ld_out, int n_out, int k_total, int* status) {
  EB_GRID_DEP_SYNC();
  constexpr int NS = kStages;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (base - raw);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kRingBytes);
  const uint32_t bar0 = base + (uint32_t)kRingBytes;
  auto w0_addr = [&](int s) { return base + s * kStageBytes; };
  auto w1_addr = [&](int s) { return base + s * kStageBytes + kWBytes; };
  auto t_addr = [&](int s) { return base + s * kStageBytes + 2 * kWBytes; };
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (NS + s); };
  const uint32_t tfull_bar = bar0 + 8u * (2 * NS), tempty_bar = bar0 + 8u * (2 * NS + 1);
  volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(bars + 2 * NS + 2);
  volatile int* s_abort = reinterpret_cast<volatile int*>(bars + 2 * NS + 3);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();   // CTA 0 of a pair is the leader
  if (threadIdx.x == 0) {
    for (int s = 0; s < NS; ++s) {
      mbar_init(full_bar(s), 1);    // the leader's arrive + all bytes of the stage of both CTAs
      mbar_init(empty_bar(s), 1);   // one tcgen05.commit (delivered to both CTAs)
    }
    mbar_init(tfull_bar, 1);                // one tcgen05.commit
    mbar_init(tempty_bar, 2 * kEpiWarps);   // one arrival per epilogue warp of both CTAs (leader's barrier)
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    prefetch_tmap(&tmT128);
    prefetch_tmap(&tmT64);
    prefetch_tmap(&tmT32);
    prefetch_tmap(&tmT16);
    prefetch_tmap(&tmT8);
    prefetch_tmap(&tmW0);
    prefetch_tmap(&tmW1);
  }
  if (warp == 1) {
    tmem_alloc_pair(smem_u32((const void*)s_tmem), kTmemCols);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();   // the peer's barriers are initialised before anything arrives on them
  tc_fence_after();
  const uint32_t tmem_base = *s_tmem;
  const int n_work = work_count[PHASE - 1];
  const int num_kb = (k_total + BK - 1) / BK;
  // The list is ordered by cost, widest tiles first.  It is dealt out in rounds of one tile per pair, the
  // direction alternating from round to round, so every pair ends up with nearly the same total cost.
  const int n_pairs = (int)(gridDim.x >> 1), my_pair = (int)(blockIdx.x >> 1);
  auto tile_of_round = [&](int r) { return r * n_pairs + ((r & 1) ? n_pairs - 1 - my_pair : my_pair); };

  if (warp == 0) {
    // ---------------- TMA producer (each CTA loads its own halves) ----------------
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      for (int r = 0; r * n_pairs < n_work; ++r) {
        const int w = tile_of_round(r);
        if (w >= n_work) continue;
        const int4 it = __ldg(work + w);
        const bool merged = it.y < 0;
        const int half = entry_cols(it.y) >> 1;   // token rows this CTA loads: a multiple of 8 (of 16 in a merged tile)
        const int tok0 = it.x + (int)rank * half;
        // merged tile: this CTA's slots are slots[x + rank * half / 16 ..); a slot beyond the tile's count
        // repeats the first one (its columns are never stored), so the byte count of a stage stays uniform
        int slot_row[kMergeSlots / 2];
#pragma unroll
        for (int i = 0; i < kMergeSlots / 2; ++i) {
          const int sl = (int)rank * (half / kSlotRows) + i;
          slot_row[i] = (merged && i < half / kSlotRows) ? __ldg(slots + it.x + (sl < -it.y ? sl : 0)).x : 0;
        }
        const int wrow0 = (PHASE == 1 ? it.w * kFeat1 : it.w * kFeat2) + (int)rank * 128;
        const int wrow1 = PHASE == 1 ? wrow0 : wrow0 + 256;
        const uint32_t tx = 2u * (2u * kWBytes + (uint32_t)half * (BK * 2));
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, s_abort, status)) goto done;
          // both CTAs' copies are counted on the leader's barrier; the leader announces the total
          const uint32_t fb = map_to_cta(full_bar(stage), 0);
          if (rank == 0) mbar_expect_tx(full_bar(stage), tx);
          tma_pair_load_3d(w0_addr(stage), &tmW0, kb * BK, wrow0, it.z, fb);
          tma_pair_load_3d(w1_addr(stage), &tmW1, kb * BK, wrow1, it.z, fb);
          const uint32_t ta = t_addr(stage);
          if (merged) {
#pragma unroll
            for (int i = 0; i < kMergeSlots / 2; ++i)
              if (i < half / kSlotRows) tma_pair_load_2d(ta + i * (kSlotRows * BK * 2), &tmT16, kb * BK, slot_row[i], fb);
          } else if (half == 128) {
            tma_pair_load_2d(ta, &tmT128, kb * BK, tok0, fb);
          } else {
            int r2 = 0;   // rows placed so far; every box starts on a multiple of 8 rows (1 KB), which keeps the swizzle phase
            if (half & 64) {
              tma_pair_load_2d(ta, &tmT64, kb * BK, tok0, fb);
              r2 = 64;
            }
            if (half & 32) {
              tma_pair_load_2d(ta + r2 * (BK * 2), &tmT32, kb * BK, tok0 + r2, fb);
              r2 += 32;
            }
            if (half & 16) {
              tma_pair_load_2d(ta + r2 * (BK * 2), &tmT16, kb * BK, tok0 + r2, fb);
              r2 += 16;
            }
            if (half & 8) tma_pair_load_2d(ta + r2 * (BK * 2), &tmT8, kb * BK, tok0 + r2, fb);
          }
          if (++stage == NS) {
            stage = 0;
            phase ^= 1u;
          }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer (leader CTA only) ----------------
    if (lane == 0 && rank == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int local = -1;
      for (int r = 0; r * n_pairs < n_work; ++r) {
        const int w = tile_of_round(r);
        if (w >= n_work) continue;
        ++local;
        const int4 it = __ldg(work + w);
        const uint32_t idesc = kIdescBase | ((uint32_t)(entry_cols(it.y) >> 3) << 17);
        if (!mbar_wait(tempty_bar, (uint32_t)(local & 1) ^ 1u, s_abort, status)) goto done;
        tc_fence_after();
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, s_abort, status)) goto done;
          tc_fence_after();
          const uint64_t d0 = smem_desc(w0_addr(stage)), d1 = smem_desc(w1_addr(stage)), dt = smem_desc(t_addr(stage));
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) {
            umma_pair_bf16(tmem_base, d0 + 2 * k, dt + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
            umma_pair_bf16(tmem_base + 256, d1 + 2 * k, dt + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
          }
          umma_pair_commit(empty_bar(stage));   // the stage is reusable in both CTAs once these MMAs have read it
          if (++stage == NS) {
            stage = 0;
            phase ^= 1u;
          }
        }
        umma_pair_commit(tfull_bar);   // both accumulators complete
      }
    }
  } else {
    // ---------------- epilogue warps ----------------
    const int q = warp & 3;                      // TMEM lane quadrant this warp may read
    const int chunk0 = ((warp - 2) >> 2) * 16;   // the two warps of a quadrant take alternate 16-column chunks
    const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
    bf16* tile = reinterpret_cast<bf16*>(smem + kRingBytes + 256) + (warp - 2) * 1024;   // 2 KB per epilogue warp
    int local = -1;
    for (int r = 0; r * n_pairs < n_work; ++r) {
      const int w = tile_of_round(r);
      if (w >= n_work) continue;
      ++local;
      const int4 it = __ldg(work + w);
      const bool merged = it.y < 0;
      const int n_cols = merged ? -it.y * kSlotRows : it.y;   // columns that may hold rows to store
      // one lane waits, the outcome is made warp-uniform before any .aligned instruction
      int ok = 1;
      if (lane == 0) ok = mbar_wait(tfull_bar, (uint32_t)(local & 1), s_abort, status) ? 1 : 0;
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) goto done;
      tc_fence_after();
      // this warp's 32 outputs start at fbase; a 16-token chunk is transposed through shared memory so that
      // global stores are 16-byte vectors: lane -> (token lane / 4 (+8), outputs 8 (lane % 4) .. +7)
      const int fbase = (PHASE == 1 ? it.w * kFeat1 : it.w * kFeat2) + (int)rank * 128 + q * 32;
      const int fcol = fbase + (lane & 3) * 8;
#pragma unroll 1
      for (int c0 = chunk0; c0 < n_cols; c0 += 32) {
        // rows of this chunk: columns c0 .. c0 + 15 are rows row0 .. row0 + n_here - 1 (a merged tile: one slot)
        int row0 = it.x + c0, n_here = min(16, it.y - c0);
        if (merged) {
          const int2 sl = __ldg(slots + it.x + (c0 >> 4));
          row0 = sl.x;
          n_here = sl.y;
        }
        uint32_t a[16], b[16];
        tmem_ld16(taddr + c0, a);
        tmem_ld16(taddr + 256 + c0, b);
        tmem_ld_wait();
        if (PHASE == 1) {
#pragma unroll
          for (int j = 0; j < 16; ++j) tile[j * 32 + lane] = __float2bfloat16_rn(silu_mul(a[j], b[j]));
        } else {
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            tile[j * 32 + lane] = __float2bfloat16_rn(__uint_as_float(a[j]));
            tile[512 + j * 32 + lane] = __float2bfloat16_rn(__uint_as_float(b[j]));
          }
        }
        __syncwarp();
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int tok = (lane >> 2) + 8 * h;
          if (tok < n_here) {
            bf16* dst = out + (size_t)(row0 + tok) * ld_out + fcol;
            const uint4* src = reinterpret_cast<const uint4*>(tile + tok * 32 + (lane & 3) * 8);
            if (fcol < n_out) *reinterpret_cast<uint4*>(dst) = src[0];
            if (PHASE == 2 && fcol + 256 < n_out) *reinterpret_cast<uint4*>(dst + 256) = src[64];   // second accumulator: +1 KB
          }
        }
        __syncwarp();
      }
      // all TMEM reads of this warp are complete (wait::ld above): hand the accumulators back
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(map_to_cta(tempty_bar, 0));
    }
  }

done:
  if (*s_abort) {
    // give copies and MMAs in flight time to land before shared memory and TMEM go away
    for (int i = 0; i < 200; ++i) __nanosleep(1000);
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();   // neither CTA leaves while its peer may still touch its memory or barriers
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, kTmemCols);
  }
}

// ---- self-test of the bounded wait ---------------------------------------------------------------
// One CTA waits on a barrier that nothing ever arrives on, with a short cycle limit, through the same
// wait routine the expert kernels use: the wait gives up, records EB_ERR_TIMEOUT and the kernel returns.
__global__ void bounded_wait_probe_kernel(long long limit_cycles, int* status, int* gave_up) {
  __shared__ uint64_t bar;
  __shared__ int s_abort;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    bool ok = mbar_wait(smem_u32(&bar), 0, &s_abort, status, limit_cycles);
    *gave_up = ok ? 0 : 1;
  }
}

// ---- tile list construction ------------------------------------------------------------------
// A group of `rows` rows is cut into ceil(rows / 256) tiles of nearly equal size, so no tile is a short
// remainder that would still stream a whole weight tile.
__device__ __forceinline__ int group_tiles(int rows) { return (rows + kTileRows - 1) / kTileRows; }
// Columns (token rows rounded up to 16) of the largest tile of a group; its cost class is that count in steps of 32.
__device__ __forceinline__ int group_cols(int rows) {
  const int t = group_tiles(rows);
  return t ? tile_cols((rows + t - 1) / t) : 0;
}

// Processing order of the groups.  The group table is device-major, so the D replicas of a shared
// expert (one group per virtual device, all reading the same weight matrix) lie far apart in it.
// Tiles are therefore listed in another order: first every routed group in table order, then the
// shared groups sorted by (layer, shared expert, device), so the replicas of one matrix are worked on
// side by side, share its tiles in L2 and the matrix leaves HBM once per step instead of D times.
// With a device filter (per-device timing) the device's own range is listed in table order.
__device__ __forceinline__ int group_at(const ModelParams& mp, const int* dev_off, int nl, int device, int g0, int i) {
  if (device >= 0) return g0 + i;
  const int routed = nl * mp.E;
  if (i < routed) {
    int d = 0;
    while (d + 1 < mp.D && i >= nl * dev_off[d + 1]) ++d;
    const int n_d = dev_off[d + 1] - dev_off[d];
    const int rel = i - nl * dev_off[d];
    return nl * (dev_off[d] + d * mp.S) + (rel / n_d) * (n_d + mp.S) + rel % n_d;
  }
  const int q = i - routed;
  const int lr = q / (mp.S * mp.D), s = (q / mp.D) % mp.S, d = q % mp.D;
  const int n_d = dev_off[d + 1] - dev_off[d];
  return nl * (dev_off[d] + d * mp.S) + lr * (n_d + mp.S) + n_d + s;
}

// The D replicas of a shared expert, when all are small, are packed into common tiles: the rows of each
// replica are cut into slots of 16 (one TMA box, one epilogue chunk), up to sixteen slots per tile, so the
// weight tile is fetched once for all of them.  `i` is a position of the processing order; returns true if
// it belongs to such a merged class and gives the class's first position and slot count.
__device__ __forceinline__ bool merged_class(const ModelParams& mp, const int* dev_off, int nl, int device, int i,
                                             const int32_t* __restrict__ group_off, int* head, int* n_slots) {
  if (device >= 0 || mp.S == 0 || mp.D < 2 || i < nl * mp.E) return false;
  const int q = i - nl * mp.E;
  const int h = i - q % mp.D;   // position of the class's replica on device 0
  int tot = 0, mx = 0;
  for (int d = 0; d < mp.D; ++d) {
    const int g = group_at(mp, dev_off, nl, device, 0, h + d);
    const int rows = group_off[g + 1] - group_off[g];
    tot += (rows + kSlotRows - 1) / kSlotRows;
    mx = rows > mx ? rows : mx;
  }
  *head = h;
  *n_slots = tot;
  return mx <= kMergeMaxRows;
}

// Cost classes of the tiles: class c holds the positions whose tiles have 32 c + 1 .. 32 (c + 1) columns.
constexpr int kClasses = kTileRows / 32;

// Block-wide exclusive scan (1024 threads) of one value per thread that belongs to one of kClasses classes:
// returns the sum of the values of the same class in the threads before this one, and adds every class's
// block total to total[].  A value packs two counters (low / high 32 bits).  Ends with a barrier.
__device__ __forceinline__ long long block_scan_by_class(int cls, long long v, long long (*s_warp)[kClasses],
                                                         long long* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  long long incl[kClasses];
#pragma unroll
  for (int c = 0; c < kClasses; ++c) incl[c] = c == cls ? v : 0;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
#pragma unroll
    for (int c = 0; c < kClasses; ++c) {
      const long long n = __shfl_up_sync(0xffffffffu, incl[c], o);
      if (lane >= o) incl[c] += n;
    }
  }
  if (lane == 31) {
#pragma unroll
    for (int c = 0; c < kClasses; ++c) s_warp[warp][c] = incl[c];
  }
  __syncthreads();
  if (warp == 0) {
#pragma unroll
    for (int c = 0; c < kClasses; ++c) {
      const long long wv = s_warp[lane][c];
      long long wi = wv;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const long long n = __shfl_up_sync(0xffffffffu, wi, o);
        if (lane >= o) wi += n;
      }
      s_warp[lane][c] = wi - wv;
      if (lane == 31) s_warp[32][c] = wi;
    }
  }
  __syncthreads();
  long long excl = 0;
#pragma unroll
  for (int c = 0; c < kClasses; ++c) {
    if (c == cls) excl = s_warp[warp][c] + incl[c] - v;
    total[c] += s_warp[32][c];
  }
  __syncthreads();
  return excl;
}

// plan: per position i of the processing order (requested group range), the group, its tile count and
// cost class; then the positions that own tiles are listed by cost class (widest tiles first, processing
// order inside a class) with the exclusive scan of their tile counts.  Widest-first order lets the
// expert kernel deal its tiles out in rounds of near-equal cost.  One scan carries all classes at once.
__global__ void __launch_bounds__(1024)
plan_kernel(ModelParams mp, const int32_t* __restrict__ group_off, const int32_t* __restrict__ step_meta, int device,
            int nt1, int nt2, int32_t* __restrict__ pgroup, int32_t* __restrict__ pslots, int4* __restrict__ prank,
            int32_t* __restrict__ order, int32_t* __restrict__ tile_pref, int32_t* __restrict__ work_count) {
  EB_GRID_DEP_SYNC();
  __shared__ long long s_warp[33][kClasses];
  __shared__ int s_dev_off[EB_MAX_D + 1];
  const int tid = threadIdx.x;
  if (tid <= mp.D) s_dev_off[tid] = mp.dev_off[tid];
  const int G = step_meta[1];
  const int g0 = device < 0 ? 0 : step_meta[3 + device];
  const int g1 = device < 0 ? G : step_meta[3 + device + 1];
  const int ng = g1 - g0;
  const int nl = step_meta[2];
  __syncthreads();
  // pass 1: tiles and class of every position; its rank and tile prefix inside its class
  long long total[kClasses];   // low 32 bits: positions of the class, high 32 bits: their tiles
#pragma unroll
  for (int c = 0; c < kClasses; ++c) total[c] = 0;
  int my_cls = -1;             // of the position this thread handled in the last chunk (the only one, as a rule)
  long long my_at = 0;
  for (int b = 0; b < ng; b += 1024) {
    const int i = b + tid;
    int tiles = 0, cols = 0;
    if (i < ng) {
      const int g = group_at(mp, s_dev_off, nl, device, g0, i);
      const int rows = group_off[g + 1] - group_off[g];
      int head, n_slots;
      pgroup[i] = g;
      pslots[i] = -1;
      if (merged_class(mp, s_dev_off, nl, device, i, group_off, &head, &n_slots)) {
        pslots[i] = n_slots;
        if (i == head && n_slots > 0) {   // the class's tiles sit at its first position
          tiles = (n_slots + kMergeSlots - 1) / kMergeSlots;
          cols = merged_cols(n_slots < kMergeSlots ? n_slots : kMergeSlots);
        }
      } else {
        tiles = group_tiles(rows);
        cols = group_cols(rows);
      }
    }
    const int cls = tiles > 0 ? (cols + 31) / 32 - 1 : -1;
    long long before[kClasses];
#pragma unroll
    for (int c = 0; c < kClasses; ++c) before[c] = total[c];
    const long long excl = block_scan_by_class(cls, tiles > 0 ? (1LL | ((long long)tiles << 32)) : 0, s_warp, total);
    my_cls = cls;
    my_at = 0;
#pragma unroll
    for (int c = 0; c < kClasses; ++c)
      if (c == cls) my_at = before[c] + excl;
    // more than one chunk of positions: parked until the class bases are known (read back by the same thread)
    if (ng > 1024 && i < ng) prank[i] = make_int4(cls, (int)(my_at & 0xffffffffLL), (int)(my_at >> 32), 0);
  }
  // class bases: widest class first
  long long base[kClasses];
  long long run = 0;
#pragma unroll
  for (int c = kClasses - 1; c >= 0; --c) {
    base[c] = run;
    run += total[c];
  }
  const int n_listed = (int)(run & 0xffffffffLL), nt = (int)(run >> 32);
  // pass 2: place every position that owns tiles
  for (int b = 0; b < ng; b += 1024) {
    const int i = b + tid;
    int cls = my_cls, rank = (int)(my_at & 0xffffffffLL), tpref = (int)(my_at >> 32);
    if (ng > 1024) {
      cls = -1;
      if (i < ng) {
        const int4 v = prank[i];
        cls = v.x;
        rank = v.y;
        tpref = v.z;
      }
    }
    if (cls >= 0) {
      long long b2 = 0;
#pragma unroll
      for (int c = 0; c < kClasses; ++c)
        if (c == cls) b2 = base[c];
      const int at = (int)(b2 & 0xffffffffLL) + rank;
      order[at] = i;
      tile_pref[at] = (int)(b2 >> 32) + tpref;
    }
  }
  if (tid == 0) {
    tile_pref[n_listed] = nt;
    work_count[0] = nt * nt1;
    work_count[1] = nt * nt2;
    work_count[2] = nt;
    work_count[3] = g0;
    work_count[4] = ng;
    work_count[5] = n_listed;
    work_count[8] = nl;
    work_count[9] = device;
  }
}

// fill: one thread per tile of the two lists (gate/up, down); tiles of a group are ordered weight-tile
// major, token-tile minor.
__global__ void __launch_bounds__(256)
fill_kernel(ModelParams mp, const int32_t* __restrict__ group_off, const int32_t* __restrict__ group_w,
            const int32_t* __restrict__ pgroup, const int32_t* __restrict__ pslots, const int32_t* __restrict__ order,
            const int32_t* __restrict__ tile_pref, const int32_t* __restrict__ work_count, int nt1, int nt2, int max1,
            int max2, int4* __restrict__ work1, int4* __restrict__ work2, int2* __restrict__ slots) {
  EB_GRID_DEP_SYNC();
  extern __shared__ int s_pref[];   // tile_pref staged once per block: the binary search below then stays on chip
  const int n_listed = work_count[5];
  const int cnt1 = work_count[0], total = cnt1 + work_count[1];
  if ((int)(blockIdx.x * blockDim.x) >= total) return;
  for (int i = threadIdx.x; i <= n_listed; i += blockDim.x) s_pref[i] = tile_pref[i];
  __syncthreads();
  for (int idx = blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += gridDim.x * blockDim.x) {
    const int list = idx >= cnt1 ? 1 : 0, local = idx - (list ? cnt1 : 0);
    const int nt = list ? nt2 : nt1;
    const int t_index = local / nt;
    // largest entry with tile_pref <= t_index (every listed position owns at least one tile)
    int lo = 0, hi = n_listed - 1;
    while (lo < hi) {
      int mid = (lo + hi + 1) >> 1;
      if (s_pref[mid] <= t_index) lo = mid; else hi = mid - 1;
    }
    const int t_g = s_pref[lo + 1] - s_pref[lo];
    const int rem = local - s_pref[lo] * nt;
    const int n = rem / t_g, m = rem % t_g;
    const int pos = order[lo], g = pgroup[pos], n_slots = pslots[pos];
    int4 it;
    if (n_slots >= 0) {
      // tile m of a merged class holds the next 16 slots of the class, replicas in device order
      const int base = kMergeSlots * (s_pref[lo] + m);
      const int first = kMergeSlots * m, n_here = min(kMergeSlots, n_slots - first);
      if (list == 0 && n == 0) {
        int c = 0;   // slots before the current replica
        for (int d = 0; d < mp.D; ++d) {
          const int gd = pgroup[pos + d];
          const int r0 = group_off[gd], rows = group_off[gd + 1] - r0;
          const int nc = (rows + kSlotRows - 1) / kSlotRows;
          for (int k = 0; k < nc; ++k, ++c)
            if (c >= first && c < first + n_here)
              slots[base + c - first] = make_int2(r0 + k * kSlotRows, min(kSlotRows, rows - k * kSlotRows));
        }
      }
      it.x = base;
      it.y = -n_here;
    } else {
      // t_g tiles of nearly equal size: the first (rows % t_g) tiles hold one row more
      const int rows = group_off[g + 1] - group_off[g];
      const int each = rows / t_g, more = rows % t_g;
      it.x = group_off[g] + m * each + min(m, more);
      it.y = each + (m < more ? 1 : 0);
    }
    it.z = group_w[g];
    it.w = n;
    if (local < (list ? max2 : max1)) (list ? work2 : work1)[local] = it;
  }
}

// ---- host side ---------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static const EncodeTiledFn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      p = nullptr;
    return (EncodeTiledFn)p;
  }();
  return fn;
}

// bf16 tensor [d2][d1][d0] (d0 innermost), box {b0, b1, 1}, 128-byte swizzle, zero fill out of bounds
bool make_map(CUtensorMap* m, const void* ptr, uint64_t d0, uint64_t d1, uint64_t d2, uint32_t b0, uint32_t b1) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[3] = {d0, d1, d2};
  cuuint64_t strides[2] = {d0 * 2, d0 * d1 * 2};
  cuuint32_t box[3] = {b0, b1, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  int rank = d2 > 0 ? 3 : 2;
  CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, rank, const_cast<void*>(ptr), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

template <int PHASE>
cudaError_t launch_ffn(eb_ctx* c, cudaStream_t st, const CUtensorMap* tT, const CUtensorMap& tW0, const CUtensorMap& tW1,
                       const int4* work, bf16* out, int ld_out, int n_out, int k_total) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(c->pair_grid);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = kSmemBytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  const int2* slots = c->slots;
  const int32_t* wc = c->work_count;
  ++g_ebi_launches;
  return cudaLaunchKernelEx(&cfg, ffn_kernel<PHASE>, tT[0], tT[1], tT[2], tT[3], tT[4], tW0, tW1, work, slots, wc, out, ld_out, n_out,
                            k_total, c->d_status);
}

}  // namespace

eb_status ebi_selftest_wait(eb_ctx* c, cudaStream_t st, long long limit_cycles, int* d_gave_up) {
  bounded_wait_probe_kernel<<<1, 32, 0, st>>>(limit_cycles, c->d_status, d_gave_up);
  EB_LAUNCH_CHECK(c, "bounded wait probe");
  return EB_OK;
}

eb_status ebi_ffn_bind(eb_ctx* c) {
  if (eb_status ds = ebi_check_device(c)) return ds;
  const eb_config& g = c->cfg;
  const uint64_t nw = (uint64_t)g.L * (g.E + g.S);
  // weight tiles: boxes of 128 rows x one k-block
  if (!make_map(&c->tm_gate, c->w_gate, g.H, g.I, nw, BK, 128) || !make_map(&c->tm_up, c->w_up, g.H, g.I, nw, BK, 128) ||
      !make_map(&c->tm_down, c->w_down, g.I, g.H, nw, BK, 128))
    return ebi_fail(c, EB_ERR_CUDA, "cuTensorMapEncodeTiled failed for the weights");
  // per context: function attributes and cluster occupancy belong to the current device
  cudaError_t e = cudaFuncSetAttribute(ffn_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(ffn_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
  if (e != cudaSuccess) return ebi_check_cuda(c, e, "cudaFuncSetAttribute");
  // how many 2-CTA clusters of this kernel the device can hold at once (one CTA per SM)
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * (c->num_sms / 2));
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = kSmemBytes;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int clusters = 0;
  e = cudaOccupancyMaxActiveClusters(&clusters, ffn_kernel<1>, &cfg);
  if (e != cudaSuccess || clusters < 1) {
    cudaGetLastError();
    return ebi_fail(c, EB_ERR_CUDA, "the device cannot hold a 2-CTA cluster of the expert kernel");
  }
  c->pair_grid = 2 * (clusters < c->num_sms / 2 ? clusters : c->num_sms / 2);
  return EB_OK;
}

eb_status ebi_ffn_run(eb_ctx* c, cudaStream_t st, const void* xp, const int32_t* group_off, const int32_t* group_w,
                      const int32_t* step_meta, void* yp, int32_t device) {
  if (!xp || !group_off || !group_w || !step_meta || !yp) return ebi_fail(c, EB_ERR_INVALID_ARG, "null pointer");
  if (eb_status ds = ebi_check_device(c)) return ds;
  if (!ebi_aligned16(xp) || !ebi_aligned16(yp)) return ebi_fail(c, EB_ERR_INVALID_ARG, "xp / yp must be 16-byte aligned");
  if (!c->w_gate) return ebi_fail(c, EB_ERR_INVALID_ARG, "weights not bound");
  if (!c->ws) return ebi_fail(c, EB_ERR_WORKSPACE, "no workspace set");
  const eb_config& g = c->cfg;
  const int rows = ebi_rows_cap(c);
  // token-row boxes of 128 / 64 / 32 / 16 / 8 rows x one k-block, over the permuted rows and over the intermediate
  CUtensorMap tok_x[5], tok_a[5];
  const int box_rows[5] = {128, 64, 32, 16, 8};
  for (int i = 0; i < 5; ++i)
    if (!make_map(&tok_x[i], xp, g.H, rows, 0, BK, box_rows[i]) || !make_map(&tok_a[i], c->act, g.I, rows, 0, BK, box_rows[i]))
      return ebi_fail(c, EB_ERR_CUDA, "cuTensorMapEncodeTiled failed for the activations");
  const int nt1 = (g.I + kFeat1 - 1) / kFeat1, nt2 = (g.H + kFeat2 - 1) / kFeat2;
  {
    KernelTimer timer(c, EBK_FFN_PLAN, st);
    ebi_launch(plan_kernel, dim3(1), dim3(1024), 0, st, c->mp, group_off, step_meta, (int)device, nt1, nt2, c->pgroup, c->pslots,
               c->prank, c->order, c->tile_pref, c->work_count);
  }
  {
    KernelTimer timer(c, EBK_FFN_FILL, st);
    ebi_launch(fill_kernel, dim3(c->num_sms), dim3(256), sizeof(int) * (size_t)(ebi_groups_cap(c) + 1), st, c->mp, group_off, group_w,
               (const int32_t*)c->pgroup,
               (const int32_t*)c->pslots, (const int32_t*)c->order, (const int32_t*)c->tile_pref,
               (const int32_t*)c->work_count, nt1, nt2, c->max_work1, c->max_work2, c->work1, c->work2, c->slots);
  }
  cudaError_t e;
  {
    KernelTimer timer(c, EBK_FFN_GATEUP, st);
    e = launch_ffn<1>(c, st, tok_x, c->tm_gate, c->tm_up, c->work1, c->act, g.I, g.I, g.H);
  }
  if (e == cudaSuccess) {
    KernelTimer timer(c, EBK_FFN_DOWN, st);
    e = launch_ffn<2>(c, st, tok_a, c->tm_down, c->tm_down, c->work2, (bf16*)yp, g.H, g.H, g.I);
  }
  if (e != cudaSuccess) return ebi_check_cuda(c, e, "expert_ffn launch");
  EB_LAUNCH_CHECK(c, "expert_ffn");
  return EB_OK;
}
