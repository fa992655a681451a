// eb_expert_ffn_grouped: expert_i of Eq. 1 (bias-free SwiGLU MLP) for every (layer, expert) group
// of a step in one grouped pass on the 5th-generation tensor cores.
//
// Two persistent launches over a device-built tile list (ragged groups, no padding rows in memory):
//   gate/up : act[r, i] = silu(sum_h xp[r,h] Wg[i,h]) * (sum_h xp[r,h] Wu[i,h])      (bf16 out)
//   down    : yp[r, h]  = sum_i act[r,i] Wd[h,i]                                      (bf16 out)
// A tile is 128 rows x 256 accumulator columns.  For gate/up the 256 columns are 128 gate rows
// and the matching 128 up rows of the weight matrices, loaded by two TMA copies into one
// contiguous K-major operand, so one tcgen05.mma feeds both and the epilogue fuses SiLU * up.
//
// Per CTA (one per SM): warp 0 = TMA producer, warp 1 = MMA issuer and TMEM owner,
// warps 2..5 = epilogue (TMEM -> registers -> bf16 -> global).  Shared memory holds a 4-stage ring of
// A tiles (128x64) and a 5-stage ring of B tiles (256x64), bf16 in the 128-byte swizzled K-major
// layout, each ring with its own barriers so the weight copies run one k-block further ahead; TMEM holds two
// 128x256 fp32 accumulators so the epilogue of tile i overlaps the MMAs of tile i+1.
// Tiles of one group are ordered weight-tile-major, so CTAs working side by side share the
// weight tile in L2 and every weight byte leaves HBM once per group; the replicas of a shared expert on
// the virtual devices are listed next to each other for the same reason.
// The small replicas of a shared expert are packed into common tiles (16- or 32-row slots, see the tile
// list construction below).  Groups with at most 32 rows load a 32-row A box (the tensor core still multiplies 128 rows,
// the extra rows are never stored), which keeps shared-memory fill traffic close to the weight
// bytes in the weight-streaming regime.
//
// Groups of more than 128 rows run on CTA pairs instead (ffn_swap_kernel, a 2-CTA cluster, described at
// its definition): there the weights are the M = 256 operand of tcgen05.mma cta_group::2 and the token rows
// are the N operand, so a ragged tile costs the rows it holds (rounded up to 32), not a full tile.
//
// Every wait on an mbarrier is bounded: on expiry the kernel records EB_ERR_TIMEOUT in the
// context status word, lets copies in flight land, frees its TMEM and returns.
#include "eb_internal.cuh"

namespace {

constexpr int BM = 128;
constexpr int BK = 64;
constexpr int BN = 256;
constexpr int kStagesA = 4;   // single-CTA kernel: ring of A tiles (token rows)
constexpr int kStagesB = 5;   // single-CTA kernel: ring of B tiles (weights): one deeper, they come from DRAM
constexpr int kSmallRows = 32;
constexpr int kSlotRows = 16;                  // rows of one slot of a merged tile
constexpr int kMergeSlots = BM / kSlotRows;    // slots of a merged tile
constexpr int kMergeMaxRows = 64;              // replicas of a shared expert are merged when none has more rows
constexpr int kABytes = BM * BK * 2;
constexpr int kASmallBytes = kSmallRows * BK * 2;
constexpr int kASlotBytes = kSlotRows * BK * 2;
constexpr int kBBytes = BN * BK * 2;
constexpr int kThreads = 192;
constexpr int kTmemCols = 512;
constexpr size_t kRingBytes = (size_t)kStagesA * kABytes + (size_t)kStagesB * kBBytes;
constexpr size_t kSmemBytes = kRingBytes + 1024 /*alignment slack*/ + 256 /*barriers*/;
static_assert(kSmemBytes <= 232448, "shared memory of one CTA");
constexpr long long kSpinLimitCycles = 4000000000LL;

// ---- PTX wrappers ----------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
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

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void prefetch_tmap(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

// ---- CTA-pair (cta_group::2) forms ------------------------------------------------------------
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
// D[tmem of both CTAs] (+)= A * B^T with M = 256 (128 rows per CTA), N = 256, K = 16
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

__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t addr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(addr), "r"(cols) : "memory");
}

// D[tmem] (+)= A[smem] * B[smem]^T, bf16 x bf16 -> fp32, M = 128, N = 256, K = 16
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// mbarrier arrives once all previously issued MMAs of this thread have completed
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

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
// Instruction descriptor: fp32 accumulate, bf16 A and B, both K-major, N = 256, M = 128.
constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);

__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ float silu_mul(uint32_t g_bits, uint32_t u_bits) {
  float g = __uint_as_float(g_bits), u = __uint_as_float(u_bits);
  return __fdividef(g, 1.0f + __expf(-g)) * u;
}
// Same value through one special-function instruction instead of two: silu(g) = h + h tanh(h), h = g / 2.
// tanh.approx.f32 is good to about 2^-11 relative, well inside the bf16 rounding of the result.
__device__ __forceinline__ float silu_mul_tanh(uint32_t g_bits, uint32_t u_bits) {
  const float h = 0.5f * __uint_as_float(g_bits), u = __uint_as_float(u_bits);
  float t;
  asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(h));
  return fmaf(h, t, h) * u;
}

// ---- the grouped GEMM kernel -----------------------------------------------------------------
// Groups of at most 128 rows, one CTA per 128-row tile.
// PHASE 1: gate/up + SwiGLU (output 128 columns per tile);  PHASE 2: down (output 256 columns per tile).
template <int PHASE>
__global__ void __launch_bounds__(kThreads, 1)
ffn_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmA_small,
           const __grid_constant__ CUtensorMap tmA_slot, const __grid_constant__ CUtensorMap tmB0, const __grid_constant__ CUtensorMap tmB1,
           const int4* __restrict__ work, const int2* __restrict__ slots, const int32_t* __restrict__ work_count,
           bf16* __restrict__ out, int ld_out, int n_out, int k_total, int* status) {
  EB_GRID_DEP_SYNC();
  // Two rings, kStagesA stages of A and kStagesB stages of B, each with its own full/empty barriers, so the
  // weight copies (DRAM latency) run one k-block further ahead than shared memory would allow with joint stages.
  constexpr int NA = kStagesA;
  constexpr int NB = kStagesB;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (base - raw);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kRingBytes);
  const uint32_t bar0 = base + (uint32_t)kRingBytes;
  auto a_addr = [&](int s) { return base + s * kABytes; };
  auto b_addr = [&](int s) { return base + kStagesA * kABytes + s * kBBytes; };
  // barriers: full_a[NA], empty_a[NA], full_b[NB], empty_b[NB], tmem_full[2], tmem_empty[2]
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (NA + s); };
  auto fullb_bar = [&](int s) { return bar0 + 8u * (2 * NA + s); };
  auto emptyb_bar = [&](int s) { return bar0 + 8u * (2 * NA + NB + s); };
  auto tfull_bar = [&](int a) { return bar0 + 8u * (2 * NA + 2 * NB + a); };
  auto tempty_bar = [&](int a) { return bar0 + 8u * (2 * NA + 2 * NB + 2 + a); };
  volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(bars + 2 * NA + 2 * NB + 4);
  volatile int* s_abort = reinterpret_cast<volatile int*>(bars + 2 * NA + 2 * NB + 5);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < NA; ++s) {
      mbar_init(full_bar(s), 1);    // producer's arrive + all bytes of the stage
      mbar_init(empty_bar(s), 1);   // one tcgen05.commit
    }
    for (int s = 0; s < NB; ++s) {
      mbar_init(fullb_bar(s), 1);
      mbar_init(emptyb_bar(s), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(tfull_bar(a), 1);                // one tcgen05.commit
      mbar_init(tempty_bar(a), 4);               // one arrival per epilogue warp
    }
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    prefetch_tmap(&tmA);
    prefetch_tmap(&tmA_small);
    prefetch_tmap(&tmA_slot);
    prefetch_tmap(&tmB0);
    if (PHASE == 1) prefetch_tmap(&tmB1);
  }
  if (warp == 1) {
    tmem_alloc(smem_u32((const void*)s_tmem), kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *s_tmem;
  const int n_work = work_count[PHASE - 1];
  const int num_kb = (k_total + BK - 1) / BK;
  const int w_first = (int)blockIdx.x, w_step = (int)gridDim.x;

  if (warp == 0) {
    // ---------------- TMA producer ----------------
    if (lane == 0) {
      int stage = 0, stage_b = 0;
      uint32_t phase = 0, phase_b = 0;
      for (int w = w_first; w < n_work; w += w_step) {
        // x = first row, y = valid rows, z = weight matrix, w = n tile; y < 0 marks a merged tile:
        // (-y & 15) slots of 16 rows each, or of 32 rows each if (-y & 16), described by slots[x ..)
        const int4 it = __ldg(work + w);
        const bool merged = it.y < 0;
        const int n_slots = merged ? ((-it.y) & 15) : 0;
        const bool big_slots = merged && ((-it.y) & 16);
        int slot_row[kMergeSlots];
#pragma unroll
        for (int i = 0; i < kMergeSlots; ++i) slot_row[i] = (merged && i < n_slots) ? __ldg(slots + it.x + i).x : 0;
        const bool small = !merged && it.y <= kSmallRows;
        const uint32_t tx_a = (uint32_t)(merged ? n_slots * (big_slots ? kASmallBytes : kASlotBytes) : small ? kASmallBytes : kABytes);
        // One specialised k loop per tile kind, so the issuing thread does the minimum between a stage
        // becoming free and its copies being in flight (that delay comes straight off the prefetch depth).
        // Single-CTA kernel: the weight copy of a k-block goes out first (it has the DRAM latency), then
        // the A copy once its own ring has room.
#define EB_B_STAGE()                                                                              \
  if (!mbar_wait(emptyb_bar(stage_b), phase_b ^ 1u, s_abort, status)) goto done;                  \
  {                                                                                               \
    const uint32_t sb = b_addr(stage_b);                                                          \
    mbar_expect_tx(fullb_bar(stage_b), kBBytes);                                                  \
    if (PHASE == 1) {                                                                             \
      tma_load_3d(sb, &tmB0, kb * BK, it.w * 128, it.z, fullb_bar(stage_b));                      \
      tma_load_3d(sb + kBBytes / 2, &tmB1, kb * BK, it.w * 128, it.z, fullb_bar(stage_b));        \
    } else {                                                                                      \
      tma_load_3d(sb, &tmB0, kb * BK, it.w * BN, it.z, fullb_bar(stage_b));                       \
    }                                                                                             \
    if (++stage_b == kStagesB) {                                                                  \
      stage_b = 0;                                                                                \
      phase_b ^= 1u;                                                                              \
    }                                                                                             \
  }
#define EB_A_STAGE_BEGIN()                                                            \
  if (!mbar_wait(empty_bar(stage), phase ^ 1u, s_abort, status)) goto done;           \
  const uint32_t sa = a_addr(stage);
#define EB_A_STAGE_END()    \
  if (++stage == NA) {      \
    stage = 0;              \
    phase ^= 1u;            \
  }
        if (!merged) {
          const CUtensorMap* amap = small ? &tmA_small : &tmA;
          for (int kb = 0; kb < num_kb; ++kb) {
            EB_B_STAGE();
            EB_A_STAGE_BEGIN();
            mbar_expect_tx(full_bar(stage), tx_a);
            tma_load_2d(sa, amap, kb * BK, it.x, full_bar(stage));
            EB_A_STAGE_END();
          }
        } else if (big_slots) {
          for (int kb = 0; kb < num_kb; ++kb) {
            EB_B_STAGE();
            EB_A_STAGE_BEGIN();
            mbar_expect_tx(full_bar(stage), tx_a);
#pragma unroll
            for (int i = 0; i < BM / kSmallRows; ++i)
              if (i < n_slots) tma_load_2d(sa + i * kASmallBytes, &tmA_small, kb * BK, slot_row[i], full_bar(stage));
            EB_A_STAGE_END();
          }
        } else {
          for (int kb = 0; kb < num_kb; ++kb) {
            EB_B_STAGE();
            EB_A_STAGE_BEGIN();
            mbar_expect_tx(full_bar(stage), tx_a);
#pragma unroll
            for (int i = 0; i < kMergeSlots; ++i)
              if (i < n_slots) tma_load_2d(sa + i * kASlotBytes, &tmA_slot, kb * BK, slot_row[i], full_bar(stage));
            EB_A_STAGE_END();
          }
        }
#undef EB_B_STAGE
#undef EB_A_STAGE_BEGIN
#undef EB_A_STAGE_END
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      int stage = 0, stage_b = 0;
      uint32_t phase = 0, phase_b = 0;
      int local = 0;
      for (int w = w_first; w < n_work; w += w_step, ++local) {
        const int as = local & 1;
        const uint32_t aphase = (local >> 1) & 1u;
        if (!mbar_wait(tempty_bar(as), aphase ^ 1u, s_abort, status)) goto done;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + as * BN;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, s_abort, status)) goto done;
          if (!mbar_wait(fullb_bar(stage_b), phase_b, s_abort, status)) goto done;
          tc_fence_after();
          const uint64_t da = smem_desc(a_addr(stage)), db = smem_desc(b_addr(stage_b));
#pragma unroll
          for (int k = 0; k < BK / 16; ++k) umma_bf16(d_tmem, da + 2 * k, db + 2 * k, kIdesc, (kb | k) != 0 ? 1u : 0u);
          // the stages are reusable once these MMAs have read them
          umma_commit(empty_bar(stage));
          umma_commit(emptyb_bar(stage_b));
          if (++stage_b == kStagesB) {
            stage_b = 0;
            phase_b ^= 1u;
          }
          if (++stage == NA) {
            stage = 0;
            phase ^= 1u;
          }
        }
        // accumulator complete
        umma_commit(tfull_bar(as));
      }
    }
  } else {
    // ---------------- epilogue warps ----------------
    const int q = warp & 3;  // TMEM lane quadrant this warp may read
    int local = 0;
    for (int w = w_first; w < n_work; w += w_step, ++local) {
      const int4 it = __ldg(work + w);
      const int as = local & 1;
      const uint32_t aphase = (local >> 1) & 1u;
      // one lane waits, the outcome is made warp-uniform before any .aligned instruction
      int ok = 1;
      if (lane == 0) ok = mbar_wait(tfull_bar(as), aphase, s_abort, status) ? 1 : 0;
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) goto done;
      tc_fence_after();
      int r = q * 32 + lane;                    // row inside the tile
      bool row_ok = r < it.y;
      int row_g = it.x + r;                     // row in the permuted order
      if (it.y < 0) {
        // merged tile: epilogue warp q owns slot q (32-row slots) or slots 2q and 2q+1 (16-row slots)
        row_ok = false;
        const int v = -it.y;
        const bool big = v & 16;
        const int slot = big ? q : 2 * q + (lane >> 4);
        const int local_row = big ? lane : (lane & 15);
        if (slot < (v & 15)) {
          const int2 sl = __ldg(slots + it.x + slot);
          row_g = sl.x + local_row;
          row_ok = local_row < sl.y;
        }
      }
      const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + as * BN;
      if (PHASE == 1) {
        bf16* dst = out + (size_t)row_g * ld_out + it.w * 128;
        const int n_left = n_out - it.w * 128;
#pragma unroll 1
        for (int c0 = 0; c0 < 128; c0 += 16) {
          uint32_t g[16], u[16];
          tmem_ld16(taddr + c0, g);
          tmem_ld16(taddr + 128 + c0, u);
          tmem_ld_wait();
          uint4 o0, o1;
          o0.x = pack_bf16(silu_mul(g[0], u[0]), silu_mul(g[1], u[1]));
          o0.y = pack_bf16(silu_mul(g[2], u[2]), silu_mul(g[3], u[3]));
          o0.z = pack_bf16(silu_mul(g[4], u[4]), silu_mul(g[5], u[5]));
          o0.w = pack_bf16(silu_mul(g[6], u[6]), silu_mul(g[7], u[7]));
          o1.x = pack_bf16(silu_mul(g[8], u[8]), silu_mul(g[9], u[9]));
          o1.y = pack_bf16(silu_mul(g[10], u[10]), silu_mul(g[11], u[11]));
          o1.z = pack_bf16(silu_mul(g[12], u[12]), silu_mul(g[13], u[13]));
          o1.w = pack_bf16(silu_mul(g[14], u[14]), silu_mul(g[15], u[15]));
          if (row_ok && c0 < n_left) *reinterpret_cast<uint4*>(dst + c0) = o0;
          if (row_ok && c0 + 8 < n_left) *reinterpret_cast<uint4*>(dst + c0 + 8) = o1;
        }
      } else {
        bf16* dst = out + (size_t)row_g * ld_out + it.w * BN;
        const int n_left = n_out - it.w * BN;
#pragma unroll 1
        for (int c0 = 0; c0 < BN; c0 += 32) {
          uint32_t a[16], b[16];
          tmem_ld16(taddr + c0, a);
          tmem_ld16(taddr + c0 + 16, b);
          tmem_ld_wait();
          uint4 o[4];
          o[0].x = pack_bf16(__uint_as_float(a[0]), __uint_as_float(a[1]));
          o[0].y = pack_bf16(__uint_as_float(a[2]), __uint_as_float(a[3]));
          o[0].z = pack_bf16(__uint_as_float(a[4]), __uint_as_float(a[5]));
          o[0].w = pack_bf16(__uint_as_float(a[6]), __uint_as_float(a[7]));
          o[1].x = pack_bf16(__uint_as_float(a[8]), __uint_as_float(a[9]));
          o[1].y = pack_bf16(__uint_as_float(a[10]), __uint_as_float(a[11]));
          o[1].z = pack_bf16(__uint_as_float(a[12]), __uint_as_float(a[13]));
          o[1].w = pack_bf16(__uint_as_float(a[14]), __uint_as_float(a[15]));
          o[2].x = pack_bf16(__uint_as_float(b[0]), __uint_as_float(b[1]));
          o[2].y = pack_bf16(__uint_as_float(b[2]), __uint_as_float(b[3]));
          o[2].z = pack_bf16(__uint_as_float(b[4]), __uint_as_float(b[5]));
          o[2].w = pack_bf16(__uint_as_float(b[6]), __uint_as_float(b[7]));
          o[3].x = pack_bf16(__uint_as_float(b[8]), __uint_as_float(b[9]));
          o[3].y = pack_bf16(__uint_as_float(b[10]), __uint_as_float(b[11]));
          o[3].z = pack_bf16(__uint_as_float(b[12]), __uint_as_float(b[13]));
          o[3].w = pack_bf16(__uint_as_float(b[14]), __uint_as_float(b[15]));
#pragma unroll
          for (int v = 0; v < 4; ++v)
            if (row_ok && c0 + 8 * v < n_left) *reinterpret_cast<uint4*>(dst + c0 + 8 * v) = o[v];
        }
      }
      // all TMEM reads of this warp are complete (wait::ld above): hand the accumulator back
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty_bar(as));
    }
  }

done:
  if (*s_abort) {
    // give copies and MMAs in flight time to land before shared memory and TMEM go away
    for (int i = 0; i < 200; ++i) __nanosleep(1000);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

// ---- CTA-pair kernel with the weights as the M operand ------------------------------------------
// Groups of more than 128 rows.  The pair's M = 256 rows are weight rows (128 per CTA) and the
// accumulator columns are token rows: N = the tile's valid rows rounded up to 32 (at most 256), so the
// tensor-core work of a ragged tile is what it holds, not a full 256-row tile.  Every k-step issues
// two MMAs that share the token operand:
//   gate/up: W0 = 256 rows of W_gate, W1 = the same 256 rows of W_up; the lane that holds gate output i
//            holds up output i of the same token, so SiLU * up fuses in registers (256 outputs per tile);
//   down   : W0, W1 = two consecutive 256-row blocks of W_down (512 outputs per tile).
// A stage is 48 KB per CTA (2 x 128 weight rows + up to 128 token rows of one k-block) for up to 1024
// tensor-core cycles: a quarter less shared-memory fill per flop than 256 x 256 tiles.  The two
// accumulators fill TMEM (2 x 256 columns), so the epilogue of a tile does not overlap the next tile's
// MMAs; eight epilogue warps (two per TMEM lane quadrant, alternating 16-column chunks) keep that gap
// short, and the producer keeps prefetching through it.  The accumulator holds outputs in lanes and
// tokens in columns: a warp stores 32 consecutive outputs of one token (64 bytes) per instruction.
constexpr int kSwStages = 4;
constexpr int kSwWBytes = 128 * BK * 2;                        // 128 weight rows of one k-block
constexpr int kSwStageBytes = 2 * kSwWBytes + kABytes;         // W0 | W1 | token rows
constexpr int kSwRingBytes = kSwStages * kSwStageBytes;
constexpr int kSwEpiWarps = 8;
constexpr size_t kSwSmemBytes = (size_t)kSwRingBytes + 1024 /*alignment slack*/ + 256 /*barriers*/ + kSwEpiWarps * 2048 /*transposes*/;
static_assert(kSwSmemBytes <= 232448, "shared memory of one CTA");
constexpr int kSwThreads = 64 + 32 * kSwEpiWarps;
constexpr int kSwTileRows = 256;                               // token rows of a tile at most
constexpr int kSwFeat1 = 256;                                  // outputs of a gate/up tile
constexpr int kSwFeat2 = 512;                                  // outputs of a down tile
constexpr uint32_t kIdescSwBase = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(256 >> 4) << 24);

__device__ __forceinline__ int sw_cols(int valid_rows) {
  const int n = (valid_rows + 31) & ~31;
  return n > kSwTileRows ? kSwTileRows : n;
}

template <int PHASE>
__global__ void __launch_bounds__(kSwThreads, 1)
ffn_swap_kernel(const __grid_constant__ CUtensorMap tmT128, const __grid_constant__ CUtensorMap tmT64,
                const __grid_constant__ CUtensorMap tmT32, const __grid_constant__ CUtensorMap tmT16,
                const __grid_constant__ CUtensorMap tmW0, const __grid_constant__ CUtensorMap tmW1,
                const int4* __restrict__ work, const int32_t* __restrict__ work_count, bf16* __restrict__ out,
                int ld_out, int n_out, int k_total, int* status) {
  EB_GRID_DEP_SYNC();
  constexpr int NS = kSwStages;
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* smem = smem_raw + (base - raw);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kSwRingBytes);
  const uint32_t bar0 = base + (uint32_t)kSwRingBytes;
  auto w0_addr = [&](int s) { return base + s * kSwStageBytes; };
  auto w1_addr = [&](int s) { return base + s * kSwStageBytes + kSwWBytes; };
  auto t_addr = [&](int s) { return base + s * kSwStageBytes + 2 * kSwWBytes; };
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
    mbar_init(tfull_bar, 1);                  // one tcgen05.commit
    mbar_init(tempty_bar, 2 * kSwEpiWarps);   // one arrival per epilogue warp of both CTAs (leader's barrier)
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    prefetch_tmap(&tmT128);
    prefetch_tmap(&tmT64);
    prefetch_tmap(&tmT32);
    prefetch_tmap(&tmT16);
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
  const int n_work = work_count[5 + PHASE - 1];
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
        const int4 it = __ldg(work + w);   // x = first row, y = valid rows, z = weight matrix, w = output tile
        const int half = sw_cols(it.y) >> 1;            // token rows this CTA loads: a multiple of 16
        const int tok0 = it.x + (int)rank * half;
        const int wrow0 = PHASE == 1 ? it.w * kSwFeat1 + (int)rank * 128 : it.w * kSwFeat2 + (int)rank * 128;
        const int wrow1 = PHASE == 1 ? wrow0 : wrow0 + 256;
        const uint32_t tx = 2u * (2u * kSwWBytes + (uint32_t)half * (BK * 2));
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, s_abort, status)) goto done;
          // both CTAs' copies are counted on the leader's barrier; the leader announces the total
          const uint32_t fb = map_to_cta(full_bar(stage), 0);
          if (rank == 0) mbar_expect_tx(full_bar(stage), tx);
          tma_pair_load_3d(w0_addr(stage), &tmW0, kb * BK, wrow0, it.z, fb);
          tma_pair_load_3d(w1_addr(stage), &tmW1, kb * BK, wrow1, it.z, fb);
          const uint32_t ta = t_addr(stage);
          if (half == 128) {
            tma_pair_load_2d(ta, &tmT128, kb * BK, tok0, fb);
          } else {
            int r = 0;   // rows placed so far; every box starts on a multiple of 16 rows (2 KB), which keeps the swizzle phase
            if (half & 64) {
              tma_pair_load_2d(ta, &tmT64, kb * BK, tok0, fb);
              r = 64;
            }
            if (half & 32) {
              tma_pair_load_2d(ta + r * (BK * 2), &tmT32, kb * BK, tok0 + r, fb);
              r += 32;
            }
            if (half & 16) tma_pair_load_2d(ta + r * (BK * 2), &tmT16, kb * BK, tok0 + r, fb);
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
        const uint32_t idesc = kIdescSwBase | ((uint32_t)(sw_cols(it.y) >> 3) << 17);
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
    const int q = warp & 3;                 // TMEM lane quadrant this warp may read
    const int chunk0 = ((warp - 2) >> 2) * 16;   // the two warps of a quadrant take alternate 16-column chunks
    const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16);
    bf16* tile = reinterpret_cast<bf16*>(smem + kSwRingBytes + 256) + (warp - 2) * 1024;   // 2 KB per epilogue warp
    int local = -1;
    for (int r = 0; r * n_pairs < n_work; ++r) {
      const int w = tile_of_round(r);
      if (w >= n_work) continue;
      ++local;
      const int4 it = __ldg(work + w);
      // one lane waits, the outcome is made warp-uniform before any .aligned instruction
      int ok = 1;
      if (lane == 0) ok = mbar_wait(tfull_bar, (uint32_t)(local & 1), s_abort, status) ? 1 : 0;
      ok = __shfl_sync(0xffffffffu, ok, 0);
      if (!ok) goto done;
      tc_fence_after();
      // this warp's 32 outputs start at fbase; a 16-token chunk is transposed through shared memory so that
      // global stores are 16-byte vectors: lane -> (token lane / 4 (+8), outputs 8 (lane % 4) .. +7)
      const int fbase = (PHASE == 1 ? it.w * kSwFeat1 : it.w * kSwFeat2) + (int)rank * 128 + q * 32;
      const int fcol = fbase + (lane & 3) * 8;
#pragma unroll 1
      for (int c0 = chunk0; c0 < it.y; c0 += 32) {
        uint32_t a[16], b[16];
        tmem_ld16(taddr + c0, a);
        tmem_ld16(taddr + 256 + c0, b);
        tmem_ld_wait();
        if (PHASE == 1) {
#pragma unroll
          for (int j = 0; j < 16; ++j) tile[j * 32 + lane] = __float2bfloat16_rn(silu_mul_tanh(a[j], b[j]));
        } else {
#pragma unroll
          for (int j = 0; j < 16; ++j) {
            tile[j * 32 + lane] = __float2bfloat16_rn(__uint_as_float(a[j]));
            tile[512 + j * 32 + lane] = __float2bfloat16_rn(__uint_as_float(b[j]));
          }
        }
        __syncwarp();
#pragma unroll
        for (int r = 0; r < 2; ++r) {
          const int tok = (lane >> 2) + 8 * r;
          if (c0 + tok < it.y) {
            bf16* dst = out + (size_t)(it.x + c0 + tok) * ld_out + fcol;
            const uint4* src = reinterpret_cast<const uint4*>(tile + tok * 32 + (lane & 3) * 8);
            if (fcol < n_out) *reinterpret_cast<uint4*>(dst) = src[0];
            if (PHASE == 2 && fcol + 256 < n_out) *reinterpret_cast<uint4*>(dst + 256) = src[64];   // second tile: +512 bf16
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
// A group runs either on single CTAs (128-row tiles: groups of at most 128 rows) or on CTA pairs (the
// kernel with the weights as the M operand: everything larger), never both, so its weights are streamed
// by one kernel only.  A pair group of `rows` rows is cut into ceil(rows / 256) tiles of nearly equal
// size, so no tile is a short remainder that would still stream a whole weight tile.
__device__ __forceinline__ bool group_uses_pairs(int rows) { return rows > BM; }
__device__ __forceinline__ int pair_tiles(int rows) { return (rows + kSwTileRows - 1) / kSwTileRows; }

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

// The D replicas of a shared expert, when all are small, are packed into common 128-row tiles: the rows
// of each replica are cut into chunks of 16 (one TMA box, half an epilogue warp), eight chunks per tile, so
// the weight tile is fetched once for all of them.  `i` is a position of the processing order; returns
// true if it belongs to such a merged class and gives the class's first position and chunk count.
__device__ __forceinline__ bool merged_class(const ModelParams& mp, const int* dev_off, int nl, int device, int i,
                                             const int32_t* __restrict__ group_off, int* head, int* chunks) {
  if (device >= 0 || mp.S == 0 || mp.D < 2 || i < nl * mp.E) return false;
  const int q = i - nl * mp.E;
  const int h = i - q % mp.D;   // position of the class's replica on device 0
  int tot16 = 0, tot32 = 0, mx = 0;
  for (int d = 0; d < mp.D; ++d) {
    const int g = group_at(mp, dev_off, nl, device, 0, h + d);
    const int rows = group_off[g + 1] - group_off[g];
    tot16 += (rows + kSlotRows - 1) / kSlotRows;
    tot32 += (rows + kSmallRows - 1) / kSmallRows;
    mx = rows > mx ? rows : mx;
  }
  *head = h;
  // 16-row slots (eight per tile) when every replica fits one, else 32-row slots (four per tile);
  // bit 30 of *chunks marks the larger slots
  *chunks = mx <= kSlotRows ? tot16 : (tot32 | (1 << 30));
  return mx <= kMergeMaxRows;
}

// Block-wide exclusive scan of one value per thread (1024 threads); returns the exclusive prefix and
// leaves the block total in *total.  Ends with a barrier, so s_warp may be reused right away.
__device__ __forceinline__ long long block_scan_excl(long long v, long long* s_warp, long long* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  long long incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    long long n = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += n;
  }
  if (lane == 31) s_warp[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    long long wv = s_warp[lane], wi = wv;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      long long n = __shfl_up_sync(0xffffffffu, wi, o);
      if (lane >= o) wi += n;
    }
    s_warp[lane] = wi - wv;
    if (lane == 31) s_warp[32] = wi;
  }
  __syncthreads();
  const long long excl = s_warp[warp] + incl - v;
  *total = s_warp[32];
  __syncthreads();
  return excl;
}

// Columns (token rows rounded up to 32) of the largest tile of a pair group: its cost class.
__device__ __forceinline__ int pair_group_cols(int rows) {
  const int t = pair_tiles(rows);
  return sw_cols((rows + t - 1) / t);
}

// plan: per group (in processing order) of the requested range, its number of 128-row tiles (single-CTA
// lists) with an exclusive scan; the pair groups (more than 128 rows) are listed separately, ordered by
// the cost of their tiles (widest first, table order inside a cost class), with the scan of their tile
// counts.  Widest-first order lets the pair kernel deal its tiles out in rounds of near-equal cost.
__global__ void __launch_bounds__(1024)
plan_kernel(ModelParams mp, const int32_t* __restrict__ group_off, const int32_t* __restrict__ step_meta, int device,
            int nt1, int nt2, int nt1p, int nt2p, int pair_mode, int32_t* __restrict__ mtile_pref,
            int32_t* __restrict__ ptile_pref, int32_t* __restrict__ pgroup, int32_t* __restrict__ ppgroup,
            int32_t* __restrict__ pchunks, int32_t* __restrict__ work_count) {
  EB_GRID_DEP_SYNC();
  __shared__ long long s_warp[33];
  __shared__ int s_dev_off[EB_MAX_D + 1];
  const int tid = threadIdx.x;
  if (tid <= mp.D) s_dev_off[tid] = mp.dev_off[tid];
  const int G = step_meta[1];
  const int g0 = device < 0 ? 0 : step_meta[3 + device];
  const int g1 = device < 0 ? G : step_meta[3 + device + 1];
  const int ng = g1 - g0;
  const int nl = step_meta[2];
  __syncthreads();
  long long carry = 0;      // single tiles so far
  int any_pairs = 0;
  for (int b = 0; b < ng; b += 1024) {
    const int i = b + tid;
    long long v = 0;
    int is_pair = 0;
    if (i < ng) {
      const int g = group_at(mp, s_dev_off, nl, device, g0, i);
      const int rows = group_off[g + 1] - group_off[g];
      int head, chunks;
      pgroup[i] = g;
      pchunks[i] = -1;
      if (merged_class(mp, s_dev_off, nl, device, i, group_off, &head, &chunks)) {
        const int per_tile = (chunks >> 30) ? BM / kSmallRows : kMergeSlots;
        v = i == head ? ((chunks & 0xffff) + per_tile - 1) / per_tile : 0;   // the class's tiles sit at its first position
        pchunks[i] = chunks;
      } else if (pair_mode && group_uses_pairs(rows)) {
        is_pair = 1;
      } else {
        v = (rows + BM - 1) / BM;
      }
    }
    long long total;
    const long long excl = block_scan_excl(v, s_warp, &total);
    if (i < ng) mtile_pref[i] = (int)(carry + excl);
    carry += total;
    any_pairs |= __syncthreads_or(is_pair);
  }
  long long pcarry = 0;   // low 32 bits: pair groups listed so far, high 32 bits: their tiles
  if (any_pairs) {
    for (int cols = kSwTileRows; cols >= 32; cols -= 32) {
      for (int b = 0; b < ng; b += 1024) {
        const int i = b + tid;
        long long v = 0;
        int g = 0;
        if (i < ng) {
          g = pgroup[i];
          const int rows = group_off[g + 1] - group_off[g];
          if (pchunks[i] < 0 && group_uses_pairs(rows) && pair_group_cols(rows) == cols)
            v = 1LL | ((long long)pair_tiles(rows) << 32);
        }
        if (!__syncthreads_or(v != 0)) continue;
        long long total;
        const long long excl = block_scan_excl(v, s_warp, &total);
        if (v) {
          const long long at = pcarry + excl;
          ppgroup[(int)(at & 0xffffffffLL)] = g;
          ptile_pref[(int)(at & 0xffffffffLL)] = (int)(at >> 32);
        }
        pcarry += total;
      }
    }
  }
  if (tid == 0) {
    const int mt = (int)carry, npg = (int)(pcarry & 0xffffffffLL), pt = (int)(pcarry >> 32);
    mtile_pref[ng] = mt;
    ptile_pref[npg] = pt;
    work_count[0] = mt * nt1;
    work_count[1] = mt * nt2;
    work_count[2] = mt;
    work_count[3] = g0;
    work_count[4] = ng;
    work_count[8] = nl;
    work_count[9] = device;
    work_count[5] = pt * nt1p;
    work_count[6] = pt * nt2p;
    work_count[7] = pt;
    work_count[10] = npg;
  }
}

// fill: one thread per tile of the four lists (single gate/up, single down, pair gate/up, pair down);
// tiles of a group are ordered weight-tile major, row-tile minor.
__global__ void __launch_bounds__(256)
fill_kernel(ModelParams mp, const int32_t* __restrict__ group_off, const int32_t* __restrict__ group_w,
            const int32_t* __restrict__ mtile_pref, const int32_t* __restrict__ ptile_pref,
            const int32_t* __restrict__ pgroup, const int32_t* __restrict__ ppgroup, const int32_t* __restrict__ pchunks,
            const int32_t* __restrict__ work_count, int nt1, int nt2, int nt1p, int nt2p, int max1, int max2,
            int maxp1, int maxp2,
            int4* __restrict__ work1, int4* __restrict__ work2, int4* __restrict__ work1p, int4* __restrict__ work2p,
            int2* __restrict__ slots) {
  EB_GRID_DEP_SYNC();
  const int ng = work_count[4], npg = work_count[10];
  const int cnt[4] = {work_count[0], work_count[1], work_count[5], work_count[6]};
  const int total = cnt[0] + cnt[1] + cnt[2] + cnt[3];
  for (int idx = blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += gridDim.x * blockDim.x) {
    int list = 0, local = idx;
    while (local >= cnt[list]) local -= cnt[list++];
    const bool pair = list >= 2;
    const int nt = pair ? ((list & 1) ? nt2p : nt1p) : ((list & 1) ? nt2 : nt1);
    const int32_t* pref = pair ? ptile_pref : mtile_pref;
    const int t_index = local / nt;
    // largest gi with pref[gi] <= t_index: groups without tiles in this list share their successor's
    // prefix, and a group that owns tiles has pref[gi + 1] > pref[gi]
    int lo = 0, hi = (pair ? npg : ng) - 1;
    while (lo < hi) {
      int mid = (lo + hi + 1) >> 1;
      if (pref[mid] <= t_index) lo = mid; else hi = mid - 1;
    }
    const int gi = lo;
    const int t_g = pref[gi + 1] - pref[gi];
    const int rem = local - pref[gi] * nt;
    const int n = rem / t_g, m = rem % t_g;
    const int g = pair ? ppgroup[gi] : pgroup[gi];
    int4 it;
    const int head = gi, chunks_raw = pair ? -1 : pchunks[gi];   // only the first position of a merged class owns tiles
    if (!pair && chunks_raw >= 0) {
      // tile m of a merged class holds the next 8 (16-row) or 4 (32-row) chunks of the class, replicas in
      // device order
      const bool big = (chunks_raw >> 30) & 1;
      const int chunks = chunks_raw & 0xffff;
      const int slot_rows = big ? kSmallRows : kSlotRows, per_tile = BM / slot_rows;
      const int base = kMergeSlots * (pref[gi] + m);
      const int first = per_tile * m, n_here = min(per_tile, chunks - first);
      if (list == 0 && n == 0) {
        int c = 0;   // chunks before the current replica
        for (int d = 0; d < mp.D; ++d) {
          const int gd = pgroup[head + d];
          const int r0 = group_off[gd], rows = group_off[gd + 1] - r0;
          const int nc = (rows + slot_rows - 1) / slot_rows;
          for (int k = 0; k < nc; ++k, ++c)
            if (c >= first && c < first + n_here)
              slots[base + c - first] = make_int2(r0 + k * slot_rows, min(slot_rows, rows - k * slot_rows));
        }
      }
      it.x = base;
      it.y = -(n_here | (big ? 16 : 0));
    } else if (pair) {
      // t_g tiles of nearly equal size: the first (rows % t_g) tiles hold one row more
      const int rows = group_off[g + 1] - group_off[g];
      const int each = rows / t_g, more = rows % t_g;
      it.x = group_off[g] + m * each + min(m, more);
      it.y = each + (m < more ? 1 : 0);
    } else {
      const int row0 = group_off[g] + m * BM;
      it.x = row0;
      it.y = min(BM, group_off[g + 1] - row0);
    }
    it.z = group_w[g];
    it.w = n;
    int4* dst = list == 0 ? work1 : list == 1 ? work2 : list == 2 ? work1p : work2p;
    const int cap = list == 0 ? max1 : list == 1 ? max2 : list == 2 ? maxp1 : maxp2;
    if (local < cap) dst[local] = it;
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
cudaError_t launch_ffn(eb_ctx* c, cudaStream_t st, const CUtensorMap& tA, const CUtensorMap& tAs, const CUtensorMap& tB0,
                       const CUtensorMap& tB1, const int4* work, bf16* out, int ld_out, int n_out, int k_total,
                       const CUtensorMap& tAslot) {
  const int2* slots = c->slots;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(c->num_sms);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = kSmemBytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 1;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  const int32_t* wc = c->work_count;
  ++g_ebi_launches;
  return cudaLaunchKernelEx(&cfg, ffn_kernel<PHASE>, tA, tAs, tAslot, tB0, tB1, work, slots, wc, out, ld_out, n_out, k_total,
                            c->d_status);
}

template <int PHASE>
cudaError_t launch_swap(eb_ctx* c, cudaStream_t st, const CUtensorMap* tT, const CUtensorMap& tW0, const CUtensorMap& tW1,
                        const int4* work, bf16* out, int ld_out, int n_out, int k_total) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(c->pair_grid);
  cfg.blockDim = dim3(kSwThreads);
  cfg.dynamicSmemBytes = kSwSmemBytes;
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
  const int32_t* wc = c->work_count;
  ++g_ebi_launches;
  return cudaLaunchKernelEx(&cfg, ffn_swap_kernel<PHASE>, tT[0], tT[1], tT[2], tT[3], tW0, tW1, work, wc, out, ld_out, n_out,
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
  if (!make_map(&c->tm_gate, c->w_gate, g.H, g.I, nw, BK, 128) ||
      !make_map(&c->tm_up, c->w_up, g.H, g.I, nw, BK, 128) ||
      !make_map(&c->tm_down, c->w_down, g.I, g.H, nw, BK, BN) ||
      !make_map(&c->tm_down_half, c->w_down, g.I, g.H, nw, BK, 128))
    return ebi_fail(c, EB_ERR_CUDA, "cuTensorMapEncodeTiled failed for the weights");
  int pair_grid = 0;
  {   // per context: function attributes and cluster occupancy belong to the current device
    cudaError_t e = cudaFuncSetAttribute(ffn_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(ffn_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(ffn_swap_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSwSmemBytes);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(ffn_swap_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSwSmemBytes);
    if (e != cudaSuccess) return ebi_check_cuda(c, e, "cudaFuncSetAttribute");
    // how many 2-CTA clusters of this kernel the device can hold at once (one CTA per SM)
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * (c->num_sms / 2));
    cfg.blockDim = dim3(kSwThreads);
    cfg.dynamicSmemBytes = kSwSmemBytes;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int clusters = 0;
    e = cudaOccupancyMaxActiveClusters(&clusters, ffn_swap_kernel<1>, &cfg);
    if (e != cudaSuccess || clusters < 1) {
      cudaGetLastError();
      clusters = 0;   // pairs unavailable: every group runs on single CTAs
    }
    pair_grid = 2 * (clusters < c->num_sms / 2 ? clusters : c->num_sms / 2);
  }
  c->pair_grid = pair_grid;
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
  CUtensorMap tm_x, tm_xs, tm_xl, tm_a, tm_as, tm_al, tm_x64, tm_a64;
  if (!make_map(&tm_x, xp, g.H, rows, 0, BK, BM) || !make_map(&tm_xs, xp, g.H, rows, 0, BK, kSmallRows) ||
      !make_map(&tm_xl, xp, g.H, rows, 0, BK, kSlotRows) || !make_map(&tm_a, c->act, g.I, rows, 0, BK, BM) ||
      !make_map(&tm_as, c->act, g.I, rows, 0, BK, kSmallRows) || !make_map(&tm_al, c->act, g.I, rows, 0, BK, kSlotRows) ||
      !make_map(&tm_x64, xp, g.H, rows, 0, BK, 64) || !make_map(&tm_a64, c->act, g.I, rows, 0, BK, 64))
    return ebi_fail(c, EB_ERR_CUDA, "cuTensorMapEncodeTiled failed for the activations");
  // token-row boxes of 128 / 64 / 32 / 16 rows for the pair kernel
  const CUtensorMap tok_x[4] = {tm_x, tm_x64, tm_xs, tm_xl}, tok_a[4] = {tm_a, tm_a64, tm_as, tm_al};
  const int nt1 = (g.I + 127) / 128, nt2 = (g.H + BN - 1) / BN;
  const int nt1p = (g.I + kSwFeat1 - 1) / kSwFeat1, nt2p = (g.H + kSwFeat2 - 1) / kSwFeat2;
  // CTA pairs only pay for groups of more than 128 rows; skip their launches when the permutation that
  // produced this step (same step_meta buffer) says no group can be that large
  bool pairs = c->pair_grid >= 2 && c->cfg.max_tokens > BM;
  if (pairs && c->hint_meta == step_meta && c->hint_max_group_rows >= 0 && c->hint_max_group_rows <= BM) pairs = false;
  {
    KernelTimer timer(c, EBK_FFN_PLAN, st);
    ebi_launch(plan_kernel, dim3(1), dim3(1024), 0, st, c->mp, group_off, step_meta, (int)device, nt1, nt2, nt1p, nt2p, pairs ? 1 : 0,
               c->mtile_pref, c->ptile_pref, c->pgroup, c->ppgroup, c->pchunks, c->work_count);
  }
  {
    KernelTimer timer(c, EBK_FFN_FILL, st);
    ebi_launch(fill_kernel, dim3(c->num_sms), dim3(256), 0, st, c->mp, group_off, group_w, (const int32_t*)c->mtile_pref,
               (const int32_t*)c->ptile_pref, (const int32_t*)c->pgroup, (const int32_t*)c->ppgroup, (const int32_t*)c->pchunks,
               (const int32_t*)c->work_count, nt1, nt2, nt1p, nt2p, c->max_work1, c->max_work2,
               c->max_work1p, c->max_work2p, c->work1, c->work2, c->work1p, c->work2p, c->slots);
  }
  cudaError_t e = cudaSuccess;
  if (pairs) {
    KernelTimer timer(c, EBK_FFN_GATEUP_PAIR, st);
    e = launch_swap<1>(c, st, tok_x, c->tm_gate, c->tm_up, c->work1p, c->act, g.I, g.I, g.H);
  }
  if (e == cudaSuccess) {
    KernelTimer timer(c, EBK_FFN_GATEUP, st);
    e = launch_ffn<1>(c, st, tm_x, tm_xs, c->tm_gate, c->tm_up, c->work1, c->act, g.I, g.I, g.H, tm_xl);
  }
  if (e == cudaSuccess && pairs) {
    KernelTimer timer(c, EBK_FFN_DOWN_PAIR, st);
    e = launch_swap<2>(c, st, tok_a, c->tm_down_half, c->tm_down_half, c->work2p, (bf16*)yp, g.H, g.H, g.I);
  }
  if (e == cudaSuccess) {
    KernelTimer timer(c, EBK_FFN_DOWN, st);
    e = launch_ffn<2>(c, st, tm_a, tm_as, c->tm_down, c->tm_down, c->work2, (bf16*)yp, g.H, g.H, g.I, tm_al);
  }
  if (e != cudaSuccess) return ebi_check_cuda(c, e, "expert_ffn launch");
  EB_LAUNCH_CHECK(c, "expert_ffn");
  return EB_OK;
}
