// eb_permute: dispatch on one GPU (Section 2.2) as a deterministic, stable counting sort of the
// (token, expert) assignments of the chosen micro-batches by (virtual device, layer, expert),
// followed by a 16-byte-vector gather of the token rows.
//
// Tokens are cut into chunks of <= 32 consecutive tokens of one micro-batch (one warp each).
//   hist   : per chunk, assignments per expert                     -> chunk_hist[chunk][E]
//   sizes  : per group, a warp scans the chunks of its layer in token order, leaving each
//            chunk's first rank inside the group                   -> chunk_base, group_size
//   scan   : exclusive prefix sum over groups                      -> group_off, group_w, step_meta
//   rank   : per chunk, ranks by warp match (in assignment order)  -> pos, row_src
//   gather : one warp per token reads the row once and writes it to its K + S rows.
// No order-dependent atomics anywhere: rows inside a group are in (micro-batch, token) order.
#include <cstring>

#include "eb_internal.cuh"

namespace {

constexpr int kWarps = 8;

struct StepShape {
  int nl;                       // active layers
  int act_layer[EB_MAX_MB];     // ascending
  int rank_of_mb[EB_MAX_MB];    // rank of the micro-batch's layer among active layers, -1 if not chosen
};

// first token (local index) of micro-batch of T tokens whose home device is >= d
__device__ __forceinline__ int home_start(int d, int T, int D) {
  if (T < (1 << 26)) return (int)(((unsigned)d * (unsigned)T + (unsigned)(D - 1)) / (unsigned)D);   // d <= 16: no overflow
  return (int)(((long long)d * T + D - 1) / D);
}
// home device of local token tl of a micro-batch of T tokens: floor(tl * D / T)
__device__ __forceinline__ int home_device(int tl, int T, int D) {
  if (T < (1 << 26)) return (int)(((unsigned)tl * (unsigned)D) / (unsigned)T);
  return (int)(((long long)tl * D) / T);
}

// Active layers of a step and every micro-batch's rank among them: threads 0..15 each place one
// micro-batch, the result lands in shared memory.  Ends with a block barrier.
__device__ __forceinline__ void step_shape_block(const BatchParams& bp, uint32_t run, StepShape* out) {
  const int j = threadIdx.x;
  if (j < 32) {   // warp 0; lanes 0..15 each own one micro-batch
    const bool sel = j < bp.n_mb && ((run >> j) & 1u);
    const int my_layer = j < bp.n_mb ? bp.layer[j] : -1;
    // is j the first chosen micro-batch sitting at its layer?
    bool first = sel;
    for (int i = 0; i < EB_MAX_MB; ++i) {
      const int li = __shfl_sync(0xffffffffu, my_layer, i);
      const bool si = (run >> i) & 1u;
      if (i < j && si && li == my_layer) first = false;
    }
    // distinct chosen layers below mine, and in total
    int below = 0, total = 0;
    for (int i = 0; i < EB_MAX_MB; ++i) {
      const int li = __shfl_sync(0xffffffffu, my_layer, i);
      const bool fi = __shfl_sync(0xffffffffu, (int)first, i) != 0;
      if (fi) {
        ++total;
        if (li < my_layer) ++below;
      }
    }
    if (j < EB_MAX_MB) {
      out->rank_of_mb[j] = sel ? below : -1;
      if (first) out->act_layer[below] = my_layer;
      if (j == 0) out->nl = total;
    }
  }
  __syncthreads();
}

// group id of (device d, active-layer rank lr, local slot) ; local slot < n_d + S
__device__ __forceinline__ int group_id(const int* dev_off, int S, int nl, int d, int lr, int local) {
  int n_d = dev_off[d + 1] - dev_off[d];
  return nl * (dev_off[d] + d * S) + lr * (n_d + S) + local;
}

__device__ __forceinline__ int mb_of_chunk(const BatchParams& bp, int c) {
  int j = 0;
  while (j + 1 < bp.n_mb && c >= bp.chunk_off[j + 1]) ++j;
  return j;
}

// ---- hist ----------------------------------------------------------------------------------
__global__ void __launch_bounds__(kWarps * 32)
hist_kernel(ModelParams mp, BatchParams bp, const eb_sched_result* __restrict__ res,
            const int32_t* __restrict__ topk_idx, int32_t* __restrict__ chunk_hist) {
  EB_GRID_DEP_SYNC();
  __shared__ int s_hist[kWarps][EB_MAX_E];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int c = blockIdx.x * kWarps + warp;
  if (c >= bp.n_chunks) return;
  const int E = mp.E, K = mp.K;
  const int j = mb_of_chunk(bp, c);
  const uint32_t run = res->run_mask;
  int* h = s_hist[warp];
  for (int e = lane; e < E; e += 32) h[e] = 0;
  __syncwarp();
  if ((run >> j) & 1u) {
    int t0 = bp.tok_off[j] + (c - bp.chunk_off[j]) * 32;
    int nt = min(32, bp.tok_off[j + 1] - t0);
    for (int a = lane; a < nt * K; a += 32) {
      const int e = topk_idx[(size_t)t0 * K + a];
      if ((unsigned)e < (unsigned)E) atomicAdd(&h[e], 1);   // an index outside [0, E) is skipped here and reported by rank
    }
  }
  __syncwarp();
  for (int e = lane; e < E; e += 32) chunk_hist[(size_t)c * E + e] = h[e];
}

// ---- sizes ---------------------------------------------------------------------------------
// One warp per group.  Routed group (d, lr, e): walks the chunks of the chosen micro-batches
// sitting at that layer in token order; writes the running count before each chunk and the total.
__global__ void __launch_bounds__(kWarps * 32)
sizes_kernel(ModelParams mp, BatchParams bp, const eb_sched_result* __restrict__ res,
             const int32_t* __restrict__ chunk_hist, int32_t* __restrict__ chunk_base,
             int32_t* __restrict__ group_size) {
  EB_GRID_DEP_SYNC();
  __shared__ int s_dev_off[EB_MAX_D + 1];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = blockIdx.x * kWarps + warp;
  const uint32_t run = res->run_mask;
  __shared__ StepShape ss;
  if (threadIdx.x <= mp.D) s_dev_off[threadIdx.x] = mp.dev_off[threadIdx.x];
  step_shape_block(bp, run, &ss);
  const int G = ss.nl * (mp.E + mp.D * mp.S);
  if (g >= G) return;
  // decode g -> (d, lr, local)
  int d = 0;
  while (d + 1 < mp.D && g >= ss.nl * (s_dev_off[d + 1] + (d + 1) * mp.S)) ++d;
  const int n_d = s_dev_off[d + 1] - s_dev_off[d];
  const int rel = g - ss.nl * (s_dev_off[d] + d * mp.S);
  const int lr = rel / (n_d + mp.S), local = rel % (n_d + mp.S);
  if (local >= n_d) {
    // shared expert: rows = chosen tokens at this layer whose home device is d (closed form)
    if (lane == 0) {
      int tot = 0;
      for (int j = 0; j < bp.n_mb; ++j)
        if (ss.rank_of_mb[j] == lr) {
          int T = bp.tok_off[j + 1] - bp.tok_off[j];
          tot += home_start(d + 1, T, mp.D) - home_start(d, T, mp.D);
        }
      group_size[g] = tot;
    }
    return;
  }
  const int e = mp.dev_list[s_dev_off[d] + local];
  int carry = 0;
  for (int j = 0; j < bp.n_mb; ++j) {
    if (ss.rank_of_mb[j] != lr) continue;
    for (int c0 = bp.chunk_off[j]; c0 < bp.chunk_off[j + 1]; c0 += 32) {
      int c = c0 + lane;
      int v = c < bp.chunk_off[j + 1] ? chunk_hist[(size_t)c * mp.E + e] : 0;
      int incl = v;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        int n = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += n;
      }
      if (c < bp.chunk_off[j + 1]) chunk_base[(size_t)c * mp.E + e] = carry + incl - v;
      carry += __shfl_sync(0xffffffffu, incl, 31);
    }
  }
  if (lane == 0) group_size[g] = carry;
}

// ---- scan ----------------------------------------------------------------------------------
__global__ void __launch_bounds__(1024)
scan_kernel(ModelParams mp, BatchParams bp, const eb_sched_result* __restrict__ res,
            const int32_t* __restrict__ group_size, int32_t* __restrict__ group_off,
            int32_t* __restrict__ group_w, int32_t* __restrict__ step_meta) {
  EB_GRID_DEP_SYNC();
  __shared__ int s_warp[32];
  __shared__ int s_carry;
  __shared__ int s_dev_off[EB_MAX_D + 1];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t run = res->run_mask;
  __shared__ StepShape ss;
  if (tid == 0) s_carry = 0;
  if (tid <= mp.D) s_dev_off[tid] = mp.dev_off[tid];
  step_shape_block(bp, run, &ss);
  const int G = ss.nl * (mp.E + mp.D * mp.S);
  for (int base = 0; base < G; base += 1024) {
    int g = base + tid;
    int v = g < G ? group_size[g] : 0;
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int n = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += n;
    }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    if (warp == 0) {
      int w = s_warp[lane], wi = w;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        int n = __shfl_up_sync(0xffffffffu, wi, o);
        if (lane >= o) wi += n;
      }
      s_warp[lane] = wi - w;  // exclusive offset of each warp
    }
    __syncthreads();
    int excl = s_carry + s_warp[warp] + incl - v;
    if (g < G) {
      group_off[g] = excl;
      // weight matrix of the group
      int d = 0;
      while (d + 1 < mp.D && g >= ss.nl * (s_dev_off[d + 1] + (d + 1) * mp.S)) ++d;
      int n_d = s_dev_off[d + 1] - s_dev_off[d];
      int rel = g - ss.nl * (s_dev_off[d] + d * mp.S);
      int lr = rel / (n_d + mp.S), local = rel % (n_d + mp.S);
      int slot = local < n_d ? mp.dev_list[s_dev_off[d] + local] : mp.E + (local - n_d);
      group_w[g] = ss.act_layer[lr] * (mp.E + mp.S) + slot;
    }
    __syncthreads();
    if (tid == 1023) s_carry = excl + v;
    __syncthreads();
  }
  if (tid == 0) {
    group_off[G] = s_carry;
    step_meta[0] = s_carry;
    step_meta[1] = G;
    step_meta[2] = ss.nl;
    for (int d = 0; d <= mp.D; ++d)
      step_meta[3 + d] = d < mp.D ? ss.nl * (s_dev_off[d] + d * mp.S) : G;
    for (int i = 4 + mp.D; i < EB_META_LEN; ++i) step_meta[i] = 0;
  }
}

// ---- rank ----------------------------------------------------------------------------------
__global__ void __launch_bounds__(kWarps * 32)
rank_kernel(ModelParams mp, BatchParams bp, const eb_sched_result* __restrict__ res,
            const int32_t* __restrict__ topk_idx, const int32_t* __restrict__ chunk_base,
            const int32_t* __restrict__ group_off, int32_t* __restrict__ pos, int32_t* __restrict__ row_src,
            int32_t* __restrict__ step_meta) {
  EB_GRID_DEP_SYNC();
  __shared__ int s_next[kWarps][EB_MAX_E];
  __shared__ int s_dev_off[EB_MAX_D + 1];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int c = blockIdx.x * kWarps + warp;
  const uint32_t run = res->run_mask;
  __shared__ StepShape ss;
  if (threadIdx.x <= mp.D) s_dev_off[threadIdx.x] = mp.dev_off[threadIdx.x];
  step_shape_block(bp, run, &ss);
  if (c >= bp.n_chunks) return;
  const int E = mp.E, K = mp.K, S = mp.S, KS = K + S;
  const int j = mb_of_chunk(bp, c);
  const int t0 = bp.tok_off[j] + (c - bp.chunk_off[j]) * 32;
  const int nt = min(32, bp.tok_off[j + 1] - t0);
  if (!((run >> j) & 1u)) {
    for (int a = lane; a < nt * KS; a += 32) pos[(size_t)t0 * KS + a] = -1;
    return;
  }
  const int lr = ss.rank_of_mb[j];
  int* next = s_next[warp];
  for (int e = lane; e < E; e += 32) {
    int d = mp.e2d[e];
    next[e] = group_off[group_id(s_dev_off, mp.S, ss.nl, d, lr, mp.e_local[e])] + chunk_base[(size_t)c * E + e];
  }
  __syncwarp();
  // routed slots, in assignment order a = t_local * K + k
  for (int a0 = 0; a0 < nt * K; a0 += 32) {
    int a = a0 + lane;
    bool valid = a < nt * K;
    int e = valid ? topk_idx[(size_t)t0 * K + a] : -1 - lane;  // distinct dummies never match
    if (valid && (unsigned)e >= (unsigned)E) {
      // routing index outside [0, E) (only possible with tables not written by eb_route): never used as an
      // index; the slot gets no row and the step's meta data counts it
      pos[(size_t)(t0 + a / K) * KS + a % K] = -1;
      atomicAdd(&step_meta[EB_META_LEN - 1], 1);
      valid = false;
      e = -1 - lane;
    }
    unsigned peers = __match_any_sync(0xffffffffu, e);
    int before = __popc(peers & ((1u << lane) - 1u));
    int p = 0;
    if (valid) {
      p = next[e] + before;
      int t = t0 + a / K, k = a % K;
      pos[(size_t)t * KS + k] = p;
      row_src[p] = t;
    }
    __syncwarp();
    if (valid && before == 0) next[e] += __popc(peers);
    __syncwarp();
  }
  // shared slots: closed-form rows
  if (S > 0 && lane < nt) {
    const int T = bp.tok_off[j + 1] - bp.tok_off[j];
    const int tl = t0 + lane - bp.tok_off[j];
    const int d = home_device(tl, T, mp.D);
    int before = 0;
    for (int j2 = 0; j2 < j; ++j2)
      if (ss.rank_of_mb[j2] == lr) {
        int T2 = bp.tok_off[j2 + 1] - bp.tok_off[j2];
        before += home_start(d + 1, T2, mp.D) - home_start(d, T2, mp.D);
      }
    const int n_d = s_dev_off[d + 1] - s_dev_off[d];
    for (int s = 0; s < S; ++s) {
      int p = group_off[group_id(s_dev_off, mp.S, ss.nl, d, lr, n_d + s)] + before + (tl - home_start(d, T, mp.D));
      pos[(size_t)(t0 + lane) * KS + K + s] = p;
      row_src[p] = t0 + lane;
    }
  }
}

// ---- fused kernel for small steps --------------------------------------------------------------
// hist + sizes + scan + rank in one block when the step has at most kFusedMaxChunks chunks and
// kFusedMaxGroups group slots: the routing decisions and the per-chunk tables live in shared memory and three kernel boundaries
// disappear (these kernels are pure latency on small steps).  Same arithmetic, same results.
constexpr int kFusedMaxChunks = 32;
constexpr int kFusedMaxGroups = 4096;
constexpr int kFusedThreads = 1024;

__global__ void __launch_bounds__(kFusedThreads)
permute_fused_kernel(ModelParams mp, BatchParams bp, const eb_sched_result* __restrict__ res,
                     const int32_t* __restrict__ topk_idx, int32_t* __restrict__ group_off,
                     int32_t* __restrict__ group_w, int32_t* __restrict__ pos, int32_t* __restrict__ row_src,
                     int32_t* __restrict__ step_meta) {
  EB_GRID_DEP_SYNC();
  extern __shared__ int s_dyn[];
  __shared__ int s_dev_off[EB_MAX_D + 1];
  __shared__ int s_warp[32];
  __shared__ int s_carry;
  const int E = mp.E, K = mp.K, S = mp.S, KS = K + S, D = mp.D;
  __shared__ int s_e2d[EB_MAX_E], s_e_local[EB_MAX_E], s_dev_list[EB_MAX_E];
  int* s_topk = s_dyn;                         // [n_tok][K]: the routing decisions
  int* s_tab = s_topk + bp.n_tok * K;          // [n_chunks][E]: histogram, then first rank of the chunk in its group
  int* s_goff = s_tab + bp.n_chunks * E;       // [G + 1]: group sizes, then offsets
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // every global read of the kernel is issued here, together: the phases below are chains of block barriers
  // and would otherwise each pay a trip to memory
  const uint32_t run = res->run_mask;
  for (int i = tid; i < bp.n_tok * K; i += kFusedThreads) s_topk[i] = topk_idx[i];
  for (int e = tid; e < E; e += kFusedThreads) {
    s_e2d[e] = mp.e2d[e];
    s_e_local[e] = mp.e_local[e];
    s_dev_list[e] = mp.dev_list[e];
  }
  __shared__ StepShape ss;
  __shared__ int s_home[EB_MAX_MB][EB_MAX_D + 1];   // first local token of every home device, per micro-batch
  if (tid == 0) s_carry = 0;
  if (tid <= D) s_dev_off[tid] = mp.dev_off[tid];
  if (tid < EB_MAX_MB * (EB_MAX_D + 1)) {
    const int j = tid / (EB_MAX_D + 1), d = tid % (EB_MAX_D + 1);
    if (j < bp.n_mb && d <= D) s_home[j][d] = home_start(d, bp.tok_off[j + 1] - bp.tok_off[j], D);
  }
  step_shape_block(bp, run, &ss);
  const int G = ss.nl * (E + D * S);

  // ---- histogram per chunk (one warp each)
  for (int c = warp; c < bp.n_chunks; c += kFusedThreads / 32) {
    int* h = s_tab + c * E;
    for (int e = lane; e < E; e += 32) h[e] = 0;
    __syncwarp();
    const int j = mb_of_chunk(bp, c);
    if ((run >> j) & 1u) {
      const int t0 = bp.tok_off[j] + (c - bp.chunk_off[j]) * 32;
      const int nt = min(32, bp.tok_off[j + 1] - t0);
      for (int a = lane; a < nt * K; a += 32) {
        const int e = s_topk[t0 * K + a];
        if ((unsigned)e < (unsigned)E) atomicAdd(&h[e], 1);
      }
    }
  }
  __syncthreads();

  // ---- group sizes; the chunk table turns into "rows of the group before this chunk"
  for (int g = tid; g < G; g += kFusedThreads) {
    int d = 0;
    while (d + 1 < D && g >= ss.nl * (s_dev_off[d + 1] + (d + 1) * S)) ++d;
    const int n_d = s_dev_off[d + 1] - s_dev_off[d];
    const int rel = g - ss.nl * (s_dev_off[d] + d * S);
    const int lr = rel / (n_d + S), local = rel % (n_d + S);
    int tot = 0;
    if (local >= n_d) {
      for (int j = 0; j < bp.n_mb; ++j)
        if (ss.rank_of_mb[j] == lr) tot += s_home[j][d + 1] - s_home[j][d];
    } else {
      const int e = s_dev_list[s_dev_off[d] + local];
      for (int j = 0; j < bp.n_mb; ++j) {
        if (ss.rank_of_mb[j] != lr) continue;
        for (int c = bp.chunk_off[j]; c < bp.chunk_off[j + 1]; ++c) {
          const int v = s_tab[c * E + e];
          s_tab[c * E + e] = tot;
          tot += v;
        }
      }
    }
    s_goff[g] = tot;
  }
  __syncthreads();

  // ---- exclusive scan over groups, weight matrix of every group, step_meta
  for (int base = 0; base < G; base += kFusedThreads) {
    const int g = base + tid;
    const int v = g < G ? s_goff[g] : 0;
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int n = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += n;
    }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    if (warp == 0) {
      int w = s_warp[lane], wi = w;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        int n = __shfl_up_sync(0xffffffffu, wi, o);
        if (lane >= o) wi += n;
      }
      s_warp[lane] = wi - w;
    }
    __syncthreads();
    const int excl = s_carry + s_warp[warp] + incl - v;
    if (g < G) {
      s_goff[g] = excl;
      group_off[g] = excl;
      int d = 0;
      while (d + 1 < D && g >= ss.nl * (s_dev_off[d + 1] + (d + 1) * S)) ++d;
      const int n_d = s_dev_off[d + 1] - s_dev_off[d];
      const int rel = g - ss.nl * (s_dev_off[d] + d * S);
      const int lr = rel / (n_d + S), local = rel % (n_d + S);
      const int slot = local < n_d ? s_dev_list[s_dev_off[d] + local] : E + (local - n_d);
      group_w[g] = ss.act_layer[lr] * (E + S) + slot;
    }
    __syncthreads();
    if (tid == kFusedThreads - 1) s_carry = excl + v;
    __syncthreads();
  }
  if (tid == 0) {
    s_goff[G] = s_carry;
    group_off[G] = s_carry;
    step_meta[0] = s_carry;
    step_meta[1] = G;
    step_meta[2] = ss.nl;
  }
  if (tid >= 32 && tid < 32 + EB_META_LEN - 3) {
    const int i = tid - 32;   // entries 3 .. EB_META_LEN-1
    step_meta[3 + i] = i < D ? ss.nl * (s_dev_off[i] + i * S) : i == D ? G : 0;
  }
  __syncthreads();

  // ---- ranks per chunk (one warp each), as in rank_kernel
  for (int c = warp; c < bp.n_chunks; c += kFusedThreads / 32) {
    const int j = mb_of_chunk(bp, c);
    const int t0 = bp.tok_off[j] + (c - bp.chunk_off[j]) * 32;
    const int nt = min(32, bp.tok_off[j + 1] - t0);
    if (!((run >> j) & 1u)) {
      for (int a = lane; a < nt * KS; a += 32) pos[(size_t)t0 * KS + a] = -1;
      continue;
    }
    const int lr = ss.rank_of_mb[j];
    int* next = s_tab + c * E;
    for (int e = lane; e < E; e += 32)
      next[e] += s_goff[group_id(s_dev_off, S, ss.nl, s_e2d[e], lr, s_e_local[e])];
    __syncwarp();
    for (int a0 = 0; a0 < nt * K; a0 += 32) {
      const int a = a0 + lane;
      bool valid = a < nt * K;
      int e = valid ? s_topk[t0 * K + a] : -1 - lane;
      if (valid && (unsigned)e >= (unsigned)E) {   // as in rank_kernel: skipped and counted, never used as an index
        pos[(size_t)(t0 + a / K) * KS + a % K] = -1;
        atomicAdd(&step_meta[EB_META_LEN - 1], 1);
        valid = false;
        e = -1 - lane;
      }
      const unsigned peers = __match_any_sync(0xffffffffu, e);
      const int before = __popc(peers & ((1u << lane) - 1u));
      if (valid) {
        const int p = next[e] + before;
        const int t = t0 + a / K, k = a % K;
        pos[(size_t)t * KS + k] = p;
        row_src[p] = t;
      }
      __syncwarp();
      if (valid && before == 0) next[e] += __popc(peers);
      __syncwarp();
    }
    if (S > 0 && lane < nt) {
      const int tl = t0 + lane - bp.tok_off[j];
      int d = 0;   // home device: the last one whose first token is not beyond tl
      while (d + 1 < D && tl >= s_home[j][d + 1]) ++d;
      int before = 0;
      for (int j2 = 0; j2 < j; ++j2)
        if (ss.rank_of_mb[j2] == lr) before += s_home[j2][d + 1] - s_home[j2][d];
      const int n_d = s_dev_off[d + 1] - s_dev_off[d];
      for (int s2 = 0; s2 < S; ++s2) {
        const int p = s_goff[group_id(s_dev_off, S, ss.nl, d, lr, n_d + s2)] + before + (tl - s_home[j][d]);
        pos[(size_t)(t0 + lane) * KS + K + s2] = p;
        row_src[p] = t0 + lane;
      }
    }
  }
}

// ---- gather --------------------------------------------------------------------------------
// A team of threads per token (one 16-byte vector each, so a whole row is in flight at once): the row
// is read once and written to each of its K + S rows.  `team` is 32..256 and divides the block.
constexpr int kGatherThreads = 256;

__global__ void __launch_bounds__(kGatherThreads)
gather_kernel(int n_tok, int H, int KS, int team, const uint4* __restrict__ x, const int32_t* __restrict__ pos,
              uint4* __restrict__ xp) {
  EB_GRID_DEP_SYNC();
  const int t = blockIdx.x * (kGatherThreads / team) + threadIdx.x / team;   // team >= 32: a warp serves one token
  if (t >= n_tok) return;
  const int lane = threadIdx.x & 31;
  const int my_pos = lane < KS ? pos[(size_t)t * KS + lane] : -1;   // lane s fetches slot s once per warp
  if (__shfl_sync(0xffffffffu, my_pos, 0) < 0) return;              // micro-batch does not run
  const int vec = H / 8;  // 16-byte vectors per row
  const uint4* src = x + (size_t)t * vec;
  for (int v0 = 0; v0 < vec; v0 += team) {
    const int v = v0 + threadIdx.x % team;
    uint4 r = make_uint4(0, 0, 0, 0);
    if (v < vec) r = __ldg(src + v);
    for (int s = 0; s < KS; ++s) {
      const int p = __shfl_sync(0xffffffffu, my_pos, s);
      if (v < vec && p >= 0) xp[(size_t)p * vec + v] = r;
    }
  }
}

static inline int team_for(int vec) { return vec <= 32 ? 32 : vec <= 64 ? 64 : vec <= 128 ? 128 : 256; }

}  // namespace

extern "C" eb_status eb_permute(eb_ctx* c, void* stream, const eb_batch* batch, const eb_sched_result* d_res,
                                const void* x, const int32_t* topk_idx, int32_t* group_off, int32_t* group_w,
                                int32_t* row_src, int32_t* pos, void* xp, int32_t* step_meta) {
  if (!c) return EB_ERR_INVALID_ARG;
  BatchParams bp;
  eb_status s = ebi_make_batch(c, batch, &bp);
  if (s != EB_OK) return s;
  if (!d_res || !x || !topk_idx || !group_off || !group_w || !row_src || !pos || !xp || !step_meta)
    return ebi_fail(c, EB_ERR_INVALID_ARG, "null pointer");
  if (!ebi_aligned16(x) || !ebi_aligned16(xp)) return ebi_fail(c, EB_ERR_INVALID_ARG, "x / xp must be 16-byte aligned");
  if (!c->ws) return ebi_fail(c, EB_ERR_WORKSPACE, "no workspace set");
  cudaStream_t st = (cudaStream_t)stream;
  const int gcap = ebi_groups_cap(c);
  const int chunk_blocks = (bp.n_chunks + kWarps - 1) / kWarps;
  if (bp.n_chunks <= kFusedMaxChunks && gcap <= kFusedMaxGroups) {
    // small step: one block does histogram, sizes, scan and ranks
    const size_t smem = sizeof(int) * ((size_t)kFusedMaxChunks * EB_MAX_E + kFusedMaxGroups + 1 + (size_t)kFusedMaxChunks * 32 * EB_MAX_K);
    if (!c->fused_attr_set) {   // per context: function attributes belong to the current device
      EB_CUDA(c, cudaFuncSetAttribute(permute_fused_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
      c->fused_attr_set = true;
    }
    KernelTimer timer(c, EBK_PERMUTE_FUSED, st);
    ebi_launch(permute_fused_kernel, dim3(1), dim3(kFusedThreads), sizeof(int) * ((size_t)bp.n_chunks * c->cfg.E + gcap + 1 + (size_t)bp.n_tok * c->cfg.K),
               st, c->mp, bp, d_res, topk_idx, group_off, group_w, pos, row_src, step_meta);
  } else {
    if (bp.n_chunks > 0) {
      KernelTimer timer(c, EBK_PERMUTE_HIST, st);
      ebi_launch(hist_kernel, dim3(chunk_blocks), dim3(kWarps * 32), 0, st, c->mp, bp, d_res, topk_idx, c->chunk_hist);
    }
    {
      KernelTimer timer(c, EBK_PERMUTE_SIZES, st);
      ebi_launch(sizes_kernel, dim3((gcap + kWarps - 1) / kWarps), dim3(kWarps * 32), 0, st, c->mp, bp, d_res,
                 (const int32_t*)c->chunk_hist, c->chunk_base, c->group_size);
    }
    {
      KernelTimer timer(c, EBK_PERMUTE_SCAN, st);
      ebi_launch(scan_kernel, dim3(1), dim3(1024), 0, st, c->mp, bp, d_res, (const int32_t*)c->group_size, group_off, group_w,
                 step_meta);
    }
    if (bp.n_chunks > 0) {
      KernelTimer timer(c, EBK_PERMUTE_RANK, st);
      ebi_launch(rank_kernel, dim3(chunk_blocks), dim3(kWarps * 32), 0, st, c->mp, bp, d_res, topk_idx,
                 (const int32_t*)c->chunk_base, (const int32_t*)group_off, pos, row_src, step_meta);
    }
  }
  if (bp.n_tok > 0) {
    KernelTimer timer(c, EBK_PERMUTE_GATHER, st);
    const int team = team_for(c->cfg.H / 8), tpb = kGatherThreads / team;
    ebi_launch(gather_kernel, dim3((bp.n_tok + tpb - 1) / tpb), dim3(kGatherThreads), 0, st, bp.n_tok, c->cfg.H,
               c->cfg.K + c->cfg.S, team, (const uint4*)x, (const int32_t*)pos, (uint4*)xp);
  }
  EB_LAUNCH_CHECK(c, "permute");
  return EB_OK;
}

// ---- eb_check_permutation ----------------------------------------------------------------------
// Device-side consistency check of a step's permutation tables (stands in for a memory checker on
// boxes where none is available): every index is range-checked before use, nothing is dereferenced
// on a bad index, and the number of violations is returned.
namespace {

__global__ void __launch_bounds__(256)
check_kernel(ModelParams mp, BatchParams bp, int rows_cap, int groups_cap, const eb_sched_result* __restrict__ res,
             const int32_t* __restrict__ topk_idx, const int32_t* __restrict__ group_off,
             const int32_t* __restrict__ group_w, const int32_t* __restrict__ row_src, const int32_t* __restrict__ pos,
             const int32_t* __restrict__ step_meta, int32_t* __restrict__ errors) {
  EB_GRID_DEP_SYNC();
  const int R = step_meta[0], G = step_meta[1];
  const uint32_t run = res->run_mask;
  const int KS = mp.K + mp.S;
  int bad = 0;
  const int tid = blockIdx.x * blockDim.x + threadIdx.x, nthr = gridDim.x * blockDim.x;
  if (R < 0 || R > rows_cap || G < 0 || G > groups_cap) {
    if (tid == 0) atomicAdd(errors, 1);
    return;
  }
  // group offsets: start at 0, ascending, end at R; weight ids in range
  for (int g = tid; g <= G; g += nthr) {
    int o = group_off[g];
    if (o < 0 || o > R) ++bad;
    if (g == 0 && o != 0) ++bad;
    if (g == G && o != R) ++bad;
    if (g < G) {
      if (group_off[g + 1] < o) ++bad;
      int w = group_w[g];
      if (w < 0 || w >= mp.L * (mp.E + mp.S)) ++bad;
    }
  }
  // pos and row_src are mutually inverse on the chosen tokens; -1 elsewhere; rows land in a group of
  // the token's layer and expert; rows of a group keep token order
  for (int i = tid; i < bp.n_tok * KS; i += nthr) {
    const int t = i / KS, slot = i % KS;
    int j = 0;
    while (j + 1 < bp.n_mb && t >= bp.tok_off[j + 1]) ++j;
    const int p = pos[i];
    if (!((run >> j) & 1u)) {
      if (p != -1) ++bad;
      continue;
    }
    if (p < 0 || p >= R) {
      ++bad;
      continue;
    }
    if (row_src[p] != t) ++bad;
    // binary search of the group holding row p
    int lo = 0, hi = G - 1;
    while (lo < hi) {
      int mid = (lo + hi + 1) >> 1;
      if (group_off[mid] <= p) lo = mid; else hi = mid - 1;
    }
    const int w = group_w[lo];
    const int layer = w / (mp.E + mp.S), e = w % (mp.E + mp.S);
    if (layer != bp.layer[j]) ++bad;
    if (slot < mp.K) {
      const int want = topk_idx[(size_t)t * mp.K + slot];
      if (want < 0 || want >= mp.E || e != want) ++bad;
    } else if (e != mp.E + (slot - mp.K)) {
      ++bad;
    }
    if (p > group_off[lo] && row_src[p - 1] >= t) ++bad;   // stable order inside the group
  }
  for (int r = tid; r < R; r += nthr) {
    int t = row_src[r];
    if (t < 0 || t >= bp.n_tok) ++bad;
  }
  if (bad) atomicAdd(errors, bad);
}

}  // namespace

extern "C" eb_status eb_check_permutation(eb_ctx* c, void* stream, const eb_batch* batch, const eb_sched_result* d_res,
                                          const int32_t* topk_idx, const int32_t* group_off, const int32_t* group_w,
                                          const int32_t* row_src, const int32_t* pos, const int32_t* step_meta,
                                          int32_t* out_errors) {
  if (!c) return EB_ERR_INVALID_ARG;
  BatchParams bp;
  eb_status s = ebi_make_batch(c, batch, &bp);
  if (s != EB_OK) return s;
  if (!d_res || !topk_idx || !group_off || !group_w || !row_src || !pos || !step_meta || !out_errors)
    return ebi_fail(c, EB_ERR_INVALID_ARG, "null pointer");
  if (!c->ws) return ebi_fail(c, EB_ERR_WORKSPACE, "no workspace set");
  cudaStream_t st = (cudaStream_t)stream;
  int32_t* d_err = c->group_size;   // scratch word; the next eb_permute rewrites it
  EB_CUDA(c, cudaMemsetAsync(d_err, 0, sizeof(int32_t), st));
  ebi_launch(check_kernel, dim3(2 * c->num_sms), dim3(256), 0, st, c->mp, bp, ebi_rows_cap(c), ebi_groups_cap(c), d_res,
             topk_idx, group_off, group_w, row_src, pos, step_meta, d_err);
  EB_LAUNCH_CHECK(c, "check_permutation");
  EB_CUDA(c, cudaMemcpyAsync(out_errors, d_err, sizeof(int32_t), cudaMemcpyDeviceToHost, st));
  EB_CUDA(c, cudaStreamSynchronize(st));
  return EB_OK;
}

// ---- eb_permute_noalloc ------------------------------------------------------------------------
// Same dispatch as eb_permute for callers that must not create device allocations: no context, no
// workspace.  The expert tables and the permutation scratch live in one file-scope device array
// that every GPU loading the library holds until the process exits.
namespace {

constexpr int kNaMaxTokens = EB_NOALLOC_MAX_TOKENS;
constexpr int kNaMaxChunks = kNaMaxTokens / 32 + EB_MAX_MB;
constexpr int kNaTableWords = 1024;                                   // e2d | dev_off | dev_list | e_local
constexpr int kNaHistWords = kNaMaxChunks * EB_MAX_E;
constexpr int kNaGroupWords = EB_MAX_MB * (EB_MAX_E + EB_MAX_D * EB_MAX_S);
constexpr int kNaWords = kNaTableWords + 2 * kNaHistWords + kNaGroupWords;
static_assert(3 * EB_MAX_E + EB_MAX_D + 1 <= kNaTableWords, "expert tables do not fit");

// About 316 KB.  In host code this name is only a handle for cudaGetSymbolAddress, never a pointer.
static __device__ __align__(256) int32_t g_noalloc_scratch[kNaWords];

constexpr int kNaMaxDevices = 64;
int32_t* g_noalloc_ptr[kNaMaxDevices] = {};

// Expert tables of one call, handed to the set-up kernel by value (they travel in the launch's parameter
// buffer, so no host memory has to outlive the call).
struct NaTables {
  int32_t n;
  int32_t v[3 * EB_MAX_E + EB_MAX_D + 1];
};
static_assert(sizeof(NaTables) <= 4000, "kernel parameter space");

// Writes the expert tables and clears the counters of the shared scratch array: every call starts from
// the same state whatever the previous call left behind.
__global__ void __launch_bounds__(256)
noalloc_setup_kernel(const __grid_constant__ NaTables t, int32_t* __restrict__ d_tab, int32_t* __restrict__ d_hist, int n_hist,
                     int32_t* __restrict__ d_gsize, int n_gsize) {
  const int tid = blockIdx.x * blockDim.x + threadIdx.x, nthr = gridDim.x * blockDim.x;
  for (int i = tid; i < t.n; i += nthr) d_tab[i] = t.v[i];
  for (int i = tid; i < n_hist; i += nthr) d_hist[i] = 0;
  for (int i = tid; i < n_gsize; i += nthr) d_gsize[i] = 0;
}

eb_status noalloc_fail(char* err, size_t cap, eb_status s, const char* msg) {
  if (err && cap) {
    size_t n = strlen(msg) < cap - 1 ? strlen(msg) : cap - 1;
    memcpy(err, msg, n);
    err[n] = 0;
  }
  return s;
}

}  // namespace

extern "C" eb_status eb_permute_noalloc(const eb_config* cfg, void* stream, const eb_batch* batch,
                                        const eb_sched_result* d_res, const void* x, const int32_t* topk_idx,
                                        int32_t* group_off, int32_t* group_w, int32_t* row_src, int32_t* pos,
                                        void* xp, int32_t* step_meta, char* err, size_t err_cap) {
  if (err && err_cap) err[0] = 0;
  if (!cfg || !cfg->expert_to_device) return noalloc_fail(err, err_cap, EB_ERR_INVALID_ARG, "null config");
  const eb_config& g = *cfg;
  if (g.L < 1 || g.E < 1 || g.E > EB_MAX_E || g.K < 1 || g.K > EB_MAX_K || g.K > g.E || g.S < 0 || g.S > EB_MAX_S ||
      g.D < 1 || g.D > EB_MAX_D || g.H < 8 || (g.H % 8))
    return noalloc_fail(err, err_cap, EB_ERR_UNSUPPORTED, "shape outside the library limits");
  for (int e = 0; e < g.E; ++e)
    if (g.expert_to_device[e] < 0 || g.expert_to_device[e] >= g.D)
      return noalloc_fail(err, err_cap, EB_ERR_INVALID_ARG, "expert_to_device entry out of range");
  if (!batch || !batch->tok_off || !batch->layer) return noalloc_fail(err, err_cap, EB_ERR_INVALID_ARG, "null batch");
  if (batch->n_mb >= 0 && batch->n_mb <= EB_MAX_MB && batch->tok_off[batch->n_mb] > kNaMaxTokens)
    return noalloc_fail(err, err_cap, EB_ERR_UNSUPPORTED,
                        "eb_permute_noalloc handles at most EB_NOALLOC_MAX_TOKENS (4096) packed tokens: "
                        "its scratch is a fixed device array; use eb_permute with a workspace for more");
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kNaMaxDevices)
    return noalloc_fail(err, err_cap, EB_ERR_CUDA, "cudaGetDevice failed or device index too large");
  eb_ctx tmp;  // host-only helper for the shared argument checks; owns no device memory
  tmp.cfg = g;
  tmp.cfg.max_tokens = kNaMaxTokens;
  tmp.device = dev;   // the checks compare against the current device: this call belongs to whichever device is current
  BatchParams bp;
  eb_status s = ebi_make_batch(&tmp, batch, &bp);
  if (s != EB_OK) return noalloc_fail(err, err_cap, s, tmp.err.c_str());
  if (!d_res || !x || !topk_idx || !group_off || !group_w || !row_src || !pos || !xp || !step_meta)
    return noalloc_fail(err, err_cap, EB_ERR_INVALID_ARG, "null pointer");
  if (!ebi_aligned16(x) || !ebi_aligned16(xp))
    return noalloc_fail(err, err_cap, EB_ERR_INVALID_ARG, "x / xp must be 16-byte aligned");

  // one-time set-up per device: resolve the device address of the scratch array
  if (!g_noalloc_ptr[dev]) {
    int32_t* p = nullptr;
    cudaError_t e = cudaGetSymbolAddress((void**)&p, g_noalloc_scratch);
    if (e != cudaSuccess || !p) return noalloc_fail(err, err_cap, EB_ERR_CUDA, cudaGetErrorString(e));
    g_noalloc_ptr[dev] = p;
  }
  int32_t* base = g_noalloc_ptr[dev];
  int32_t* d_tab = base;
  int32_t* d_hist = base + kNaTableWords;
  int32_t* d_cbase = d_hist + kNaHistWords;
  int32_t* d_gsize = d_cbase + kNaHistWords;

  // expert tables, same layout as a context's: e2d | dev_off | dev_list | e_local
  NaTables tables;
  int32_t* tab = tables.v;
  tables.n = 3 * g.E + g.D + 1;
  int32_t* h_off = tab + g.E;
  int32_t* h_list = h_off + g.D + 1;
  int32_t* h_local = h_list + g.E;
  int n = 0;
  for (int d = 0; d < g.D; ++d) {
    h_off[d] = n;
    for (int e = 0; e < g.E; ++e)
      if (g.expert_to_device[e] == d) {
        h_local[e] = n - h_off[d];
        h_list[n++] = e;
      }
  }
  h_off[g.D] = n;
  for (int e = 0; e < g.E; ++e) tab[e] = g.expert_to_device[e];
  ModelParams mp;
  mp.L = g.L; mp.E = g.E; mp.K = g.K; mp.S = g.S; mp.H = g.H; mp.I = g.I; mp.D = g.D;
  mp.renorm = g.renorm_topk ? 1 : 0;
  mp.e2d = d_tab;
  mp.dev_off = d_tab + g.E;
  mp.dev_list = mp.dev_off + g.D + 1;
  mp.e_local = mp.dev_list + g.E;

  cudaStream_t st = (cudaStream_t)stream;
  // the array keeps the previous call's contents: tables rewritten, counters start from zero every call
  noalloc_setup_kernel<<<64, 256, 0, st>>>(tables, d_tab, d_hist, kNaHistWords, d_gsize, kNaGroupWords);
  cudaError_t ce = cudaGetLastError();
  if (ce != cudaSuccess) return noalloc_fail(err, err_cap, EB_ERR_CUDA, cudaGetErrorString(ce));

  const int gcap = EB_MAX_MB * (g.E + g.D * g.S);
  const int chunk_blocks = (bp.n_chunks + kWarps - 1) / kWarps;
  if (bp.n_chunks > 0) hist_kernel<<<chunk_blocks, kWarps * 32, 0, st>>>(mp, bp, d_res, topk_idx, d_hist);
  sizes_kernel<<<(gcap + kWarps - 1) / kWarps, kWarps * 32, 0, st>>>(mp, bp, d_res, d_hist, d_cbase, d_gsize);
  scan_kernel<<<1, 1024, 0, st>>>(mp, bp, d_res, d_gsize, group_off, group_w, step_meta);
  if (bp.n_chunks > 0)
    rank_kernel<<<chunk_blocks, kWarps * 32, 0, st>>>(mp, bp, d_res, topk_idx, d_cbase, group_off, pos, row_src, step_meta);
  if (bp.n_tok > 0) {
    const int team = team_for(g.H / 8), tpb = kGatherThreads / team;
    gather_kernel<<<(bp.n_tok + tpb - 1) / tpb, kGatherThreads, 0, st>>>(bp.n_tok, g.H, g.K + g.S, team, (const uint4*)x,
                                                                         pos, (uint4*)xp);
  }
  ce = cudaGetLastError();
  if (ce != cudaSuccess) return noalloc_fail(err, err_cap, EB_ERR_CUDA, cudaGetErrorString(ce));
  return EB_OK;
}
