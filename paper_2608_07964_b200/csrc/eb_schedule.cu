// eb_schedule: Schedule(S, m) of Algorithm 1 as one thread block.
//
// MaxUtil (Section 4.2) enumerates every subset of the pool with at least m members.  The pool
// is split into a low and a high half; the summed load vector of each half-subset is tabulated
// in shared memory (2 x 256 x D entries at most), so a subset costs D additions and a maximum.
// Utilisation (Eq. 3 for one step) is sum(W) / (D * max(W)); D is common to all candidates, so
// candidates are compared exactly by cross-multiplying sum and max in 64-bit integers.
// Total order: higher utilisation, then more members, then the numerically smaller mask.
// CumUtil / DiffPeak (Section 5.2) are sequential and run on one thread; topping their result up to m
// members scores the remaining pool members in parallel, one lane each.
#include <algorithm>

#include "eb_internal.cuh"

namespace {

constexpr int kThreads = 1024;
constexpr int kMaxBlocks = 64;

struct Cand {
  long long num;   // sum_d W_d  (D if there is no work: U := 1)
  long long peak;  // max_d W_d  (1 if there is no work)
  int n;           // members
  unsigned sub;    // subset in pool-relative bit positions (order preserving w.r.t. the real mask)
};

__device__ __forceinline__ bool better(const Cand& a, const Cand& b) {
  if (b.n < 0) return a.n >= 0;
  if (a.n < 0) return false;
  long long l = a.num * b.peak, r = b.num * a.peak;
  if (l != r) return l > r;
  if (a.n != b.n) return a.n > b.n;
  return a.sub < b.sub;
}

__device__ __forceinline__ Cand make_cand(const long long* w, int D, int n, unsigned sub) {
  long long num = 0, peak = 0;
  for (int d = 0; d < D; ++d) {
    num += w[d];
    peak = w[d] > peak ? w[d] : peak;
  }
  Cand c;
  if (peak == 0) {
    c.num = D;
    c.peak = 1;
  } else {
    c.num = num;
    c.peak = peak;
  }
  c.n = n;
  c.sub = sub;
  return c;
}

// best candidate of the warp, in every lane
__device__ __forceinline__ Cand warp_best(Cand c) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    Cand oth;
    oth.num = __shfl_xor_sync(0xffffffffu, c.num, o);
    oth.peak = __shfl_xor_sync(0xffffffffu, c.peak, o);
    oth.n = __shfl_xor_sync(0xffffffffu, c.n, o);
    oth.sub = __shfl_xor_sync(0xffffffffu, c.sub, o);
    if (better(oth, c)) c = oth;
  }
  return c;
}

__global__ void __launch_bounds__(kThreads)
schedule_kernel(int D, int n_mb, uint32_t pool_mask, int m, int policy, const int32_t* __restrict__ mb_load,
                eb_sched_result* __restrict__ res, Cand* __restrict__ block_best, unsigned* __restrict__ block_counter) {
  EB_GRID_DEP_SYNC();
  __shared__ bool s_last;
  __shared__ int s_load[EB_MAX_MB][EB_MAX_D];
  __shared__ int s_lo[256][EB_MAX_D];
  __shared__ int s_hi[256][EB_MAX_D];
  __shared__ int s_member[EB_MAX_MB];
  __shared__ Cand s_best[kThreads / 32];
  __shared__ uint32_t s_run;
  __shared__ uint32_t s_seq_run;
  __shared__ int s_seq_n;
  __shared__ long long s_seq_w[EB_MAX_D];

  const int tid = threadIdx.x;
  for (int i = tid; i < EB_MAX_MB * EB_MAX_D; i += kThreads) {
    int j = i / EB_MAX_D, d = i % EB_MAX_D;
    s_load[j][d] = (j < n_mb && d < D) ? mb_load[j * D + d] : 0;
  }
  const int np = __popc(pool_mask);
  if (tid < EB_MAX_MB && ((pool_mask >> tid) & 1u)) s_member[__popc(pool_mask & ((1u << tid) - 1u))] = tid;
  __syncthreads();

  if (np <= m || policy == EB_POLICY_ALL) {
    if (tid == 0) s_run = pool_mask;
  } else if (policy == EB_POLICY_MAXUTIL) {
    const int nlo = np < 8 ? np : 8, nhi = np - nlo;
    for (int i = tid; i < (1 << nlo) * EB_MAX_D; i += kThreads) {
      int s = i / EB_MAX_D, d = i % EB_MAX_D, acc = 0;
      for (int b = 0; b < nlo; ++b)
        if ((s >> b) & 1) acc += s_load[s_member[b]][d];
      s_lo[s][d] = acc;
    }
    for (int i = tid; i < (1 << nhi) * EB_MAX_D; i += kThreads) {
      int s = i / EB_MAX_D, d = i % EB_MAX_D, acc = 0;
      for (int b = 0; b < nhi; ++b)
        if ((s >> b) & 1) acc += s_load[s_member[nlo + b]][d];
      s_hi[s][d] = acc;
    }
    __syncthreads();
    Cand best;
    best.n = -1; best.num = 0; best.peak = 1; best.sub = 0;
    const unsigned total = 1u << np, lomask = (1u << nlo) - 1u;
    for (unsigned sub = blockIdx.x * kThreads + tid + 1; sub < total; sub += gridDim.x * kThreads) {
      int n = __popc(sub);
      if (n < m) continue;
      long long w[EB_MAX_D];
      const int* lo = s_lo[sub & lomask];
      const int* hi = s_hi[sub >> nlo];
#pragma unroll
      for (int d = 0; d < EB_MAX_D; ++d) w[d] = (long long)lo[d] + hi[d];
      Cand c = make_cand(w, D, n, sub);
      if (better(c, best)) best = c;
    }
    // warp then block reduction under the total order (any reduction order gives the same winner)
    best = warp_best(best);
    if ((tid & 31) == 0) s_best[tid >> 5] = best;
    __syncthreads();
    if (tid < 32) {
      Cand b = warp_best(s_best[tid]);
      if (tid == 0) s_best[0] = b;
    }
    if (gridDim.x > 1) {
      // every block leaves its best candidate in global memory; the block that arrives last reduces them
      if (tid == 0) {
        block_best[blockIdx.x] = s_best[0];
        __threadfence();
        const unsigned arrived = atomicAdd(block_counter, 1u);
        s_last = arrived == gridDim.x - 1;
      }
      __syncthreads();
      if (!s_last) return;
      __threadfence();
      if (tid < 32) {
        Cand b;
        b.n = -1; b.num = 0; b.peak = 1; b.sub = 0;
        for (int i = tid; i < (int)gridDim.x; i += 32) {
          const Cand o = block_best[i];
          if (better(o, b)) b = o;
        }
        b = warp_best(b);
        if (tid == 0) {
          s_best[0] = b;
          *block_counter = 0;   // ready for the next call
        }
      }
    }
    if (tid == 0) {
      const Cand b = s_best[0];
      uint32_t mask = 0;
      for (int k = 0; k < np; ++k)
        if ((b.sub >> k) & 1u) mask |= 1u << s_member[k];
      s_run = mask;
    }
  } else if (tid == 0) {
    // CumUtil / DiffPeak: ascending pool members, the first always taken
    long long w[EB_MAX_D];
    for (int d = 0; d < EB_MAX_D; ++d) w[d] = s_load[s_member[0]][d];
    uint32_t run = 1u << s_member[0];
    int n = 1;
    uint32_t peaks = 0;
    auto peak_dev = [&](int j) {
      int best = 0;
      for (int d = 1; d < D; ++d)
        if (s_load[j][d] > s_load[j][best]) best = d;
      return best;
    };
    peaks |= 1u << peak_dev(s_member[0]);
    for (int k = 1; k < np; ++k) {
      int j = s_member[k];
      bool take;
      if (policy == EB_POLICY_CUMUTIL) {
        long long w2[EB_MAX_D];
        for (int d = 0; d < EB_MAX_D; ++d) w2[d] = w[d] + s_load[j][d];
        Cand cur = make_cand(w, D, 0, 0), nxt = make_cand(w2, D, 0, 0);
        take = nxt.num * cur.peak > cur.num * nxt.peak;
      } else {
        take = !((peaks >> peak_dev(j)) & 1u);
      }
      if (take) {
        for (int d = 0; d < EB_MAX_D; ++d) w[d] += s_load[j][d];
        run |= 1u << j;
        peaks |= 1u << peak_dev(j);
        ++n;
      }
    }
    s_seq_run = run;
    s_seq_n = n;
    for (int d = 0; d < EB_MAX_D; ++d) s_seq_w[d] = w[d];
  }
  if (policy == EB_POLICY_CUMUTIL || policy == EB_POLICY_DIFFPEAK) {
    if (!(np <= m)) {
      // top up to m members: repeatedly add the member whose inclusion gives the highest utilisation
      // (lowest index on ties); lane k of warp 0 scores pool member k
      __syncthreads();
      if (tid < 32) {
        uint32_t run = s_seq_run;
        int n = s_seq_n;
        while (n < m) {
          Cand cu;
          cu.n = -1; cu.num = 0; cu.peak = 1; cu.sub = 0;
          if (tid < np && !((run >> s_member[tid]) & 1u)) {
            long long w2[EB_MAX_D];
            for (int d = 0; d < EB_MAX_D; ++d) w2[d] = s_seq_w[d] + s_load[s_member[tid]][d];
            cu = make_cand(w2, D, 1, (unsigned)tid);   // equal sizes: ties fall to the lower index
          }
          for (int o = 16; o > 0; o >>= 1) {
            Cand oth;
            oth.num = __shfl_xor_sync(0xffffffffu, cu.num, o);
            oth.peak = __shfl_xor_sync(0xffffffffu, cu.peak, o);
            oth.n = __shfl_xor_sync(0xffffffffu, cu.n, o);
            oth.sub = __shfl_xor_sync(0xffffffffu, cu.sub, o);
            if (better(oth, cu)) cu = oth;
          }
          if (cu.n < 0) break;
          const int bj = s_member[cu.sub];
          __syncwarp();
          if (tid < EB_MAX_D) s_seq_w[tid] += s_load[bj][tid];
          __syncwarp();
          run |= 1u << bj;
          ++n;
        }
        if (tid == 0) s_run = run;
      }
    }
  }
  __syncthreads();
  if (tid < 32) {
    // lane d sums the chosen micro-batches' load on device d (zero beyond D); the warp adds and maximises
    const uint32_t run = s_run;
    long long v = 0;
    if (tid < EB_MAX_D) {
      for (int j = 0; j < EB_MAX_MB; ++j)
        if ((run >> j) & 1u) v += s_load[j][tid];
      res->joint_load[tid] = (int32_t)v;
    }
    long long num = v, peak = v;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      num += __shfl_xor_sync(0xffffffffu, num, o);
      const long long p2 = __shfl_xor_sync(0xffffffffu, peak, o);
      peak = p2 > peak ? p2 : peak;
    }
    if (tid == 0) {
      res->run_mask = run;
      res->defer_mask = pool_mask & ~run;
      res->n_run = __popc(run);
      res->status = EB_OK;
      res->util_num = num;
      res->util_den = (long long)D * peak;
    }
  }
}

}  // namespace

extern "C" eb_status eb_schedule(eb_ctx* c, void* stream, const eb_batch* batch, int32_t m, eb_policy policy,
                                 const int32_t* mb_load, eb_sched_result* d_res, eb_sched_result* h_res) {
  if (!c) return EB_ERR_INVALID_ARG;
  BatchParams bp;
  eb_status s = ebi_make_batch(c, batch, &bp);
  if (s != EB_OK) return s;
  if (!mb_load || !d_res) return ebi_fail(c, EB_ERR_INVALID_ARG, "null pointer");
  if (m < 1) return ebi_fail(c, EB_ERR_INVALID_ARG, "m must be at least 1");
  if ((int)policy < 0 || (int)policy > EB_POLICY_ALL) return ebi_fail(c, EB_ERR_INVALID_ARG, "unknown policy");
  cudaStream_t st = (cudaStream_t)stream;
  {
    // MaxUtil over a large pool: the subsets are split over several blocks (one SM cannot enumerate 2^16
    // subsets quickly); everything else is one block
    int np = 0;
    for (int j = 0; j < bp.n_mb; ++j) np += (batch->pool_mask >> j) & 1u;
    int blocks = 1;
    if (policy == EB_POLICY_MAXUTIL && np > m && np > 11) blocks = std::min(kMaxBlocks, 1 << (np - 10));
    KernelTimer timer(c, EBK_SCHEDULE, st);
    ebi_launch(schedule_kernel, dim3(blocks), dim3(kThreads), 0, st, c->cfg.D, bp.n_mb, batch->pool_mask, (int)m,
               (int)policy, mb_load, d_res, (Cand*)c->d_sched_scratch, (unsigned*)(c->d_sched_scratch + kMaxBlocks * sizeof(Cand)));
  }
  EB_LAUNCH_CHECK(c, "schedule");
  if (h_res) {
    EB_CUDA(c, cudaMemcpyAsync(h_res, d_res, sizeof(eb_sched_result), cudaMemcpyDeviceToHost, st));
    EB_CUDA(c, cudaStreamSynchronize(st));
  }
  return EB_OK;
}
