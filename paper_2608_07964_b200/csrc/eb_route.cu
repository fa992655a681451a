// eb_route: top-k softmax gating (Section 2.1) and per-micro-batch workload vectors (Section 2.3).
//
// One warp per token.  Lane i holds logits i, i+32, ...  (E <= 256 -> at most 8 per lane).
// K rounds of a warp arg-max under the order (value descending, index ascending) pick the
// experts; the decision uses only comparisons on the raw fp32 logits, so it is exact.
// Loads are integer counts added with integer atomics in global memory (order independent, hence
// deterministic); a clearing kernel zeroes the rows of the micro-batches being routed first.  (Gathering
// the counts per block in shared memory was tried: it needs several tokens per block to pay, and the lost
// parallelism cost more than the atomics it saved.)
#include "eb_internal.cuh"

namespace {

constexpr int kWarpsPerBlock = 8;
constexpr int kMaxPerLane = EB_MAX_E / 32;

__global__ void __launch_bounds__(kWarpsPerBlock * 32)
route_kernel(ModelParams mp, BatchParams bp, uint32_t route_mask, const float* __restrict__ logits,
             int32_t* __restrict__ topk_idx, float* __restrict__ topk_w, int32_t* __restrict__ mb_load,
             int32_t* __restrict__ mb_cnt) {
  EB_GRID_DEP_SYNC();
  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int t = blockIdx.x * kWarpsPerBlock + warp;
  if (t >= bp.n_tok) return;
  int j = 0;
  while (j + 1 < bp.n_mb && t >= bp.tok_off[j + 1]) ++j;
  if (!((route_mask >> j) & 1u)) return;

  const int E = mp.E, K = mp.K;
  const float* z = logits + (size_t)t * E;
  float v[kMaxPerLane];
  bool taken[kMaxPerLane];
#pragma unroll
  for (int i = 0; i < kMaxPerLane; ++i) {
    int e = lane + 32 * i;
    v[i] = e < E ? z[e] : 0.f;
    taken[i] = e >= E;
  }

  float z_top = 0.f, my_p = 0.f, p_sum = 0.f;
  int my_e = -1;
  for (int k = 0; k < K; ++k) {
    // lane-local best under (value desc, index asc)
    float bv = 0.f;
    int be = 0x7fffffff;
#pragma unroll
    for (int i = 0; i < kMaxPerLane; ++i) {
      int e = lane + 32 * i;
      if (!taken[i] && (be == 0x7fffffff || v[i] > bv)) {  // ascending i keeps the lower index on ties
        bv = v[i];
        be = e;
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      float ov = __shfl_xor_sync(0xffffffffu, bv, o);
      int oe = __shfl_xor_sync(0xffffffffu, be, o);
      bool other = oe != 0x7fffffff && (be == 0x7fffffff || ov > bv || (ov == bv && oe < be));
      if (other) {
        bv = ov;
        be = oe;
      }
    }
#pragma unroll
    for (int i = 0; i < kMaxPerLane; ++i)
      if (lane + 32 * i == be) taken[i] = true;
    if (k == 0) z_top = bv;
    float p = expf(bv - z_top);
    p_sum += p;
    if (lane == k) {
      my_e = be;
      my_p = p;
    }
  }
  if (!mp.renorm) {
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < kMaxPerLane; ++i)
      if (lane + 32 * i < E) s += expf(v[i] - z_top);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    p_sum = s;
  }
  if (lane < K) {
    topk_idx[(size_t)t * K + lane] = my_e;
    topk_w[(size_t)t * K + lane] = my_p / p_sum;
    atomicAdd(&mb_cnt[j * E + my_e], 1);
    atomicAdd(&mb_load[j * mp.D + mp.e2d[my_e]], 1);
  }
}

__global__ void route_clear_kernel(ModelParams mp, BatchParams bp, uint32_t route_mask, int32_t* mb_load,
                                   int32_t* mb_cnt) {
  EB_GRID_DEP_SYNC();
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  int per = mp.E + mp.D;
  if (i >= bp.n_mb * per) return;
  int j = i / per, r = i % per;
  if (!((route_mask >> j) & 1u)) return;
  if (r < mp.E) mb_cnt[j * mp.E + r] = 0;
  else mb_load[j * mp.D + (r - mp.E)] = 0;
}

}  // namespace

extern "C" eb_status eb_route(eb_ctx* c, void* stream, const eb_batch* batch, uint32_t route_mask,
                              const float* logits, int32_t* topk_idx, float* topk_w, int32_t* mb_load,
                              int32_t* mb_cnt) {
  if (!c) return EB_ERR_INVALID_ARG;
  BatchParams bp;
  eb_status s = ebi_make_batch(c, batch, &bp);
  if (s != EB_OK) return s;
  if (!logits || !topk_idx || !topk_w || !mb_load || !mb_cnt) return ebi_fail(c, EB_ERR_INVALID_ARG, "null pointer");
  if (bp.n_mb < 32 && (route_mask >> bp.n_mb) != 0) return ebi_fail(c, EB_ERR_INVALID_ARG, "route_mask beyond n_mb");
  if (bp.n_mb == 0 || route_mask == 0) return EB_OK;
  cudaStream_t st = (cudaStream_t)stream;
  KernelTimer timer(c, EBK_ROUTE, st);
  int n = bp.n_mb * (c->cfg.E + c->cfg.D);
  ebi_launch(route_clear_kernel, dim3((n + 255) / 256), dim3(256), 0, st, c->mp, bp, route_mask, mb_load, mb_cnt);
  if (bp.n_tok > 0) {
    int blocks = (bp.n_tok + kWarpsPerBlock - 1) / kWarpsPerBlock;
    ebi_launch(route_kernel, dim3(blocks), dim3(kWarpsPerBlock * 32), 0, st, c->mp, bp, route_mask, logits, topk_idx, topk_w,
               mb_load, mb_cnt);
  }
  EB_LAUNCH_CHECK(c, "route");
  return EB_OK;
}
