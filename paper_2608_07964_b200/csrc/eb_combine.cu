// eb_combine: weighted aggregation of Eq. 1 in gather form; optionally the residual of the MoE block,
// h_{l+1} = h'_l + MLP(h'_l) (Section 2.1), in the same pass.
//
// A team of threads per token, one 16-byte column vector each (a whole row in flight at once).  A
// thread loads its vector from the K + S expert-output rows of the token (independent loads, all
// in flight together), accumulates in fp32 in the
// fixed order k = 0..K-1 then s = 0..S-1, and stores bf16 (round to nearest even).  Gather form
// means no atomics and a result that does not depend on scheduling.
#include <utility>

#include "eb_internal.cuh"

namespace {

constexpr int kThreads = 256;
constexpr int kMaxSlots = EB_MAX_K + EB_MAX_S;

__device__ __forceinline__ void fma8(float* acc, const uint4& v, float w) {
  const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float2 f = __bfloat1622float2(h[i]);
    acc[2 * i] = fmaf(w, f.x, acc[2 * i]);
    acc[2 * i + 1] = fmaf(w, f.y, acc[2 * i + 1]);
  }
}

template <int KS>
__global__ void __launch_bounds__(kThreads)
combine_kernel(int n_tok, int H, int K, int team, const uint4* __restrict__ yp, const int32_t* __restrict__ pos,
               const float* __restrict__ topk_w, const uint4* residual, uint4* out) {   // residual may be `out` itself
  EB_GRID_DEP_SYNC();
  const int t = blockIdx.x * (kThreads / team) + threadIdx.x / team;   // team >= 32: a warp serves one token
  if (t >= n_tok) return;
  const int lane = threadIdx.x & 31;
  // lane s fetches slot s once per warp; the values are broadcast with shuffles
  const int my_pos = lane < KS ? pos[(size_t)t * KS + lane] : -1;
  const float my_w = lane < K ? topk_w[(size_t)t * K + lane] : 1.0f;
  if (__shfl_sync(0xffffffffu, my_pos, 0) < 0) return;  // micro-batch did not run: row untouched
  const int vec = H / 8;
  int p[KS];
  float w[KS];
#pragma unroll
  for (int s = 0; s < KS; ++s) {
    p[s] = __shfl_sync(0xffffffffu, my_pos, s);
    w[s] = __shfl_sync(0xffffffffu, my_w, s);
  }
  for (int v = threadIdx.x % team; v < vec; v += team) {
    uint4 r[KS];
#pragma unroll
    for (int s = 0; s < KS; ++s) r[s] = p[s] >= 0 ? __ldg(yp + (size_t)p[s] * vec + v) : make_uint4(0, 0, 0, 0);   // no row: adds 0
    uint4 res = make_uint4(0, 0, 0, 0);
    if (residual) res = residual[(size_t)t * vec + v];
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int s = 0; s < KS; ++s) fma8(acc, r[s], w[s]);
    if (residual) {   // added last: out = sum + h'
      const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&res);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float2 f = __bfloat1622float2(h[i]);
        acc[2 * i] += f.x;
        acc[2 * i + 1] += f.y;
      }
    }
    uint4 o;
    __nv_bfloat162* oh = reinterpret_cast<__nv_bfloat162*>(&o);
#pragma unroll
    for (int i = 0; i < 4; ++i) oh[i] = __floats2bfloat162_rn(acc[2 * i], acc[2 * i + 1]);
    out[(size_t)t * vec + v] = o;
  }
}

typedef void (*combine_fn)(int, int, int, int, const uint4*, const int32_t*, const float*, const uint4*, uint4*);

// kernel for every slot count 1 .. kMaxSlots (entry 0 unused)
template <int... Is>
const combine_fn* combine_table(std::integer_sequence<int, Is...>) {
  static const combine_fn table[] = {nullptr, combine_kernel<Is + 1>...};
  return table;
}

}  // namespace

extern "C" eb_status eb_combine(eb_ctx* c, void* stream, const eb_batch* batch, const eb_sched_result* d_res,
                                const void* yp, const int32_t* pos, const float* topk_w, void* out) {
  return eb_combine_residual(c, stream, batch, d_res, yp, pos, topk_w, nullptr, out);
}

extern "C" eb_status eb_combine_residual(eb_ctx* c, void* stream, const eb_batch* batch, const eb_sched_result* d_res,
                                         const void* yp, const int32_t* pos, const float* topk_w, const void* residual,
                                         void* out) {
  if (!c) return EB_ERR_INVALID_ARG;
  BatchParams bp;
  eb_status s = ebi_make_batch(c, batch, &bp);
  if (s != EB_OK) return s;
  if (!d_res || !yp || !pos || !topk_w || !out) return ebi_fail(c, EB_ERR_INVALID_ARG, "null pointer");
  if (!ebi_aligned16(yp) || !ebi_aligned16(out) || !ebi_aligned16(residual))
    return ebi_fail(c, EB_ERR_INVALID_ARG, "yp / out / residual must be 16-byte aligned");
  if (bp.n_tok == 0) return EB_OK;
  const combine_fn* table = combine_table(std::make_integer_sequence<int, kMaxSlots>());
  cudaStream_t st = (cudaStream_t)stream;
  const int KS = c->cfg.K + c->cfg.S;
  KernelTimer timer(c, EBK_COMBINE, st);
  const int vec = c->cfg.H / 8;
  const int team = vec <= 32 ? 32 : vec <= 64 ? 64 : vec <= 128 ? 128 : 256, tpb = kThreads / team;
  ebi_launch(table[KS], dim3((bp.n_tok + tpb - 1) / tpb), dim3(kThreads), 0, st, bp.n_tok, c->cfg.H, c->cfg.K, team,
             (const uint4*)yp, pos, topk_w, (const uint4*)residual, (uint4*)out);
  EB_LAUNCH_CHECK(c, "combine");
  return EB_OK;
}
