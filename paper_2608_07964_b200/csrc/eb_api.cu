// Context life cycle, argument checking, workspace carve-up, whole-step wrappers.
#include <algorithm>
#include <cstdio>
#include <cstring>
#include <new>

#include "eb_internal.cuh"

std::atomic<unsigned long long> g_ebi_launches{0};

extern "C" uint64_t eb_launch_count(void) { return g_ebi_launches.load(); }

int32_t ebi_rows_cap(const eb_ctx* c) { return c->cfg.max_tokens * (c->cfg.K + c->cfg.S); }
int32_t ebi_groups_cap(const eb_ctx* c) { return EB_MAX_MB * (c->cfg.E + c->cfg.D * c->cfg.S); }

eb_status ebi_fail(eb_ctx* c, eb_status s, const std::string& msg) {
  if (c) c->err = msg;
  return s;
}

eb_status ebi_check_cuda(eb_ctx* c, cudaError_t e, const char* what) {
  if (e == cudaSuccess) return EB_OK;
  std::string m = std::string(what) + ": " + cudaGetErrorString(e);
  return ebi_fail(c, EB_ERR_CUDA, m);
}

eb_status ebi_check_device(eb_ctx* c) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return ebi_fail(c, EB_ERR_CUDA, "cudaGetDevice failed");
  if (dev != c->device) return ebi_fail(c, EB_ERR_INVALID_ARG, "the context was created on another device than the current one");
  return EB_OK;
}

eb_status ebi_make_batch(eb_ctx* c, const eb_batch* b, BatchParams* out) {
  eb_status ds = ebi_check_device(c);
  if (ds != EB_OK) return ds;
  if (!b || !b->tok_off || !b->layer) return ebi_fail(c, EB_ERR_INVALID_ARG, "null batch");
  if (b->n_mb < 0 || b->n_mb > EB_MAX_MB) return ebi_fail(c, EB_ERR_UNSUPPORTED, "n_mb out of range");
  if (b->n_mb < 32 && (b->pool_mask >> b->n_mb) != 0)
    return ebi_fail(c, EB_ERR_INVALID_ARG, "pool_mask has bits beyond n_mb");
  if (b->tok_off[0] != 0) return ebi_fail(c, EB_ERR_INVALID_ARG, "tok_off[0] must be 0");
  BatchParams p;
  memset(&p, 0, sizeof(p));
  p.n_mb = b->n_mb;
  int chunks = 0;
  for (int j = 0; j < b->n_mb; ++j) {
    int t0 = b->tok_off[j], t1 = b->tok_off[j + 1];
    if (t1 < t0) return ebi_fail(c, EB_ERR_INVALID_ARG, "tok_off must be ascending");
    if (b->layer[j] < 0 || b->layer[j] >= c->cfg.L) return ebi_fail(c, EB_ERR_INVALID_ARG, "layer out of range");
    p.tok_off[j] = t0;
    p.layer[j] = b->layer[j];
    p.chunk_off[j] = chunks;
    chunks += (t1 - t0 + 31) / 32;
  }
  p.tok_off[b->n_mb] = b->tok_off[b->n_mb];
  p.chunk_off[b->n_mb] = chunks;
  for (int j = b->n_mb + 1; j <= EB_MAX_MB; ++j) {
    p.tok_off[j] = p.tok_off[b->n_mb];
    p.chunk_off[j] = chunks;
  }
  p.n_tok = p.tok_off[b->n_mb];
  p.n_chunks = chunks;
  if (p.n_tok > c->cfg.max_tokens) return ebi_fail(c, EB_ERR_INVALID_ARG, "more tokens than max_tokens");
  *out = p;
  return EB_OK;
}

static size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

constexpr size_t kGuardBytes = 256;
constexpr int kGuardByte = 0xA5;

// Lays the workspace regions out; with base == nullptr only the total size is computed.
static size_t carve(eb_ctx* c, char* base) {
  const eb_config& g = c->cfg;
  size_t off = 0;
  c->n_guards = 0;
  auto take = [&](size_t bytes) {
    char* p = base ? base + off : nullptr;
    off = align_up(off + bytes, 256);
    // a guard of kGuardBytes after every region: filled with a pattern by eb_set_workspace, never written by any
    // kernel, checked by eb_check_workspace_guards
    if (c->n_guards < EB_MAX_GUARDS) c->guard_off[c->n_guards++] = off;
    off += kGuardBytes;
    return p;
  };
  c->max_chunks = (g.max_tokens + 31) / 32 + EB_MAX_MB;
  int rows = ebi_rows_cap(c), gcap = ebi_groups_cap(c);
  c->max_tiles = rows / 256 + gcap;                    // a group of r rows has ceil(r / 256) tiles
  c->max_work1 = c->max_tiles * ((g.I + 255) / 256);   // 256 outputs per gate/up tile
  c->max_work2 = c->max_tiles * ((g.H + 511) / 512);   // 512 outputs per down tile
  c->chunk_hist = (int32_t*)take(sizeof(int32_t) * (size_t)c->max_chunks * g.E);
  c->chunk_base = (int32_t*)take(sizeof(int32_t) * (size_t)c->max_chunks * g.E);
  c->group_size = (int32_t*)take(sizeof(int32_t) * (size_t)gcap);
  c->pgroup = (int32_t*)take(sizeof(int32_t) * (size_t)gcap);
  c->pslots = (int32_t*)take(sizeof(int32_t) * (size_t)gcap);
  c->prank = (int4*)take(sizeof(int4) * (size_t)gcap);
  c->order = (int32_t*)take(sizeof(int32_t) * (size_t)gcap);
  c->tile_pref = (int32_t*)take(sizeof(int32_t) * (size_t)(gcap + 1));
  c->work_count = (int32_t*)take(sizeof(int32_t) * 16);
  c->work1 = (int4*)take(sizeof(int4) * (size_t)c->max_work1);
  c->work2 = (int4*)take(sizeof(int4) * (size_t)c->max_work2);
  c->slots = (int2*)take(sizeof(int2) * 16 * (size_t)c->max_tiles);
  c->act = (bf16*)take(sizeof(bf16) * (size_t)rows * g.I);
  return off;
}

extern "C" eb_status eb_create(const eb_config* cfg, eb_ctx** out) {
  if (!cfg || !out || !cfg->expert_to_device) return EB_ERR_INVALID_ARG;
  *out = nullptr;
  const eb_config& g = *cfg;
  if (g.L < 1 || g.E < 1 || g.E > EB_MAX_E || g.K < 1 || g.K > EB_MAX_K || g.K > g.E || g.S < 0 ||
      g.S > EB_MAX_S || g.D < 1 || g.D > EB_MAX_D || g.H < 8 || g.I < 8 || (g.H % 8) || (g.I % 8) ||
      g.max_tokens < 1)
    return EB_ERR_UNSUPPORTED;
  if ((int64_t)g.max_tokens * (g.K + g.S) > (int64_t)1 << 30) return EB_ERR_UNSUPPORTED;
  for (int e = 0; e < g.E; ++e)
    if (g.expert_to_device[e] < 0 || g.expert_to_device[e] >= g.D) return EB_ERR_INVALID_ARG;

  eb_ctx* c = new (std::nothrow) eb_ctx();
  if (!c) return EB_ERR_CUDA;
  c->cfg = g;
  c->e2d.assign(g.expert_to_device, g.expert_to_device + g.E);
  c->cfg.expert_to_device = c->e2d.data();
  cudaDeviceProp prop;
  if (cudaGetDevice(&c->device) != cudaSuccess || cudaGetDeviceProperties(&prop, c->device) != cudaSuccess ||
      prop.major != 10) {
    delete c;
    return EB_ERR_CUDA;
  }
  c->num_sms = prop.multiProcessorCount;

  // host tables: experts sorted by (device, expert)
  std::vector<int32_t> tab(3 * g.E + g.D + 1);
  int32_t* h_e2d = tab.data();
  int32_t* h_off = h_e2d + g.E;
  int32_t* h_list = h_off + g.D + 1;
  int32_t* h_local = h_list + g.E;
  int n = 0;
  for (int d = 0; d < g.D; ++d) {
    h_off[d] = n;
    for (int e = 0; e < g.E; ++e)
      if (c->e2d[e] == d) {
        h_local[e] = n - h_off[d];
        h_list[n++] = e;
      }
  }
  h_off[g.D] = n;
  std::copy(c->e2d.begin(), c->e2d.end(), h_e2d);
  bool ok = cudaMalloc(&c->d_tables, tab.size() * sizeof(int32_t)) == cudaSuccess &&
            cudaMemcpy(c->d_tables, tab.data(), tab.size() * sizeof(int32_t), cudaMemcpyHostToDevice) == cudaSuccess &&
            cudaMalloc(&c->d_status, sizeof(int32_t)) == cudaSuccess &&
            cudaMemset(c->d_status, 0, sizeof(int32_t)) == cudaSuccess &&
            cudaMalloc(&c->d_sched_scratch, 4096) == cudaSuccess &&
            cudaMemset(c->d_sched_scratch, 0, 4096) == cudaSuccess;
  for (int i = 0; ok && i < 2 * EBK_COUNT; ++i) ok = cudaEventCreate(&c->ev[i]) == cudaSuccess;
  if (!ok) {
    eb_destroy(c);
    return EB_ERR_CUDA;
  }
  ModelParams& mp = c->mp;
  mp.L = g.L; mp.E = g.E; mp.K = g.K; mp.S = g.S; mp.H = g.H; mp.I = g.I; mp.D = g.D;
  mp.renorm = g.renorm_topk ? 1 : 0;
  mp.e2d = c->d_tables;
  mp.dev_off = c->d_tables + g.E;
  mp.dev_list = mp.dev_off + g.D + 1;
  mp.e_local = mp.dev_list + g.E;
  carve(c, nullptr);
  *out = c;
  return EB_OK;
}

extern "C" eb_status eb_destroy(eb_ctx* c) {
  if (!c) return EB_ERR_INVALID_ARG;
  if (c->d_tables) cudaFree(c->d_tables);
  if (c->d_status) cudaFree(c->d_status);
  if (c->d_sched_scratch) cudaFree(c->d_sched_scratch);
  for (int i = 0; i < 2 * EBK_COUNT; ++i)
    if (c->ev[i]) cudaEventDestroy(c->ev[i]);
  for (int i = 0; i < EB_HOST_SLOTS; ++i) {
    if (c->ev_in[i]) cudaEventDestroy(c->ev_in[i]);
    if (c->ev_step[i]) cudaEventDestroy(c->ev_step[i]);
    if (c->ev_out[i]) cudaEventDestroy(c->ev_out[i]);
  }
  if (c->s_in) cudaStreamDestroy(c->s_in);
  if (c->s_out) cudaStreamDestroy(c->s_out);
  delete c;
  return EB_OK;
}

extern "C" eb_status eb_bind_weights(eb_ctx* c, const void* w_gate, const void* w_up, const void* w_down) {
  if (!c) return EB_ERR_INVALID_ARG;
  if (!w_gate || !w_up || !w_down) return ebi_fail(c, EB_ERR_INVALID_ARG, "null weights");
  if (!ebi_aligned16(w_gate) || !ebi_aligned16(w_up) || !ebi_aligned16(w_down))
    return ebi_fail(c, EB_ERR_INVALID_ARG, "weights must be 16-byte aligned");
  c->w_gate = (const bf16*)w_gate;
  c->w_up = (const bf16*)w_up;
  c->w_down = (const bf16*)w_down;
  eb_status s = ebi_ffn_bind(c);
  if (s != EB_OK) c->w_gate = c->w_up = c->w_down = nullptr;
  return s;
}

extern "C" size_t eb_workspace_bytes(const eb_ctx* c) {
  if (!c) return 0;
  eb_ctx tmp;
  tmp.cfg = c->cfg;
  return carve(&tmp, nullptr);
}

extern "C" eb_status eb_set_workspace(eb_ctx* c, void* dev_ptr, size_t bytes) {
  if (!c) return EB_ERR_INVALID_ARG;
  if (!dev_ptr || (reinterpret_cast<uintptr_t>(dev_ptr) & 255u))
    return ebi_fail(c, EB_ERR_INVALID_ARG, "workspace must be a 256-byte aligned device pointer");
  if (bytes < eb_workspace_bytes(c)) return ebi_fail(c, EB_ERR_WORKSPACE, "workspace too small");
  c->ws = dev_ptr;
  c->ws_bytes = bytes;
  carve(c, (char*)dev_ptr);
  for (int i = 0; i < c->n_guards; ++i)
    EB_CUDA(c, cudaMemset((char*)dev_ptr + c->guard_off[i], kGuardByte, kGuardBytes));
  return EB_OK;
}

extern "C" int32_t eb_rows_capacity(const eb_ctx* c) { return c ? ebi_rows_cap(c) : 0; }
extern "C" int32_t eb_groups_capacity(const eb_ctx* c) { return c ? ebi_groups_cap(c) : 0; }

extern "C" eb_status eb_expert_ffn_grouped(eb_ctx* c, void* stream, const void* xp, const int32_t* group_off,
                                           const int32_t* group_w, const int32_t* step_meta, void* yp) {
  if (!c) return EB_ERR_INVALID_ARG;
  return ebi_ffn_run(c, (cudaStream_t)stream, xp, group_off, group_w, step_meta, yp, -1);
}

extern "C" eb_status eb_expert_ffn_device(eb_ctx* c, void* stream, const void* xp, const int32_t* group_off,
                                          const int32_t* group_w, const int32_t* step_meta, void* yp,
                                          int32_t device) {
  if (!c) return EB_ERR_INVALID_ARG;
  if (device < 0 || device >= c->cfg.D) return ebi_fail(c, EB_ERR_INVALID_ARG, "device out of range");
  return ebi_ffn_run(c, (cudaStream_t)stream, xp, group_off, group_w, step_meta, yp, device);
}

static eb_status check_buffers(eb_ctx* c, const eb_step_buffers* b) {
  if (!b) return ebi_fail(c, EB_ERR_INVALID_ARG, "null buffers");
  const void* p[] = {b->logits, b->x, b->topk_idx, b->topk_w, b->mb_load, b->mb_cnt, b->sched, b->group_off,
                     b->group_w, b->row_src, b->pos, b->xp, b->yp, b->step_meta, b->out};
  for (const void* q : p)
    if (!q || !ebi_aligned16(q)) return ebi_fail(c, EB_ERR_INVALID_ARG, "step buffer null or not 16-byte aligned");
  return EB_OK;
}

extern "C" eb_status eb_step(eb_ctx* c, void* stream, const eb_batch* batch, uint32_t route_mask, int32_t m,
                             eb_policy policy, const eb_step_buffers* b) {
  if (!c) return EB_ERR_INVALID_ARG;
  eb_status s = check_buffers(c, b);
  if (s != EB_OK) return s;
  if ((s = eb_route(c, stream, batch, route_mask, b->logits, b->topk_idx, b->topk_w, b->mb_load, b->mb_cnt)) != EB_OK) return s;
  if ((s = eb_schedule(c, stream, batch, m, policy, b->mb_load, b->sched, nullptr)) != EB_OK) return s;
  if ((s = eb_permute(c, stream, batch, b->sched, b->x, b->topk_idx, b->group_off, b->group_w, b->row_src, b->pos,
                      b->xp, b->step_meta)) != EB_OK) return s;
  if ((s = eb_expert_ffn_grouped(c, stream, b->xp, b->group_off, b->group_w, b->step_meta, b->yp)) != EB_OK) return s;
  if (!ebi_aligned16(b->residual)) return ebi_fail(c, EB_ERR_INVALID_ARG, "residual not 16-byte aligned");
  return eb_combine_residual(c, stream, batch, b->sched, b->yp, b->pos, b->topk_w, b->residual, b->out);
}

extern "C" eb_status eb_step_host(eb_ctx* c, void* stream, const eb_batch* batch, uint32_t route_mask, int32_t m,
                                  eb_policy policy, const eb_step_buffers* b, const float* h_logits,
                                  const void* h_x, void* h_out, eb_sched_result* h_res) {
  if (!c) return EB_ERR_INVALID_ARG;
  if (!h_logits || !h_x || !h_out) return ebi_fail(c, EB_ERR_INVALID_ARG, "null host buffer");
  eb_status s = check_buffers(c, b);
  if (s != EB_OK) return s;
  BatchParams bp;
  if ((s = ebi_make_batch(c, batch, &bp)) != EB_OK) return s;
  cudaStream_t st = (cudaStream_t)stream;
  size_t T = (size_t)bp.n_tok;
  if (T) {
    EB_CUDA(c, cudaMemcpyAsync(b->logits, h_logits, T * c->cfg.E * sizeof(float), cudaMemcpyHostToDevice, st));
    EB_CUDA(c, cudaMemcpyAsync(b->x, h_x, T * c->cfg.H * sizeof(bf16), cudaMemcpyHostToDevice, st));
  }
  if ((s = eb_step(c, stream, batch, route_mask, m, policy, b)) != EB_OK) return s;
  if (T) EB_CUDA(c, cudaMemcpyAsync(h_out, b->out, T * c->cfg.H * sizeof(bf16), cudaMemcpyDeviceToHost, st));
  if (h_res) EB_CUDA(c, cudaMemcpyAsync(h_res, b->sched, sizeof(eb_sched_result), cudaMemcpyDeviceToHost, st));
  EB_CUDA(c, cudaStreamSynchronize(st));
  return EB_OK;
}

static eb_status host_pipeline_init(eb_ctx* c) {
  if (c->s_in) return EB_OK;
  EB_CUDA(c, cudaStreamCreateWithFlags(&c->s_in, cudaStreamNonBlocking));
  EB_CUDA(c, cudaStreamCreateWithFlags(&c->s_out, cudaStreamNonBlocking));
  for (int i = 0; i < EB_HOST_SLOTS; ++i) {
    EB_CUDA(c, cudaEventCreateWithFlags(&c->ev_in[i], cudaEventDisableTiming));
    EB_CUDA(c, cudaEventCreateWithFlags(&c->ev_step[i], cudaEventDisableTiming));
    EB_CUDA(c, cudaEventCreateWithFlags(&c->ev_out[i], cudaEventDisableTiming));
  }
  return EB_OK;
}

extern "C" eb_status eb_step_host_submit(eb_ctx* c, void* stream, const eb_batch* batch, uint32_t route_mask, int32_t m,
                                         eb_policy policy, const eb_step_buffers* b, const float* h_logits,
                                         const void* h_x, void* h_out, eb_sched_result* h_res, int32_t slot) {
  if (!c) return EB_ERR_INVALID_ARG;
  if (slot < 0 || slot >= EB_HOST_SLOTS) return ebi_fail(c, EB_ERR_INVALID_ARG, "slot out of range");
  if (c->slot_busy[slot]) return ebi_fail(c, EB_ERR_INVALID_ARG, "slot still in flight: call eb_step_host_wait first");
  if (!h_logits || !h_x || !h_out) return ebi_fail(c, EB_ERR_INVALID_ARG, "null host buffer");
  eb_status s = check_buffers(c, b);
  if (s != EB_OK) return s;
  BatchParams bp;
  if ((s = ebi_make_batch(c, batch, &bp)) != EB_OK) return s;
  if ((s = host_pipeline_init(c)) != EB_OK) return s;
  cudaStream_t st = (cudaStream_t)stream;
  const size_t T = (size_t)bp.n_tok;
  if (T) {
    EB_CUDA(c, cudaMemcpyAsync(b->logits, h_logits, T * c->cfg.E * sizeof(float), cudaMemcpyHostToDevice, c->s_in));
    EB_CUDA(c, cudaMemcpyAsync(b->x, h_x, T * c->cfg.H * sizeof(bf16), cudaMemcpyHostToDevice, c->s_in));
  }
  EB_CUDA(c, cudaEventRecord(c->ev_in[slot], c->s_in));
  EB_CUDA(c, cudaStreamWaitEvent(st, c->ev_in[slot], 0));
  if ((s = eb_step(c, stream, batch, route_mask, m, policy, b)) != EB_OK) return s;
  EB_CUDA(c, cudaEventRecord(c->ev_step[slot], st));
  EB_CUDA(c, cudaStreamWaitEvent(c->s_out, c->ev_step[slot], 0));
  if (T) EB_CUDA(c, cudaMemcpyAsync(h_out, b->out, T * c->cfg.H * sizeof(bf16), cudaMemcpyDeviceToHost, c->s_out));
  if (h_res) EB_CUDA(c, cudaMemcpyAsync(h_res, b->sched, sizeof(eb_sched_result), cudaMemcpyDeviceToHost, c->s_out));
  EB_CUDA(c, cudaEventRecord(c->ev_out[slot], c->s_out));
  c->slot_busy[slot] = true;
  return EB_OK;
}

extern "C" eb_status eb_step_host_wait(eb_ctx* c, int32_t slot) {
  if (!c) return EB_ERR_INVALID_ARG;
  if (slot < 0 || slot >= EB_HOST_SLOTS) return ebi_fail(c, EB_ERR_INVALID_ARG, "slot out of range");
  if (!c->slot_busy[slot]) return EB_OK;
  c->slot_busy[slot] = false;
  EB_CUDA(c, cudaEventSynchronize(c->ev_out[slot]));
  return EB_OK;
}

extern "C" eb_status eb_device_status(eb_ctx* c, int32_t* out_status) {
  if (!c || !out_status) return EB_ERR_INVALID_ARG;
  EB_CUDA(c, cudaDeviceSynchronize());
  EB_CUDA(c, cudaMemcpy(out_status, c->d_status, sizeof(int32_t), cudaMemcpyDeviceToHost));
  EB_CUDA(c, cudaMemset(c->d_status, 0, sizeof(int32_t)));
  return EB_OK;
}

namespace {
struct GuardList {
  int n;
  unsigned long long off[EB_MAX_GUARDS];
};
__global__ void check_guards_kernel(const unsigned char* ws, GuardList g, int* bad) {
  int n = 0;
  for (int i = 0; i < g.n; ++i)
    for (int b = threadIdx.x; b < (int)kGuardBytes; b += blockDim.x)
      if (ws[g.off[i] + b] != (unsigned char)kGuardByte) ++n;
  if (n) atomicAdd(bad, n);
}
}  // namespace

extern "C" eb_status eb_check_workspace_guards(eb_ctx* c, void* stream, int32_t* out_bad) {
  if (!c || !out_bad) return EB_ERR_INVALID_ARG;
  if (eb_status ds = ebi_check_device(c)) return ds;
  if (!c->ws) return ebi_fail(c, EB_ERR_WORKSPACE, "no workspace set");
  cudaStream_t st = (cudaStream_t)stream;
  GuardList g;
  g.n = c->n_guards;
  for (int i = 0; i < c->n_guards; ++i) g.off[i] = c->guard_off[i];
  int* d_bad = c->work_count + 14;   // scratch word of the workspace
  EB_CUDA(c, cudaMemsetAsync(d_bad, 0, sizeof(int), st));
  check_guards_kernel<<<1, 256, 0, st>>>((const unsigned char*)c->ws, g, d_bad);
  EB_LAUNCH_CHECK(c, "check_workspace_guards");
  EB_CUDA(c, cudaMemcpyAsync(out_bad, d_bad, sizeof(int32_t), cudaMemcpyDeviceToHost, st));
  EB_CUDA(c, cudaStreamSynchronize(st));
  return EB_OK;
}

extern "C" eb_status eb_selftest_bounded_wait(eb_ctx* c, void* stream, int64_t limit_cycles, int32_t* out_gave_up) {
  if (!c || !out_gave_up) return EB_ERR_INVALID_ARG;
  if (limit_cycles < 1 || limit_cycles > 2000000000LL) return ebi_fail(c, EB_ERR_INVALID_ARG, "limit_cycles out of range");
  if (!c->ws) return ebi_fail(c, EB_ERR_WORKSPACE, "no workspace set");
  cudaStream_t st = (cudaStream_t)stream;
  int* d_flag = c->work_count + 15;   // scratch word of the workspace
  eb_status s = ebi_selftest_wait(c, st, limit_cycles, d_flag);
  if (s != EB_OK) return s;
  EB_CUDA(c, cudaMemcpyAsync(out_gave_up, d_flag, sizeof(int32_t), cudaMemcpyDeviceToHost, st));
  EB_CUDA(c, cudaStreamSynchronize(st));
  return EB_OK;
}

static const char* kKernelNames[EBK_COUNT] = {
    "route", "schedule", "permute_hist", "permute_sizes", "permute_scan", "permute_rank",
    "permute_gather", "ffn_plan", "ffn_fill", "ffn_gateup", "ffn_down", "combine", "permute_fused"};

extern "C" int32_t eb_num_kernels(void) { return EBK_COUNT; }
extern "C" const char* eb_kernel_name(int32_t i) { return (i >= 0 && i < EBK_COUNT) ? kKernelNames[i] : ""; }

extern "C" eb_status eb_set_timing(eb_ctx* c, int32_t enabled) {
  if (!c) return EB_ERR_INVALID_ARG;
  c->timing = enabled != 0;
  for (int i = 0; i < EBK_COUNT; ++i) c->ev_valid[i] = false;
  return EB_OK;
}

extern "C" eb_status eb_kernel_ms(eb_ctx* c, float* ms) {
  if (!c || !ms) return EB_ERR_INVALID_ARG;
  for (int i = 0; i < EBK_COUNT; ++i) {
    ms[i] = -1.f;
    if (!c->ev_valid[i]) continue;
    EB_CUDA(c, cudaEventSynchronize(c->ev[2 * i + 1]));
    EB_CUDA(c, cudaEventElapsedTime(&ms[i], c->ev[2 * i], c->ev[2 * i + 1]));
  }
  return EB_OK;
}

extern "C" const char* eb_status_string(eb_status s) {
  switch (s) {
    case EB_OK: return "ok";
    case EB_ERR_INVALID_ARG: return "invalid argument";
    case EB_ERR_UNSUPPORTED: return "unsupported shape";
    case EB_ERR_WORKSPACE: return "workspace missing or too small";
    case EB_ERR_CUDA: return "CUDA error";
    case EB_ERR_TIMEOUT: return "device-side wait timed out";
  }
  return "unknown";
}

extern "C" const char* eb_last_error(const eb_ctx* c) { return c ? c->err.c_str() : ""; }
