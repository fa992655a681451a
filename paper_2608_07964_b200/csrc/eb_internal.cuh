// Internal declarations shared by the translation units of libeb (not part of the ABI).
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <string>
#include <vector>

#include "eb.h"

typedef __nv_bfloat16 bf16;

enum { EB_MAX_GUARDS = 24 };

// Kernel ids for the optional per-kernel event timing.
enum EbKernel {
  EBK_ROUTE = 0,
  EBK_SCHEDULE,
  EBK_PERMUTE_HIST,
  EBK_PERMUTE_SIZES,
  EBK_PERMUTE_SCAN,
  EBK_PERMUTE_RANK,
  EBK_PERMUTE_GATHER,
  EBK_FFN_PLAN,
  EBK_FFN_FILL,
  EBK_FFN_GATEUP,
  EBK_FFN_DOWN,
  EBK_COMBINE,
  EBK_PERMUTE_FUSED,
  EBK_COUNT
};

// Micro-batch description passed to kernels by value.
struct BatchParams {
  int32_t n_mb;
  int32_t n_tok;
  int32_t n_chunks;                 // chunks of <= 32 tokens, never straddling a micro-batch
  int32_t tok_off[EB_MAX_MB + 1];
  int32_t layer[EB_MAX_MB];
  int32_t chunk_off[EB_MAX_MB + 1]; // first chunk of every micro-batch
};

// Model description passed to kernels by value.
struct ModelParams {
  int32_t L, E, K, S, H, I, D, renorm;
  const int32_t* e2d;       // [E] expert -> device
  const int32_t* dev_off;   // [D+1] first entry of each device in dev_list
  const int32_t* dev_list;  // [E] routed experts sorted by (device, expert)
  const int32_t* e_local;   // [E] index of the expert among its device's experts
};

struct eb_ctx {
  eb_config cfg;
  int device = 0;
  int num_sms = 0;
  std::vector<int32_t> e2d;
  int32_t* d_tables = nullptr;  // e2d | dev_off | dev_list | e_local
  ModelParams mp;
  int32_t* d_status = nullptr;
  char* d_sched_scratch = nullptr;  // per-block candidates and arrival counter of the multi-block scheduler

  const bf16* w_gate = nullptr;
  const bf16* w_up = nullptr;
  const bf16* w_down = nullptr;
  CUtensorMap tm_gate, tm_up, tm_down;
  int pair_grid = 0;               // CTAs launched for the expert kernels: two per 2-CTA cluster the device holds at once

  // workspace carve-up
  void* ws = nullptr;
  size_t ws_bytes = 0;
  int n_guards = 0;                // guard areas between the regions below (debugging aid)
  size_t guard_off[EB_MAX_GUARDS] = {};
  int32_t* chunk_hist = nullptr;   // [max_chunks][E]
  int32_t* chunk_base = nullptr;   // [max_chunks][E]
  int32_t* group_size = nullptr;   // [G_cap]
  int32_t* pgroup = nullptr;       // [G_cap] group at each position of the processing order
  int32_t* pslots = nullptr;       // [G_cap] 16-row slots of the merged shared-expert class of the position, -1 otherwise
  int4* prank = nullptr;           // [G_cap] (cost class, rank and tiles before it inside the class) when a plan has more than 1024 positions
  int32_t* order = nullptr;        // [G_cap] positions that own tiles, widest tiles first
  int32_t* tile_pref = nullptr;    // [G_cap + 1] tiles before each entry of `order`
  int32_t* work_count = nullptr;   // [16]: tile counts of the two lists, group range, layers, device filter
  int4* work1 = nullptr;           // gate/up tile list
  int4* work2 = nullptr;           // down tile list
  int2* slots = nullptr;           // [16 * max_tiles] (first row, rows) of the 16-row slots of merged tiles
  bf16* act = nullptr;             // [R_cap][I]
  int32_t max_chunks = 0, max_tiles = 0, max_work1 = 0, max_work2 = 0;

  bool fused_attr_set = false;
  // eb_step_host_submit / eb_step_host_wait: copy streams and per-slot events, created on first use
  cudaStream_t s_in = nullptr, s_out = nullptr;
  cudaEvent_t ev_in[EB_HOST_SLOTS] = {}, ev_step[EB_HOST_SLOTS] = {}, ev_out[EB_HOST_SLOTS] = {};
  bool slot_busy[EB_HOST_SLOTS] = {};
  bool timing = false;
  cudaEvent_t ev[2 * EBK_COUNT] = {};
  bool ev_valid[EBK_COUNT] = {};

  std::string err;
};

int32_t ebi_rows_cap(const eb_ctx* c);
int32_t ebi_groups_cap(const eb_ctx* c);
eb_status ebi_fail(eb_ctx* c, eb_status s, const std::string& msg);
eb_status ebi_check_cuda(eb_ctx* c, cudaError_t e, const char* what);
eb_status ebi_make_batch(eb_ctx* c, const eb_batch* b, BatchParams* out);
// EB_OK if the calling thread's current device is the one the context was created on.
eb_status ebi_check_device(eb_ctx* c);

// Brackets a launch with events when timing is enabled.
struct KernelTimer {
  eb_ctx* c;
  int id;
  cudaStream_t s;
  KernelTimer(eb_ctx* ctx, int kid, cudaStream_t st) : c(ctx), id(kid), s(st) {
    if (c->timing) cudaEventRecord(c->ev[2 * id], s);
  }
  ~KernelTimer() {
    if (c->timing) {
      cudaEventRecord(c->ev[2 * id + 1], s);
      c->ev_valid[id] = true;
    }
  }
};

#define EB_CUDA(ctx, expr)                                              \
  do {                                                                  \
    cudaError_t _e = (expr);                                            \
    if (_e != cudaSuccess) return ebi_check_cuda((ctx), _e, #expr);     \
  } while (0)

#define EB_LAUNCH_CHECK(ctx, what)                                      \
  do {                                                                  \
    cudaError_t _e = cudaGetLastError();                                \
    if (_e != cudaSuccess) return ebi_check_cuda((ctx), _e, what);      \
  } while (0)

// Every kernel of the library begins with EB_GRID_DEP_SYNC(): it waits until the kernels before it in
// the stream have finished (and their writes are visible), then lets the kernel after it start being
// scheduled.  With launches made through ebi_launch (programmatic stream serialisation) the launch
// latency of each small kernel overlaps the previous kernel; with ordinary launches it is a no-op.
#define EB_GRID_DEP_SYNC() asm volatile("griddepcontrol.wait;\n\tgriddepcontrol.launch_dependents;" ::: "memory")

// Number of kernels this library has launched in the process (all contexts).
extern std::atomic<unsigned long long> g_ebi_launches;

template <typename... KArgs, typename... Args>
static inline cudaError_t ebi_launch(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                     Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  ++g_ebi_launches;
  return cudaLaunchKernelEx(&cfg, kernel, args...);
}

static inline bool ebi_aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Entry points of the per-step stages (defined in their own translation units).
eb_status ebi_ffn_run(eb_ctx* c, cudaStream_t st, const void* xp, const int32_t* group_off,
                      const int32_t* group_w, const int32_t* step_meta, void* yp, int32_t device);
eb_status ebi_ffn_bind(eb_ctx* c);
eb_status ebi_selftest_wait(eb_ctx* c, cudaStream_t st, long long limit_cycles, int* d_gave_up);
