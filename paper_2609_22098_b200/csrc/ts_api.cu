// Context management, workspace sizing and error strings of the TreeSpark C ABI.
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "ts_internal.h"
#include "ts_tc.cuh"

namespace ts {

static thread_local char g_err[512] = "no error";

int32_t set_error(int32_t code, const char* msg) {
  snprintf(g_err, sizeof(g_err), "%s", msg);
  return code;
}

int32_t set_cuda_error(const char* where, cudaError_t e) {
  snprintf(g_err, sizeof(g_err), "%s: CUDA error %d (%s)", where, (int)e, cudaGetErrorString(e));
  return TS_ERR_CUDA;
}

// Vocabulary tiling of the scoring kernel: the W tile [r][TV] stays in shared memory next to the
// per-thread head rows [r][threads] and the noise-bound table; the tile count is a whole number of
// waves over the SMs.
static bool choose_tile(const ts_config& c, int num_sms, int max_smem, TileCfg* out) {
  const size_t es = c.dt_W == TS_DTYPE_BF16 ? 2 : 4;
  const size_t fixed = (size_t)c.r * SCORE_THREADS * 4 + 512 * 4;  // head rows + both noise-bound tables
  const size_t budget = (size_t)max_smem > fixed + 1024 ? (size_t)max_smem - fixed - 1024 : 0;
  int tv_max = (int)(budget / ((size_t)c.r * es) / 64) * 64;
  if (tv_max < 64) return false;
  if (tv_max > 4096) tv_max = 4096;
  const int min_tiles = (c.V + tv_max - 1) / tv_max;
  const int waves = (min_tiles + num_sms - 1) / num_sms;
  const int want = waves * num_sms;
  int tv = ((c.V + want - 1) / want + 63) / 64 * 64;
  if (tv > tv_max) tv = tv_max;
  out->TV = tv;
  out->ntiles = (c.V + tv - 1) / tv;
  out->smem = (size_t)c.r * tv * es + fixed;
  return out->ntiles <= 32 * 16;
}

// Which kernels serve this configuration (and with which wait limits), from the configuration, the
// device and the test switches.  False: no vocabulary tiling fits shared memory.
static bool select_paths(ts_ctx* ctx) {
  const ts_config& c = ctx->cfg;
  const unsigned tm = ctx->test_mode;
  // tensor cores for bf16 inputs whose rows allow 16-byte chunks; the fp32 FMA kernel otherwise
  ctx->use_mma = (c.dt_U == TS_DTYPE_BF16 && c.r % 8 == 0 && c.V % 8 == 0 && ctx->cc_major == 10 && !(tm & TS_TEST_FORCE_FMA)) ? 1 : 0;
  ctx->tma_state = (tm & TS_TEST_NO_TMA) ? -1 : 0;
  ctx->tmapW_ptr = nullptr;
  if (ctx->use_mma && !choose_tile_mma(c, ctx->num_sms, ctx->max_smem, !(tm & TS_TEST_NO_TMA), &ctx->tile)) ctx->use_mma = 0;
  if (!ctx->use_mma && !choose_tile(c, ctx->num_sms, ctx->max_smem, &ctx->tile)) return false;
  ctx->few_ok = (few_supported(ctx) && !(tm & TS_TEST_NO_FEW)) ? 1 : 0;
  ctx->wait_limit = (tm & TS_TEST_SHORT_WAITS) ? 4096u : WAIT_LIMIT;
  return true;
}

}  // namespace ts

using namespace ts;

extern "C" const char* ts_last_error_string(void) { return g_err; }

extern "C" int32_t ts_create(const ts_config* cfg, ts_ctx** out) {
  if (!cfg || !out) return set_error(TS_ERR_INVALID, "ts_create: null argument");
  *out = nullptr;
  if (cfg->V < 1 || cfg->D < 1 || cfg->r < 1 || cfg->K < 1 || cfg->Nmax < 1 || cfg->max_batch < 1)
    return set_error(TS_ERR_INVALID, "ts_create: sizes must be positive");
  if (cfg->K > TS_KMAX || cfg->D > TS_DMAX || cfg->Nmax > 256 || cfg->r > RMAX || cfg->max_batch > 4096 ||
      cfg->V > (1 << 24))
    return set_error(TS_ERR_UNSUPPORTED, "ts_create: K<=16, D<=16, Nmax<=256, r<=256, batch<=4096, V<=2^24 required");
  if (cfg->dt_U != cfg->dt_A || cfg->dt_U != cfg->dt_W || cfg->dt_U != cfg->dt_Z ||
      (cfg->dt_U != TS_DTYPE_F32 && cfg->dt_U != TS_DTYPE_BF16))
    return set_error(TS_ERR_UNSUPPORTED, "ts_create: U, A, W, Z must share one dtype (f32 or bf16)");
  if (cfg->calib_mode != 0 && cfg->calib_mode != 1) return set_error(TS_ERR_INVALID, "ts_create: calib_mode");
  if (cfg->calib_mode == 1) {
    if (!cfg->calib_table || !(cfg->calib_hi > cfg->calib_lo))
      return set_error(TS_ERR_INVALID, "ts_create: table mode needs calib_table and calib_hi > calib_lo");
    for (int d = 0; d < cfg->D; ++d)
      for (int i = 0; i < TS_CALIB_KNOTS; ++i) {
        const float y = cfg->calib_table[d * TS_CALIB_KNOTS + i];
        if (!(y > 0.f && y <= 1.f) || (i && y < cfg->calib_table[d * TS_CALIB_KNOTS + i - 1]))
          return set_error(TS_ERR_INVALID, "ts_create: calibration table must be non-decreasing in (0,1]");
      }
  }
  ts_ctx* ctx = new ts_ctx();
  ctx->cfg = *cfg;
  ctx->cfg.calib_table = nullptr;
  ctx->d_table = nullptr;
  ctx->prof = new Prof();
  ctx->ablation = 0;
  cudaError_t e = cudaGetDevice(&ctx->device);
  cudaDeviceProp prop;
  if (e == cudaSuccess) e = cudaGetDeviceProperties(&prop, ctx->device);
  if (e != cudaSuccess) { delete (Prof*)ctx->prof; delete ctx; return set_cuda_error("ts_create", e); }
  ctx->num_sms = prop.multiProcessorCount;
  ctx->max_smem = (int)prop.sharedMemPerBlockOptin;
  ctx->cc_major = prop.major;
  ctx->test_mode = 0;
  if (!select_paths(ctx)) {
    delete (Prof*)ctx->prof; delete ctx;
    return set_error(TS_ERR_UNSUPPORTED, "ts_create: no vocabulary tiling fits shared memory");
  }
  ctx->vt_TV = ((cfg->V + ctx->num_sms - 1) / ctx->num_sms + 63) / 64 * 64;
  ctx->vt_n = (cfg->V + ctx->vt_TV - 1) / ctx->vt_TV;
  if (cfg->calib_mode == 1) {
    const size_t bytes = (size_t)cfg->D * TS_CALIB_KNOTS * sizeof(float);
    e = cudaMalloc(&ctx->d_table, bytes);
    if (e == cudaSuccess) e = cudaMemcpy(ctx->d_table, cfg->calib_table, bytes, cudaMemcpyHostToDevice);
    if (e != cudaSuccess) { cudaFree(ctx->d_table); delete (Prof*)ctx->prof; delete ctx; return set_cuda_error("ts_create", e); }
  }
  ctx->calib.mode = cfg->calib_mode;
  ctx->calib.a = cfg->platt_a; ctx->calib.b = cfg->platt_b;
  ctx->calib.lo = cfg->calib_lo; ctx->calib.hi = cfg->calib_hi;
  ctx->calib.table = ctx->d_table;
  e = score_setup(ctx);
  if (e == cudaSuccess) e = verify_setup(ctx);
  if (e == cudaSuccess) e = expand_setup(ctx);
  if (e != cudaSuccess) { cudaFree(ctx->d_table); delete (Prof*)ctx->prof; delete ctx; return set_cuda_error("ts_create", e); }
  *out = ctx;
  return TS_OK;
}

extern "C" int32_t ts_destroy(ts_ctx* ctx) {
  if (!ctx) return TS_OK;
  if (ctx->d_table) cudaFree(ctx->d_table);
  Prof* p = (Prof*)ctx->prof;
  if (p) { for (cudaEvent_t e : p->ev) cudaEventDestroy(e); delete p; }
  delete ctx;
  return TS_OK;
}

extern "C" int32_t ts_set_ablation(ts_ctx* ctx, uint32_t flags) {
  if (!ctx) return set_error(TS_ERR_INVALID, "ts_set_ablation: null context");
  if (flags & ~(uint32_t)TS_ABLATE_CALIB_QT) return set_error(TS_ERR_INVALID, "ts_set_ablation: unknown switch");
  ctx->ablation = flags;
  return TS_OK;
}

extern "C" int32_t ts_set_test_mode(ts_ctx* ctx, uint32_t flags) {
  if (!ctx) return set_error(TS_ERR_INVALID, "ts_set_test_mode: null context");
  const uint32_t known = TS_TEST_FORCE_FMA | TS_TEST_NO_TMA | TS_TEST_NO_FEW | TS_TEST_NO_SEED | TS_TEST_SHORT_WAITS | TS_TEST_LOST_ARRIVAL | TS_TEST_PERSIST | TS_TEST_NO_UMMA | TS_TEST_NO_TAIL;
  if (flags & ~known) return set_error(TS_ERR_INVALID, "ts_set_test_mode: unknown switch");
  const unsigned before = ctx->test_mode;
  ctx->test_mode = flags;
  if (!select_paths(ctx)) {
    ctx->test_mode = before;
    select_paths(ctx);
    return set_error(TS_ERR_UNSUPPORTED, "ts_set_test_mode: no vocabulary tiling fits shared memory on that path");
  }
  const cudaError_t e = score_setup(ctx);
  if (e != cudaSuccess) return set_cuda_error("ts_set_test_mode", e);
  return TS_OK;
}

extern "C" size_t ts_workspace_bytes(const ts_ctx* ctx, int32_t batch) {
  if (!ctx || batch < 1 || batch > ctx->cfg.max_batch) return 0;
  return make_layout(ctx, batch).total;
}

static const char* kKernelNames[K_COUNT] = {"expand_init", "score_tile", "score_merge", "expand_level", "expand_finalize",
                                            "zrow_stats", "verify_greedy", "verify_walk", "verify_check", "score_few", "allocate_select", "allocate_cut",
                                            "calib_accumulate", "calib_refit", "attention_inputs", "score_seed", "expand_persistent"};

extern "C" const char* ts_kernel_name(int32_t id) { return (id >= 0 && id < K_COUNT) ? kKernelNames[id] : nullptr; }

extern "C" int32_t ts_profile_enable(ts_ctx* ctx, int32_t capacity) {
  if (!ctx || capacity < 0) return set_error(TS_ERR_INVALID, "ts_profile_enable: bad argument");
  Prof* p = (Prof*)ctx->prof;
  for (cudaEvent_t e : p->ev) cudaEventDestroy(e);
  p->ev.clear(); p->ids.clear(); p->used = 0; p->on = false;
  for (int i = 0; i < 2 * capacity; ++i) {
    cudaEvent_t e;
    cudaError_t err = cudaEventCreate(&e);
    if (err != cudaSuccess) return set_cuda_error("ts_profile_enable", err);
    p->ev.push_back(e);
  }
  p->ids.assign((size_t)capacity, 0);
  p->on = capacity > 0;
  return TS_OK;
}

extern "C" int32_t ts_profile_read(ts_ctx* ctx, int32_t n, double* ms, int64_t* launches, int32_t reset) {
  if (!ctx || n < 0 || (n > 0 && (!ms || !launches))) return set_error(TS_ERR_INVALID, "ts_profile_read: bad argument");
  Prof* p = (Prof*)ctx->prof;
  for (int i = 0; i < n; ++i) { ms[i] = 0.0; launches[i] = i < K_COUNT ? p->launches[i] : 0; }
  for (size_t s = 0; s < p->used; ++s) {
    cudaError_t err = cudaEventSynchronize(p->ev[2 * s + 1]);
    float t = 0.f;
    if (err == cudaSuccess) err = cudaEventElapsedTime(&t, p->ev[2 * s], p->ev[2 * s + 1]);
    if (err != cudaSuccess) return set_cuda_error("ts_profile_read", err);
    if (p->ids[s] < n) ms[p->ids[s]] += t;
  }
  if (reset) { p->used = 0; for (int i = 0; i < K_COUNT; ++i) p->launches[i] = 0; }
  return TS_OK;
}
