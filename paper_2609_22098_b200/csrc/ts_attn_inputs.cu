// Inputs of the target forward over the flattened trees (Section 3.2 item 3): token ids, position ids
// and the dense additive attention mask, expanded from the ancestor bitmasks the expansion emits.
// One CTA per (request, group of rows); a warp writes one mask row at a time, 128 bytes per store
// instruction.  Pure write traffic: B * (Nmax+1)^2 floats.
#include "ts_internal.h"

namespace ts {

constexpr int ATT_THREADS = 256;
constexpr int ATT_ROWS = 32;   // mask rows per CTA

struct AttnArgs {
  int B, N, words;
  const int* anchor; const int* base_pos; const int* n_nodes; const int* tok; const int* depth;
  const uint64_t* mask;
  int* flat_tok; int* pos_ids; float* dense;
};

__global__ void __launch_bounds__(ATT_THREADS) attention_inputs_kernel(const AttnArgs a) {
  const int b = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  pdl_wait();                 // the trees come from the kernels before this one
  pdl_launch_dependents();
  const int N = a.N, R = N + 1;
  const int n = min(max(a.n_nodes[b], 0), N);
  const int row0 = blockIdx.y * ATT_ROWS;
  if (blockIdx.y == 0) {
    const int base = a.base_pos ? a.base_pos[b] : 0;
    for (int i = threadIdx.x; i < R; i += ATT_THREADS) {
      const bool used = i <= n;
      if (a.flat_tok) a.flat_tok[(size_t)b * R + i] = i == 0 ? a.anchor[b] : (used ? a.tok[(size_t)b * N + i - 1] : -1);
      if (a.pos_ids) a.pos_ids[(size_t)b * R + i] = i == 0 ? base : (used ? base + a.depth[(size_t)b * N + i - 1] : 0);
    }
  }
  if (!a.dense) return;
  for (int i = row0 + warp; i < min(row0 + ATT_ROWS, R); i += ATT_THREADS / 32) {
    float* out = a.dense + ((size_t)b * R + i) * R;
    const bool used = i >= 1 && i <= n;
    const uint64_t* bits = a.mask + ((size_t)b * N + (i - 1)) * a.words;
    for (int j0 = 0; j0 < R; j0 += 32) {
      const int j = j0 + lane;
      if (j >= R) break;
      bool on;
      if (i == 0) on = j == 0;                       // the root sees itself
      else if (!used) on = j == i;                   // an unused row sees itself
      else on = j == 0 || ((bits[(j - 1) >> 6] >> ((j - 1) & 63)) & 1ull);
      out[j] = on ? 0.f : -INFINITY;
    }
  }
}

}  // namespace ts

extern "C" int32_t ts_emit_attention_inputs(ts_ctx* ctx, int32_t B, const int32_t* anchor_tok, const int32_t* base_pos,
                                            const int32_t* n_nodes, const int32_t* tok, const int32_t* depth,
                                            const uint64_t* mask, int32_t* flat_tok, int32_t* pos_ids, float* dense_mask,
                                            void* stream) {
  using namespace ts;
  if (!ctx) return set_error(TS_ERR_INVALID, "ts_emit_attention_inputs: null context");
  const void* req[] = {anchor_tok, n_nodes, tok, depth, mask};
  for (const void* p : req)
    if (bad_ptr(p)) return set_error(TS_ERR_INVALID, "ts_emit_attention_inputs: null or misaligned pointer");
  const void* opt[] = {base_pos, flat_tok, pos_ids, dense_mask};
  for (const void* p : opt)
    if (p && ((uintptr_t)p & 3u)) return set_error(TS_ERR_INVALID, "ts_emit_attention_inputs: misaligned pointer");
  if (!flat_tok && !pos_ids && !dense_mask) return set_error(TS_ERR_INVALID, "ts_emit_attention_inputs: no output requested");
  const ts_config& c = ctx->cfg;
  if (B < 1 || B > c.max_batch) return set_error(TS_ERR_INVALID, "ts_emit_attention_inputs: B out of range");
  AttnArgs a{};
  a.B = B; a.N = c.Nmax; a.words = (c.Nmax + 63) / 64;
  a.anchor = anchor_tok; a.base_pos = base_pos; a.n_nodes = n_nodes; a.tok = tok; a.depth = depth; a.mask = mask;
  a.flat_tok = flat_tok; a.pos_ids = pos_ids; a.dense = dense_mask;
  cudaStream_t st = (cudaStream_t)stream;
  const dim3 grid(B, (c.Nmax + 1 + ATT_ROWS - 1) / ATT_ROWS);
  cudaError_t e;
  {
    ProfScope ps(ctx, K_ATTN_INPUTS, st);
    e = launch_kernel(attention_inputs_kernel, grid, dim3(ATT_THREADS), 0, st, true, a);
  }
  if (e == cudaSuccess) e = cudaGetLastError();
  if (e != cudaSuccess) return set_cuda_error("ts_emit_attention_inputs", e);
  return TS_OK;
}
