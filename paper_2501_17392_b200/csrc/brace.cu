// Host side of the BRACE ring-aggregation library: context, argument checks,
// the ring-schedule driver and kernel launches.  C ABI declared in brace.h.
#include "brace.h"

#include <cuda_runtime.h>

#include <cmath>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "brace_kernels.cuh"

using namespace brace;

namespace {

constexpr int kThreads = 256;
constexpr int64_t kMailAlign = 128;   // mailbox length granularity (entries)
constexpr int kDefaultSmCount = 148;  // B200; replaced by the device's own count when a context gets a workspace

enum Phase { kIdle = 0, kReducing = 1, kReduced = 2, kConsensusDone = 3, kGathering = 4, kDone = 5 };

inline int64_t round_up(int64_t x, int64_t m) { return (x + m - 1) / m * m; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

struct brace_ctx {
  int n = 0, f = 0;
  int64_t d = 0;
  brace_params p{};
  Part pt{};
  int lam_i = 0;
  int lam_lo = 0;
  int entry_bytes = 1;
  int64_t seg_max = 0, seg_pad = 0;
  char* ws = nullptr;
  size_t ws_bytes = 0;
  char* mail[2] = {nullptr, nullptr};
  int* d_ids = nullptr;
  // schedule state
  int phase = kIdle;
  int rs_done = 0;   // share-reduce hops completed in the current round
  int ag_done = 0;   // share-only hops completed in the current round
  int last_cuda = 0;
  bool no_ctx_call = false;   // the context lives on the stack of a context-free entry point
  // ids currently stored in d_ids (Byzantine first, then honest), and their staging copy
  std::vector<int> ids_on_device;
  std::vector<int> ids_staging;
  std::vector<char> is_byz;
  bool ids_valid = false;
  int sm_count = kDefaultSmCount;
  size_t stats_smem_set[3] = {0, 0, 0};   // dynamic shared memory already granted to the staged statistics kernels
  // launch tuning (0 = default)
  int fused_variant = 0;
  int fused_grid = 0;
  int step_vpt = 0;
  int spread_mode = 0;   // 0/1 = owner row + share-only launch when the layout allows, 2 = fused kernel writes all rows
  int stats_vw = 0;
  int stats_table = 0;
  int gen_simple = 0;    // 1 = kind 5 with generated draws runs the plain kernel (no compaction of the normals)   // 1 = statistics kernel addresses rows through the offset table even when they are consecutive
};

namespace {

bool params_ok(const brace_params* p) {
  if (!p) return false;
  if (p->rule < BRACE_RULE_SIGN_CONSENSUS || p->rule > BRACE_RULE_ABS_CONSENSUS) return false;
  if (!std::isfinite(p->lambda)) return false;
  if (p->zero_sign < -1 || p->zero_sign > 1) return false;
  if (p->granule < 1) return false;
  if (p->agg_mode < BRACE_AGG_AUTO || p->agg_mode > BRACE_AGG_FUSED) return false;
  return true;
}

int entry_bytes_for(int n, int rule) {
  if (rule == BRACE_RULE_SUM) return 4;
  if (n <= 127) return 1;
  if (n <= 32767) return 2;
  return 0;
}

Part make_part(int n, int64_t d, int64_t G) {
  Part pt;
  pt.d = d;
  pt.G = G;
  pt.Q = (d + G - 1) / G;
  pt.n = n;
  return pt;
}

int64_t seg_end(const Part& pt, int j) { return j + 1 == pt.n ? pt.d : pt.begin(j + 1); }

int64_t longest_segment(const Part& pt) {
  int64_t mx = 0;
  for (int j = 0; j < pt.n; ++j) {
    int64_t len = seg_end(pt, j) - pt.begin(j);
    if (len > mx) mx = len;
  }
  return mx;
}

size_t ids_bytes(int n) { return (size_t)round_up((int64_t)n * 4, 256); }

size_t workspace_need(int n, int64_t d, const brace_params* p) {
  const int eb = entry_bytes_for(n, p->rule);
  if (eb == 0) return 0;
  const Part pt = make_part(n, d, p->granule);
  const int64_t longest = longest_segment(pt);
  const int64_t pad = round_up(longest > 0 ? longest : 1, kMailAlign);
  const size_t one_set = (size_t)round_up((int64_t)n * pad * eb, 256);
  return 2 * one_set + ids_bytes(n);
}

// Integer thresholds of the consensus map bit = (S > hi) | (S < lo), S in [-n, n].
void consensus_thresholds(const brace_params* p, int n, int* hi, int* lo) {
  double fl = std::floor((double)p->lambda);
  if (fl < -(double)n - 1.0) fl = -(double)n - 1.0;
  if (fl > (double)n) fl = (double)n;
  const int never = -2147483647 - 1;
  if (p->rule == BRACE_RULE_MAJORITY_SIGN) {         // sign of the sign-sum; a tie gives -1
    *hi = 0;
    *lo = never;
  } else if (p->rule == BRACE_RULE_ABS_CONSENSUS) {  // |S| > lambda, both directions count alike
    *hi = (int)fl;
    *lo = -(int)fl;
    if (fl < 0.0) { *hi = -n - 1; *lo = never; }     // |S| >= 0 > lambda: always +1
  } else {                                           // Eq. (1)
    *hi = (int)fl;
    *lo = never;
  }
}

// cudaError_t of the last failed runtime call made by a context-free entry point on this thread
thread_local int g_last_cuda_no_ctx = 0;

int cuda_fail(brace_ctx* ctx, cudaError_t err) {
  ctx->last_cuda = (int)err;
  if (ctx->no_ctx_call) g_last_cuda_no_ctx = (int)err;
  return BRACE_ERR_CUDA;
}

int check_launch(brace_ctx* ctx, cudaError_t launch_err = cudaSuccess) {
  cudaError_t err = cudaGetLastError();
  if (launch_err != cudaSuccess) err = launch_err;
  if (err != cudaSuccess) return cuda_fail(ctx, err);
  return BRACE_OK;
}

inline unsigned tiles(int64_t items, int64_t per_block) {
  int64_t t = (items + per_block - 1) / per_block;
  return (unsigned)(t > 0 ? t : 1);
}

// ---- launches of the per-hop kernels -------------------------------------------------

// Launch with programmatic stream serialization: the kernel may begin while its
// predecessor on the stream drains; it synchronises on the device (pdl_wait).
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = 0;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

bool vec_layout_ok(const brace_ctx* ctx, const float* U, int64_t ld) {
  return (ctx->p.granule % 4 == 0) && (ld % 4 == 0) && aligned16(U);
}

int launch_rs_step(brace_ctx* ctx, int step, const float* U, int64_t ld, cudaStream_t st) {
  cudaError_t perr = cudaSuccess;
  const int n = ctx->n;
  const int in_set = step & 1, out_set = (step + 1) & 1;
  const bool vec = vec_layout_ok(ctx, U, ld);
  // float4 per thread: enough loads in flight for long sub-vectors, enough CTAs for short ones
  int vpt = 0;
  if (vec) {
    vpt = ctx->step_vpt > 0 ? ctx->step_vpt : 4;
    while (vpt > 1 && (int64_t)n * ((ctx->seg_max + 1024 * vpt - 1) / (1024 * vpt)) < 4 * ctx->sm_count) vpt >>= 1;
  }
  const int64_t per_block = vec ? (int64_t)kThreads * 4 * vpt : kThreads;
  dim3 grid(tiles(ctx->seg_max, per_block), (unsigned)n);
  const bool zs = ctx->p.zero_sign != 0;
  const int zsv = ctx->p.zero_sign;
#define BRACE_RS_SIGN(P, VPT, ZS)                                                                            \
  perr = launch_pdl(rs_step_sign_kernel<P, VPT, ZS>, grid, dim3(kThreads), st, ctx->pt, U, ld,                       \
             (const P*)ctx->mail[in_set], (P*)ctx->mail[out_set], ctx->seg_pad, step, zsv)
#define BRACE_RS_SIGN_P(P)                                                                         \
  do {                                                                                             \
    switch (vpt) {                                                                                 \
      case 4: if (zs) BRACE_RS_SIGN(P, 4, true); else BRACE_RS_SIGN(P, 4, false); break;           \
      case 2: if (zs) BRACE_RS_SIGN(P, 2, true); else BRACE_RS_SIGN(P, 2, false); break;           \
      case 1: if (zs) BRACE_RS_SIGN(P, 1, true); else BRACE_RS_SIGN(P, 1, false); break;           \
      default: if (zs) BRACE_RS_SIGN(P, 0, true); else BRACE_RS_SIGN(P, 0, false); break;          \
    }                                                                                              \
  } while (0)
  if (ctx->p.rule == BRACE_RULE_SUM) {
    dim3 gsum(tiles(ctx->seg_max, vec ? kThreads * 4 : kThreads), (unsigned)n);
    if (vec)
      perr = launch_pdl(rs_step_sum_kernel<true>, gsum, dim3(kThreads), st, ctx->pt, U, ld,
                 (const float*)ctx->mail[in_set], (float*)ctx->mail[out_set], ctx->seg_pad, step);
    else
      perr = launch_pdl(rs_step_sum_kernel<false>, gsum, dim3(kThreads), st, ctx->pt, U, ld,
                 (const float*)ctx->mail[in_set], (float*)ctx->mail[out_set], ctx->seg_pad, step);
  } else if (ctx->entry_bytes == 1) {
    BRACE_RS_SIGN_P(int8_t);
  } else {
    BRACE_RS_SIGN_P(int16_t);
  }
#undef BRACE_RS_SIGN_P
#undef BRACE_RS_SIGN
  return check_launch(ctx, perr);
}

int launch_consensus(brace_ctx* ctx, void* out, int64_t out_ld, cudaStream_t st) {
  cudaError_t perr = cudaSuccess;
  const int n = ctx->n;
  const int set = (n - 1) & 1;   // the last hop n-2 wrote set (n-1)&1
  if (ctx->p.rule == BRACE_RULE_SUM) {
    const bool vec = (ctx->p.granule % 4 == 0) && (out_ld % 4 == 0) && aligned16(out);
    dim3 grid(tiles(ctx->seg_max, vec ? kThreads * 4 : kThreads), (unsigned)n);
    if (vec)
      perr = launch_pdl(consensus_sum_kernel<true>, grid, dim3(kThreads), st, ctx->pt, (const float*)ctx->mail[set],
                 ctx->seg_pad, (float*)out, out_ld, ctx->p.mean);
    else
      perr = launch_pdl(consensus_sum_kernel<false>, grid, dim3(kThreads), st, ctx->pt, (const float*)ctx->mail[set],
                 ctx->seg_pad, (float*)out, out_ld, ctx->p.mean);
  } else {
    dim3 grid(tiles(ctx->seg_max / 32 + 2, kThreads), (unsigned)n);
    if (ctx->entry_bytes == 1)
      perr = launch_pdl(consensus_sign_kernel<int8_t>, grid, dim3(kThreads), st, ctx->pt, (const int8_t*)ctx->mail[set],
                 ctx->seg_pad, (uint32_t*)out, out_ld, ctx->lam_i, ctx->lam_lo);
    else
      perr = launch_pdl(consensus_sign_kernel<int16_t>, grid, dim3(kThreads), st, ctx->pt, (const int16_t*)ctx->mail[set],
                 ctx->seg_pad, (uint32_t*)out, out_ld, ctx->lam_i, ctx->lam_lo);
  }
  return check_launch(ctx, perr);
}

int launch_ag_step(brace_ctx* ctx, int step, void* out, int64_t out_ld, cudaStream_t st) {
  cudaError_t perr = cudaSuccess;
  const int n = ctx->n;
  if (ctx->p.rule == BRACE_RULE_SUM) {
    const bool vec = (ctx->p.granule % 4 == 0) && (out_ld % 4 == 0) && aligned16(out);
    dim3 grid(tiles(ctx->seg_max, vec ? kThreads * 4 : kThreads), (unsigned)n);
    if (vec)
      perr = launch_pdl(ag_step_f32_kernel<true>, grid, dim3(kThreads), st, ctx->pt, (float*)out, out_ld, step);
    else
      perr = launch_pdl(ag_step_f32_kernel<false>, grid, dim3(kThreads), st, ctx->pt, (float*)out, out_ld, step);
  } else {
    const bool wide = (ctx->p.granule % 128 == 0) && (out_ld % 4 == 0) && aligned16(out);
    if (wide) {
      dim3 grid(tiles(ctx->seg_max / 128 + 2, kThreads), (unsigned)n);
      perr = launch_pdl(ag_step_bits_kernel<4>, grid, dim3(kThreads), st, ctx->pt, (uint32_t*)out, out_ld, step);
    } else {
      dim3 grid(tiles(ctx->seg_max / 32 + 2, kThreads), (unsigned)n);
      perr = launch_pdl(ag_step_bits_kernel<1>, grid, dim3(kThreads), st, ctx->pt, (uint32_t*)out, out_ld, step);
    }
  }
  return check_launch(ctx, perr);
}

// ---- fused round ------------------------------------------------------------------------

bool fused_layout_ok(const brace_ctx* ctx, const float* U, int64_t ld, const void* out, int64_t out_ld) {
  if (ctx->p.granule % 128 != 0 || ld % 4 != 0 || !aligned16(U)) return false;
  if (ctx->p.rule == BRACE_RULE_SUM && (out_ld % 4 != 0 || !aligned16(out))) return false;
  return true;
}

void fused_geometry(const brace_ctx* ctx, FusedArgs& a, int64_t tile) {
  a.tiles_per_seg = (int)((ctx->seg_max + tile - 1) / tile);
  if (a.tiles_per_seg < 1) a.tiles_per_seg = 1;
  a.units = (int64_t)a.tiles_per_seg * ctx->n;
}

int launch_fused(brace_ctx* ctx, const float* U, int64_t ld, void* out, int64_t out_ld, cudaStream_t st) {
  FusedArgs a;
  a.pt = ctx->pt;
  a.U = U;
  a.ld = ld;
  a.mail0 = ctx->mail[0];
  a.mail1 = ctx->mail[1];
  a.seg_pad = ctx->seg_pad;
  a.out = out;
  a.out_ld = out_ld;
  a.lam = ctx->lam_i;
  a.lam_lo = ctx->lam_lo;
  a.zs = ctx->p.zero_sign;
  a.mean = ctx->p.mean;
  // with 16-byte aligned output rows: the kernel writes each sub-vector's result to its owner's row and one
  // share-only launch spreads it (long bursts per row instead of one tile's piece per row); worth a second
  // launch only on large problems
  const bool spread = (out_ld % 4 == 0) && aligned16(out) && ctx->spread_mode != 2 &&
                      (ctx->spread_mode == 1 || (int64_t)ctx->n * ctx->d >= (int64_t)1 << 27);
  a.owner_only = spread ? 1 : 0;
  const bool zs = ctx->p.zero_sign != 0;
  // variant: tile width (float4 per thread per client) x clients prefetched
  int variant = ctx->fused_variant;
  if (variant == 0) variant = 1;
  auto grid_for = [&](int64_t units) -> unsigned {
    int64_t g = units;
    if (ctx->fused_grid > 0 && g > ctx->fused_grid) g = ctx->fused_grid;
    const int64_t cap = (int64_t)ctx->sm_count * 4096;
    if (g > cap) g = cap;
    return (unsigned)(g > 0 ? g : 1);
  };
#define BRACE_FUSED_SIGN(VPT, UNR, TPB)                                                         \
  do {                                                                                          \
    fused_geometry(ctx, a, (int64_t)TPB * 4 * VPT);                                             \
    const unsigned g = grid_for(a.units);                                                       \
    if (ctx->entry_bytes == 1) {                                                                \
      if (zs) fused_sign_kernel<int8_t, VPT, UNR, true, TPB><<<g, TPB, 0, st>>>(a);             \
      else    fused_sign_kernel<int8_t, VPT, UNR, false, TPB><<<g, TPB, 0, st>>>(a);            \
    } else {                                                                                    \
      if (zs) fused_sign_kernel<int16_t, VPT, UNR, true, TPB><<<g, TPB, 0, st>>>(a);            \
      else    fused_sign_kernel<int16_t, VPT, UNR, false, TPB><<<g, TPB, 0, st>>>(a);           \
    }                                                                                           \
  } while (0)
#define BRACE_FUSED_SUM(VPT, UNR)                                                               \
  do {                                                                                          \
    fused_geometry(ctx, a, (int64_t)256 * 4 * VPT);                                             \
    const unsigned g = grid_for(a.units);                                                       \
    fused_sum_kernel<VPT, UNR><<<g, 256, 0, st>>>(a);                                           \
  } while (0)
  if (ctx->p.rule == BRACE_RULE_SUM) {
    switch (variant) {
      case 2: case 4: BRACE_FUSED_SUM(2, 4); break;
      case 3: BRACE_FUSED_SUM(1, 4); break;
      default: BRACE_FUSED_SUM(1, 8); break;
    }
  } else {
    switch (variant) {
      case 2: BRACE_FUSED_SIGN(2, 4, 256); break;
      case 3: BRACE_FUSED_SIGN(1, 4, 256); break;
      case 4: BRACE_FUSED_SIGN(2, 8, 256); break;
      case 5: BRACE_FUSED_SIGN(1, 16, 256); break;
      case 6: BRACE_FUSED_SIGN(1, 8, 128); break;
      default: BRACE_FUSED_SIGN(1, 8, 256); break;
    }
  }
#undef BRACE_FUSED_SIGN
#undef BRACE_FUSED_SUM
  int rc = check_launch(ctx);
  if (rc != BRACE_OK || !spread) return rc;
  const int rows_per_group = 8;
  const unsigned groups = (unsigned)((ctx->n + rows_per_group - 1) / rows_per_group);
  cudaError_t perr;
  if (ctx->p.rule == BRACE_RULE_SUM) {
    dim3 grid(tiles(ctx->seg_max, kThreads * 4), (unsigned)ctx->n, groups);
    perr = launch_pdl(ag_all_f32_kernel, grid, dim3(kThreads), st, ctx->pt, (float*)out, out_ld, rows_per_group);
  } else {
    dim3 grid(tiles(ctx->seg_max / 128 + 2, kThreads), (unsigned)ctx->n, groups);
    perr = launch_pdl(ag_all_bits_kernel, grid, dim3(kThreads), st, ctx->pt, (uint32_t*)out, out_ld, rows_per_group);
  }
  return check_launch(ctx, perr);
}

// ---- argument checks shared by the ring calls -----------------------------------------------

int check_device_ctx(const brace_ctx* ctx) {
  if (!ctx) return BRACE_ERR_INVALID_ARG;
  if (!ctx->ws) return BRACE_ERR_WORKSPACE;
  return BRACE_OK;
}

int check_out(const brace_ctx* ctx, const void* out, int64_t out_ld) {
  if (!out) return BRACE_ERR_INVALID_ARG;
  const int64_t need = ctx->p.rule == BRACE_RULE_SUM ? ctx->d : (ctx->d + 31) / 32;
  if (out_ld < need) return BRACE_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(out) & 3u) != 0) return BRACE_ERR_INVALID_ARG;
  return BRACE_OK;
}

int check_updates(const brace_ctx* ctx, const float* U, int64_t ld) {
  if (!U || ld < ctx->d) return BRACE_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(U) & 3u) != 0) return BRACE_ERR_INVALID_ARG;
  return BRACE_OK;
}

int run_stepwise(brace_ctx* ctx, const float* U, int64_t ld, void* out, int64_t out_ld, cudaStream_t st) {
  const int n = ctx->n;
  for (int s = 0; s < n - 1; ++s) {
    int rc = launch_rs_step(ctx, s, U, ld, st);
    if (rc != BRACE_OK) return rc;
  }
  int rc = launch_consensus(ctx, out, out_ld, st);
  if (rc != BRACE_OK) return rc;
  for (int t = 0; t < n - 1; ++t) {
    rc = launch_ag_step(ctx, t, out, out_ld, st);
    if (rc != BRACE_OK) return rc;
  }
  return BRACE_OK;
}

// Resolve the Byzantine id list and make sure it is on the device (Byzantine ids
// first, honest ids after in increasing order).  The upload is skipped when the
// device copy is already current, so steady-state calls enqueue kernels only.
int stage_ids(brace_ctx* ctx, const int32_t* h_byz_ids, cudaStream_t st) {
  const int n = ctx->n, f = ctx->f;
  std::vector<int>& ids = ctx->ids_staging;          // sized n at init: nothing is allocated here
  std::vector<char>& is_byz = ctx->is_byz;
  std::fill(is_byz.begin(), is_byz.end(), (char)0);
  for (int b = 0; b < f; ++b) {
    const int id = h_byz_ids ? h_byz_ids[b] : b;
    if (id < 0 || id >= n || is_byz[(size_t)id]) return BRACE_ERR_INVALID_ARG;
    is_byz[(size_t)id] = 1;
    ids[(size_t)b] = id;
  }
  int pos = f;
  for (int i = 0; i < n; ++i)
    if (!is_byz[(size_t)i]) ids[(size_t)pos++] = i;
  if (ctx->ids_valid && ids == ctx->ids_on_device) return BRACE_OK;
  // a new id list has to be uploaded: not while the stream is being captured (the copy would be
  // recorded instead of executed, and later calls would skip it)
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  cudaError_t err = cudaStreamIsCapturing(st, &cap);
  if (err != cudaSuccess) return cuda_fail(ctx, err);
  if (cap != cudaStreamCaptureStatusNone) return BRACE_ERR_UNSUPPORTED;
  err = cudaMemcpyAsync(ctx->d_ids, ids.data(), (size_t)n * sizeof(int), cudaMemcpyHostToDevice, st);
  if (err != cudaSuccess) return cuda_fail(ctx, err);
  ctx->ids_on_device = ids;                           // same size: no allocation
  ctx->ids_valid = true;
  return BRACE_OK;
}

int inject_impl(brace_ctx* ctx, const brace_attack* atk, const float* H, int64_t ld_h, float* Uo, int64_t ld_u,
                cudaStream_t st) {
  if (!atk) return BRACE_ERR_INVALID_ARG;
  if (atk->kind == BRACE_ATTACK_NONE || ctx->f == 0) return BRACE_OK;
  if (atk->kind < BRACE_ATTACK_SCALE_OWN || atk->kind > BRACE_ATTACK_SPARSE_NOISE) return BRACE_ERR_INVALID_ARG;
  if (!H || !Uo || ld_h < ctx->d || ld_u < ctx->d) return BRACE_ERR_INVALID_ARG;
  const int kind = atk->kind;
  const bool needs_noise = kind == BRACE_ATTACK_GAUSSIAN || kind == BRACE_ATTACK_SPARSE_NOISE;
  if (atk->draws != BRACE_DRAWS_SUPPLIED && atk->draws != BRACE_DRAWS_GENERATED) return BRACE_ERR_INVALID_ARG;
  const bool generated = needs_noise && atk->draws == BRACE_DRAWS_GENERATED;
  if (generated && atk->round >= (1u << 24)) return BRACE_ERR_INVALID_ARG;
  if (needs_noise && !generated && (!atk->noise || atk->noise_ld < ctx->d)) return BRACE_ERR_INVALID_ARG;
  if (kind == BRACE_ATTACK_SPARSE_NOISE && !generated && (!atk->uniform || atk->uniform_ld < ctx->d))
    return BRACE_ERR_INVALID_ARG;
  int rc = stage_ids(ctx, atk->h_byz_ids, st);
  if (rc != BRACE_OK) return rc;
  const bool rows16 = (ld_h % 4 == 0) && (ld_u % 4 == 0) && aligned16(H) && aligned16(Uo);
  if (generated && kind == BRACE_ATTACK_SPARSE_NOISE && atk->prob < 0.5f && ctx->gen_simple == 0) {
    // uniform < prob  <=>  its 24-bit numerator < ceil(prob * 2^24) (the product is exact in float32)
    const float scaled = std::ceil(atk->prob * 16777216.0f);
    const uint32_t thr = scaled <= 0.0f ? 0u : (uint32_t)scaled;   // NaN and negatives: nothing passes
    dim3 grid(tiles((ctx->d + 7) / 8, kThreads), (unsigned)ctx->f);
    inject_sparse_generated_kernel<<<grid, kThreads, 0, st>>>(ctx->d_ids, Uo, ld_u, ctx->d, atk->seed, atk->round,
                                                             atk->sigma, thr, (ld_u % 4 == 0 && aligned16(Uo)) ? 1 : 0);
    return check_launch(ctx);
  }
  if (generated) {
    dim3 grid(tiles((ctx->d + 3) / 4, kThreads), (unsigned)ctx->f);
    inject_generated_kernel<<<grid, kThreads, 0, st>>>(kind, ctx->d_ids, Uo, ld_u, ctx->d, atk->seed, atk->round,
                                                      atk->sigma, atk->prob, (ld_u % 4 == 0 && aligned16(Uo)) ? 1 : 0);
    return check_launch(ctx);
  }
  if (kind == BRACE_ATTACK_SCALED_MEAN || kind == BRACE_ATTACK_MEAN_SHIFT) {
    const int m = ctx->n - ctx->f;
    const int mpad = (m + 7) / 8 * 8;
    if (kind == BRACE_ATTACK_MEAN_SHIFT && m <= 127 && ctx->stats_vw == 0) {
      // two passes: register-resident variant, one coordinate per thread, all honest values in registers
      const std::vector<int>& ids = ctx->ids_on_device;
      const int f = ctx->f;
      bool strided = (ld_h * 4 < ((int64_t)1 << 32)) && ctx->stats_table == 0;
      for (int r = 1; r < m && strided; ++r) strided = ids[(size_t)f + r] == ids[(size_t)f] + r;
      for (int b = 1; b < f && strided; ++b) strided = ids[(size_t)b] == ids[0] + b;
      const unsigned blocks = tiles(ctx->d, kStatsThreads);
      if (strided) {
        const float* H0 = H + (int64_t)ids[(size_t)f] * ld_h;
        float* U0 = Uo + (int64_t)ids[0] * ld_u;
        HonestRows none{};
#define BRACE_STATS_REG(MFULL)                                                                               \
  case MFULL:                                                                                                \
    inject_stats_reg_kernel<MFULL, 3, true><<<blocks, kStatsThreads, 0, st>>>(kind, none, (uint32_t)(ld_h * 4), nullptr, f, m, \
                                                                    H0, U0, ld_u, ctx->d, atk->scale, atk->kappa);    \
    break
        switch (m / 4 * 4) {
          BRACE_STATS_REG(0); BRACE_STATS_REG(4); BRACE_STATS_REG(8); BRACE_STATS_REG(12); BRACE_STATS_REG(16);
          BRACE_STATS_REG(20); BRACE_STATS_REG(24); BRACE_STATS_REG(28); BRACE_STATS_REG(32); BRACE_STATS_REG(36);
          BRACE_STATS_REG(40); BRACE_STATS_REG(44); BRACE_STATS_REG(48); BRACE_STATS_REG(52); BRACE_STATS_REG(56);
          BRACE_STATS_REG(60); BRACE_STATS_REG(64); BRACE_STATS_REG(68); BRACE_STATS_REG(72); BRACE_STATS_REG(76);
          BRACE_STATS_REG(80); BRACE_STATS_REG(84); BRACE_STATS_REG(88); BRACE_STATS_REG(92); BRACE_STATS_REG(96);
          BRACE_STATS_REG(100); BRACE_STATS_REG(104); BRACE_STATS_REG(108); BRACE_STATS_REG(112);
          BRACE_STATS_REG(116); BRACE_STATS_REG(120);
          default: BRACE_STATS_REG(124);
        }
#undef BRACE_STATS_REG
        return check_launch(ctx);
      }
      HonestRows rows;
      for (int r = 0; r < 128; ++r)
        rows.byte_off[r] = (int64_t)ids[(size_t)f + (size_t)(r < m ? r : m - 1)] * ld_h * 4;
#define BRACE_STATS_REG(MFULL)                                                                                \
  case MFULL:                                                                                                 \
    inject_stats_reg_kernel<MFULL, 7, false><<<blocks, kStatsThreads, 0, st>>>(kind, rows, 0u, ctx->d_ids, f, m, H, Uo, ld_u, \
                                                                     ctx->d, atk->scale, atk->kappa);         \
    break
      switch (m / 8 * 8) {
        BRACE_STATS_REG(0); BRACE_STATS_REG(8); BRACE_STATS_REG(16); BRACE_STATS_REG(24); BRACE_STATS_REG(32);
        BRACE_STATS_REG(40); BRACE_STATS_REG(48); BRACE_STATS_REG(56); BRACE_STATS_REG(64); BRACE_STATS_REG(72);
        BRACE_STATS_REG(80); BRACE_STATS_REG(88); BRACE_STATS_REG(96); BRACE_STATS_REG(104); BRACE_STATS_REG(112);
        default: BRACE_STATS_REG(120);
      }
#undef BRACE_STATS_REG
      return check_launch(ctx);
    }
    // staged variant: one column (vw floats wide) of all m honest rows per thread in shared memory
    const bool rows8 = (ld_h % 2 == 0) && (ld_u % 2 == 0) && (reinterpret_cast<uintptr_t>(H) & 7u) == 0 &&
                       (reinterpret_cast<uintptr_t>(Uo) & 7u) == 0;
    int vw = ctx->stats_vw > 0 ? ctx->stats_vw : 4;
    if (vw == 4 && !rows16) vw = 2;
    if (vw == 2 && !rows8) vw = 1;
    const bool layout_ok = true;
    int T = 1024 / vw;
    while (T > 32 && (size_t)mpad * T * vw * 4 > 40 * 1024) T >>= 1;
    const size_t smem = (size_t)mpad * T * vw * 4 + (size_t)mpad * 8;
    if (layout_ok && smem <= 200 * 1024) {
      auto kern = vw == 1 ? inject_stats_smem_kernel<1, 12>
                          : (vw == 2 ? inject_stats_smem_kernel<2, 12> : inject_stats_smem_kernel<4, 12>);
      size_t& granted = ctx->stats_smem_set[vw == 1 ? 0 : (vw == 2 ? 1 : 2)];
      if (smem > 48 * 1024 && smem > granted) {      // once per context and kernel, not on every call
        cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (err != cudaSuccess) return cuda_fail(ctx, err);
        granted = smem;
      }
      int64_t blocks = (ctx->d + (int64_t)T * vw - 1) / ((int64_t)T * vw);
      const int64_t cap = (int64_t)ctx->sm_count * 64;
      if (blocks > cap) blocks = cap;
      kern<<<(unsigned)blocks, T, smem, st>>>(kind, ctx->d_ids, ctx->f, ctx->n, H, ld_h, Uo, ld_u, ctx->d,
                                             atk->scale, atk->kappa);
    } else {
      // two passes over the honest rows in global memory: keep the set of coordinates in
      // flight small enough that the second pass finds the first one's lines in L2
      int64_t blocks = (ctx->d + kThreads - 1) / kThreads;
      const int64_t cap = (int64_t)ctx->sm_count * 4;
      if (blocks > cap) blocks = cap;
      inject_stats_kernel<8><<<(unsigned)blocks, kThreads, 0, st>>>(kind, ctx->d_ids, ctx->f, ctx->n, H, ld_h, Uo,
                                                                   ld_u, ctx->d, atk->scale, atk->kappa);
    }
  } else {
    const bool draws16 = (!needs_noise || (atk->noise_ld % 4 == 0 && aligned16(atk->noise))) &&
                         (kind != BRACE_ATTACK_SPARSE_NOISE || (atk->uniform_ld % 4 == 0 && aligned16(atk->uniform)));
    if (rows16 && draws16) {
      dim3 grid(tiles(ctx->d, kThreads * 4), (unsigned)ctx->f);
      inject_elementwise_vec_kernel<<<grid, kThreads, 0, st>>>(kind, ctx->d_ids, H, ld_h, Uo, ld_u, atk->noise,
                                                              atk->noise_ld, atk->uniform, atk->uniform_ld, ctx->d,
                                                              atk->scale, atk->sigma, atk->prob);
    } else {
      dim3 grid(tiles(ctx->d, kThreads), (unsigned)ctx->f);
      inject_elementwise_kernel<<<grid, kThreads, 0, st>>>(kind, ctx->d_ids, H, ld_h, Uo, ld_u, atk->noise,
                                                          atk->noise_ld, atk->uniform, atk->uniform_ld, ctx->d,
                                                          atk->scale, atk->sigma, atk->prob);
    }
  }
  return check_launch(ctx);
}

int aggregate_impl(brace_ctx* ctx, const float* U, int64_t ld, void* out, int64_t out_ld, cudaStream_t st) {
  int rc = check_updates(ctx, U, ld);
  if (rc != BRACE_OK) return rc;
  rc = check_out(ctx, out, out_ld);
  if (rc != BRACE_OK) return rc;
  const bool can_fuse = fused_layout_ok(ctx, U, ld, out, out_ld);
  int mode = ctx->p.agg_mode;
  if (mode == BRACE_AGG_FUSED && !can_fuse) return BRACE_ERR_UNSUPPORTED;
  if (mode == BRACE_AGG_AUTO) mode = can_fuse ? BRACE_AGG_FUSED : BRACE_AGG_STEPWISE;
  rc = (mode == BRACE_AGG_FUSED) ? launch_fused(ctx, U, ld, out, out_ld, st)
                                 : run_stepwise(ctx, U, ld, out, out_ld, st);
  if (rc != BRACE_OK) {
    ctx->phase = kIdle;
    return rc;
  }
  ctx->phase = kDone;
  ctx->rs_done = ctx->n - 1;
  ctx->ag_done = ctx->n - 1;
  return BRACE_OK;
}

}  // namespace

// ---- round without a caller workspace ---------------------------------------------------------
// Mailbox scratch for brace_aggregate_static.  Every GPU that loads the library
// holds these bytes until the process exits.  In host code the symbol's name is
// only a handle: the device address is fetched with cudaGetSymbolAddress (on
// every call, for the device that is current then: the lookup allocates nothing,
// and a cached pointer would go stale after cudaDeviceReset or under another
// context) and that pointer is what the kernels receive.
constexpr size_t kStaticScratchBytes = (size_t)BRACE_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// =============================================================================================
// C ABI
// =============================================================================================
extern "C" {

const char* brace_status_string(int status) {
  switch (status) {
    case BRACE_OK: return "ok";
    case BRACE_ERR_INVALID_ARG: return "invalid argument";
    case BRACE_ERR_UNSUPPORTED: return "unsupported configuration";
    case BRACE_ERR_BAD_STEP: return "ring step called out of order";
    case BRACE_ERR_WORKSPACE: return "workspace missing, too small or misaligned";
    case BRACE_ERR_CUDA: return "CUDA runtime error";
    case BRACE_ERR_TIMEOUT: return "device-side wait timed out";
    default: return "unknown status";
  }
}

int brace_default_params(brace_params* p) {
  if (!p) return BRACE_ERR_INVALID_ARG;
  p->rule = BRACE_RULE_SIGN_CONSENSUS;
  p->lambda = 0.0f;
  p->zero_sign = 0;
  p->granule = 128;
  p->mean = 0;
  p->agg_mode = BRACE_AGG_AUTO;
  return BRACE_OK;
}

size_t brace_workspace_bytes(int32_t n, int64_t d, const brace_params* params) {
  if (n < 2 || d < 1 || !params_ok(params)) return 0;
  return workspace_need(n, d, params);
}

int brace_init(brace_ctx** out, int32_t n, int32_t f, int64_t d, const brace_params* params, void* d_workspace,
               size_t workspace_bytes, brace_stream_t /*stream*/) {
  if (!out) return BRACE_ERR_INVALID_ARG;
  *out = nullptr;
  if (n < 2 || f < 0 || f >= n || d < 1 || !params_ok(params)) return BRACE_ERR_INVALID_ARG;
  const int eb = entry_bytes_for(n, params->rule);
  if (eb == 0) return BRACE_ERR_UNSUPPORTED;
  const size_t need = workspace_need(n, d, params);
  const bool host_only = (d_workspace == nullptr && workspace_bytes == 0);
  if (!host_only) {
    if (!d_workspace || workspace_bytes < need) return BRACE_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(d_workspace) & 255u) != 0) return BRACE_ERR_WORKSPACE;
  }
  brace_ctx* ctx = new (std::nothrow) brace_ctx();
  if (!ctx) return BRACE_ERR_INVALID_ARG;
  try {                                              // host vectors are sized once, here
    ctx->ids_on_device.assign((size_t)n, 0);
    ctx->ids_staging.assign((size_t)n, 0);
    ctx->is_byz.assign((size_t)n, 0);
  } catch (...) {
    delete ctx;
    return BRACE_ERR_INVALID_ARG;
  }
  ctx->n = n;
  ctx->f = f;
  ctx->d = d;
  ctx->p = *params;
  ctx->pt = make_part(n, d, params->granule);
  consensus_thresholds(params, n, &ctx->lam_i, &ctx->lam_lo);
  ctx->entry_bytes = eb;
  ctx->seg_max = longest_segment(ctx->pt);
  ctx->seg_pad = round_up(ctx->seg_max > 0 ? ctx->seg_max : 1, kMailAlign);
  if (!host_only) {
    ctx->ws = static_cast<char*>(d_workspace);
    ctx->ws_bytes = workspace_bytes;
    const size_t one_set = (size_t)round_up((int64_t)n * ctx->seg_pad * eb, 256);
    ctx->mail[0] = ctx->ws;
    ctx->mail[1] = ctx->ws + one_set;
    ctx->d_ids = reinterpret_cast<int*>(ctx->ws + 2 * one_set);
    int dev = 0, sms = 0;                            // grid sizing follows the device that is current now
    if (cudaGetDevice(&dev) == cudaSuccess &&
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && sms > 0)
      ctx->sm_count = sms;
  }
  *out = ctx;
  return BRACE_OK;
}

int brace_destroy(brace_ctx* ctx) {
  if (!ctx) return BRACE_ERR_INVALID_ARG;
  delete ctx;
  return BRACE_OK;
}

int brace_segment(const brace_ctx* ctx, int32_t j, int64_t* begin, int64_t* end) {
  if (!ctx || !begin || !end || j < 0 || j >= ctx->n) return BRACE_ERR_INVALID_ARG;
  *begin = ctx->pt.begin(j);
  *end = seg_end(ctx->pt, j);
  return BRACE_OK;
}

int brace_comm_cost(const brace_ctx* ctx, int32_t m_bits, brace_cost* cost) {
  if (!ctx || !cost || m_bits < 1) return BRACE_ERR_INVALID_ARG;
  const int n = ctx->n;
  const int64_t d = ctx->d, m = m_bits;
  const int used = ctx->p.rule == BRACE_RULE_SUM ? 32 : 8 * ctx->entry_bytes;
  int need = 1;
  while ((1LL << need) < 2LL * n + 1) ++need;
  std::memset(cost, 0, sizeof(*cost));
  cost->sc_bits = m * n * d;
  cost->rar_closed_form = 2.0 * (double)m * (double)d * (double)(n - 1) / (double)n;
  cost->brace_closed_form = (double)d * (double)(n - 1) * (double)(m + 1) / (double)n;
  cost->partial_bits_used = used;
  cost->partial_bits_min = need;
  for (int c = 0; c < n; ++c) {
    const int skip_rs = (c + 1) % n, skip_ag = (c + 2) % n;   // the sub-vectors client c never sends
    const int64_t rs = d - (seg_end(ctx->pt, skip_rs) - ctx->pt.begin(skip_rs));
    const int64_t ag = d - (seg_end(ctx->pt, skip_ag) - ctx->pt.begin(skip_ag));
    const int64_t rar = (rs + ag) * m, brace_bits = rs * m + ag, packed = rs * used + ag;
    if (c == 0 || rar < cost->rar_bits_min) cost->rar_bits_min = rar;
    if (c == 0 || rar > cost->rar_bits_max) cost->rar_bits_max = rar;
    if (c == 0 || brace_bits < cost->brace_bits_min) cost->brace_bits_min = brace_bits;
    if (c == 0 || brace_bits > cost->brace_bits_max) cost->brace_bits_max = brace_bits;
    if (c == 0 || packed < cost->packed_bits_min) cost->packed_bits_min = packed;
    if (c == 0 || packed > cost->packed_bits_max) cost->packed_bits_max = packed;
  }
  return BRACE_OK;
}

int brace_last_cuda_error(const brace_ctx* ctx) { return ctx ? ctx->last_cuda : g_last_cuda_no_ctx; }

int brace_set_tuning(brace_ctx* ctx, int32_t fused_variant, int32_t fused_grid) {
  if (!ctx || fused_variant < 0 || fused_grid < 0) return BRACE_ERR_INVALID_ARG;
  const int spread_code = fused_variant / 1000;  // thousands digit: 1 = always spread with a share-only launch, 2 = never
  fused_variant %= 1000;
  const int stats_code = fused_variant / 100;    // hundreds digit: floats per thread of the statistics kernel
  const int step_code = (fused_variant / 10) % 10;   // tens digit: float4 per thread of the hop kernel
  fused_variant %= 10;
  if (fused_variant > 6 || (step_code != 0 && step_code != 1 && step_code != 2 && step_code != 4) ||
      (stats_code != 0 && stats_code != 1 && stats_code != 2 && stats_code != 4 && stats_code != 8 && stats_code != 9))
    return BRACE_ERR_INVALID_ARG;
  if (spread_code < 0 || spread_code > 2) return BRACE_ERR_INVALID_ARG;
  ctx->spread_mode = spread_code;
  ctx->step_vpt = step_code;
  ctx->stats_vw = (stats_code == 8 || stats_code == 9) ? 0 : stats_code;
  ctx->stats_table = stats_code == 8 ? 1 : 0;
  ctx->gen_simple = stats_code == 9 ? 1 : 0;
  ctx->fused_variant = fused_variant;
  ctx->fused_grid = fused_grid;
  return BRACE_OK;
}

int brace_inject_attack(brace_ctx* ctx, const brace_attack* attack, const float* d_honest, int64_t ld_honest,
                        float* d_updates, int64_t ld_updates, brace_stream_t stream) {
  int rc = check_device_ctx(ctx);
  if (rc != BRACE_OK) return rc;
  return inject_impl(ctx, attack, d_honest, ld_honest, d_updates, ld_updates, static_cast<cudaStream_t>(stream));
}

int brace_draw_matrix(int32_t what, uint64_t seed, uint32_t round, int32_t first_client, int32_t rows, int64_t d,
                      float* d_out, int64_t ld, float mu, float sigma, brace_stream_t stream) {
  if ((what != BRACE_DRAW_UNIFORM && what != BRACE_DRAW_NORMAL) || !d_out || rows < 1 || d < 1 || ld < d ||
      first_client < 0 || round >= (1u << 24) || rows > 65535)
    return BRACE_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(d_out) & 3u) != 0) return BRACE_ERR_INVALID_ARG;
  brace_ctx ctx;
  ctx.no_ctx_call = true;
  dim3 grid(tiles((d + 3) / 4, kThreads), (unsigned)rows);
  draw_matrix_kernel<<<grid, kThreads, 0, static_cast<cudaStream_t>(stream)>>>(
      what, seed, round, first_client, d_out, ld, d, mu, sigma, (ld % 4 == 0 && aligned16(d_out)) ? 1 : 0);
  return check_launch(&ctx);
}

int brace_quantize(brace_ctx* ctx, const float* d_updates, int64_t ld, int8_t* d_q, int64_t ld_q,
                   brace_stream_t stream) {
  int rc = check_device_ctx(ctx);
  if (rc != BRACE_OK) return rc;
  rc = check_updates(ctx, d_updates, ld);
  if (rc != BRACE_OK) return rc;
  if (!d_q || ld_q < ctx->d) return BRACE_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  dim3 grid(tiles(ctx->d, kThreads), (unsigned)ctx->n);
  if (ctx->p.zero_sign != 0)
    quantize_kernel<true><<<grid, kThreads, 0, st>>>(d_updates, ld, d_q, ld_q, ctx->d, ctx->p.zero_sign);
  else
    quantize_kernel<false><<<grid, kThreads, 0, st>>>(d_updates, ld, d_q, ld_q, ctx->d, 0);
  return check_launch(ctx);
}

int brace_apply_update(brace_ctx* ctx, const void* d_out, int64_t out_ld, float* d_weights, int64_t ld_weights,
                       float eta, brace_stream_t stream) {
  int rc = check_device_ctx(ctx);
  if (rc != BRACE_OK) return rc;
  rc = check_out(ctx, d_out, out_ld);
  if (rc != BRACE_OK) return rc;
  if (!d_weights || ld_weights < ctx->d || !std::isfinite(eta)) return BRACE_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(d_weights) & 3u) != 0) return BRACE_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const bool wvec = (ld_weights % 4 == 0) && aligned16(d_weights);
  constexpr int kUpt = 4;                            // float4 per thread on the aligned path
  dim3 grid_v(tiles(ctx->d, kThreads * 4 * kUpt), (unsigned)ctx->n);
  dim3 grid_s(tiles(ctx->d, kThreads * 4), (unsigned)ctx->n);
  if (ctx->p.rule == BRACE_RULE_SUM) {
    // the rows hold the sum (or already the mean): w <- w - (eta/n) * sum, or w - eta * mean
    const float scale = ctx->p.mean ? eta : eta / (float)ctx->n;
    const bool vec = wvec && (out_ld % 4 == 0) && aligned16(d_out);
    if (vec)
      apply_update_f32_kernel<true, kUpt><<<grid_v, kThreads, 0, st>>>((const float*)d_out, out_ld, d_weights,
                                                                      ld_weights, ctx->d, scale);
    else
      apply_update_f32_kernel<false, 1><<<grid_s, kThreads, 0, st>>>((const float*)d_out, out_ld, d_weights,
                                                                    ld_weights, ctx->d, scale);
  } else {
    if (wvec)
      apply_update_bits_kernel<true, kUpt><<<grid_v, kThreads, 0, st>>>((const uint32_t*)d_out, out_ld, d_weights,
                                                                       ld_weights, ctx->d, eta);
    else
      apply_update_bits_kernel<false, 1><<<grid_s, kThreads, 0, st>>>((const uint32_t*)d_out, out_ld, d_weights,
                                                                     ld_weights, ctx->d, eta);
  }
  return check_launch(ctx);
}

int brace_coordinate_stat(brace_ctx* ctx, int32_t kind, int32_t trim, const float* d_updates, int64_t ld,
                          float* d_result, brace_stream_t stream) {
  if (!ctx) return BRACE_ERR_INVALID_ARG;
  int rc = check_updates(ctx, d_updates, ld);
  if (rc != BRACE_OK) return rc;
  if (!d_result || (kind != BRACE_STAT_MEDIAN && kind != BRACE_STAT_TRIMMED_MEAN)) return BRACE_ERR_INVALID_ARG;
  if (kind == BRACE_STAT_TRIMMED_MEAN && (trim < 0 || 2 * (int64_t)trim >= ctx->n)) return BRACE_ERR_INVALID_ARG;
  if (ctx->n > 128) return BRACE_ERR_UNSUPPORTED;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const unsigned blocks = tiles(ctx->d, kStatThreads);
  const int n = ctx->n;
#define BRACE_STAT(NB) \
  case NB: coordinate_stat_kernel<NB><<<blocks, kStatThreads, 0, st>>>(kind, trim, n, d_updates, ld, d_result, ctx->d); break
  switch (n <= 4 ? 4 : (n + 7) / 8 * 8) {            // n rounded up to a multiple of 8 (4 for the smallest)
    BRACE_STAT(4); BRACE_STAT(8); BRACE_STAT(16); BRACE_STAT(24); BRACE_STAT(32); BRACE_STAT(40); BRACE_STAT(48);
    BRACE_STAT(56); BRACE_STAT(64); BRACE_STAT(72); BRACE_STAT(80); BRACE_STAT(88); BRACE_STAT(96); BRACE_STAT(104);
    BRACE_STAT(112); BRACE_STAT(120);
    default: BRACE_STAT(128);
  }
#undef BRACE_STAT
  return check_launch(ctx);
}

int brace_ring_reduce_scatter_step(brace_ctx* ctx, int32_t step, const float* d_updates, int64_t ld,
                                   brace_stream_t stream) {
  int rc = check_device_ctx(ctx);
  if (rc != BRACE_OK) return rc;
  rc = check_updates(ctx, d_updates, ld);
  if (rc != BRACE_OK) return rc;
  if (step < 0 || step > ctx->n - 2) return BRACE_ERR_BAD_STEP;
  if (step != 0 && !(ctx->phase == kReducing && ctx->rs_done == step)) return BRACE_ERR_BAD_STEP;
  rc = launch_rs_step(ctx, step, d_updates, ld, static_cast<cudaStream_t>(stream));
  if (rc != BRACE_OK) {
    ctx->phase = kIdle;
    return rc;
  }
  ctx->rs_done = step + 1;
  ctx->ag_done = 0;
  ctx->phase = (ctx->rs_done == ctx->n - 1) ? kReduced : kReducing;
  return BRACE_OK;
}

int brace_consensus(brace_ctx* ctx, void* d_out, int64_t out_ld, brace_stream_t stream) {
  int rc = check_device_ctx(ctx);
  if (rc != BRACE_OK) return rc;
  rc = check_out(ctx, d_out, out_ld);
  if (rc != BRACE_OK) return rc;
  if (ctx->phase != kReduced) return BRACE_ERR_BAD_STEP;
  rc = launch_consensus(ctx, d_out, out_ld, static_cast<cudaStream_t>(stream));
  if (rc != BRACE_OK) {
    ctx->phase = kIdle;
    return rc;
  }
  ctx->phase = kConsensusDone;
  ctx->ag_done = 0;
  return BRACE_OK;
}

int brace_ring_allgather_step(brace_ctx* ctx, int32_t step, void* d_out, int64_t out_ld, brace_stream_t stream) {
  int rc = check_device_ctx(ctx);
  if (rc != BRACE_OK) return rc;
  rc = check_out(ctx, d_out, out_ld);
  if (rc != BRACE_OK) return rc;
  if (step < 0 || step > ctx->n - 2) return BRACE_ERR_BAD_STEP;
  const bool in_order =
      (ctx->phase == kConsensusDone && step == 0) || (ctx->phase == kGathering && step == ctx->ag_done);
  if (!in_order) return BRACE_ERR_BAD_STEP;
  rc = launch_ag_step(ctx, step, d_out, out_ld, static_cast<cudaStream_t>(stream));
  if (rc != BRACE_OK) {
    ctx->phase = kIdle;
    return rc;
  }
  ctx->ag_done = step + 1;
  ctx->phase = (ctx->ag_done == ctx->n - 1) ? kDone : kGathering;
  return BRACE_OK;
}

int brace_aggregate(brace_ctx* ctx, const float* d_updates, int64_t ld, void* d_out, int64_t out_ld,
                    brace_stream_t stream) {
  int rc = check_device_ctx(ctx);
  if (rc != BRACE_OK) return rc;
  return aggregate_impl(ctx, d_updates, ld, d_out, out_ld, static_cast<cudaStream_t>(stream));
}

int brace_aggregate_host(brace_ctx* ctx, const brace_attack* attack, const float* h_updates, int64_t ld, void* h_out,
                         int64_t out_ld, float* d_updates_stage, float* d_noise_stage, float* d_uniform_stage,
                         void* d_out_stage, brace_stream_t stream) {
  int rc = check_device_ctx(ctx);
  if (rc != BRACE_OK) return rc;
  if (!h_updates || !h_out || !d_updates_stage || !d_out_stage || ld < ctx->d) return BRACE_ERR_INVALID_ARG;
  rc = check_out(ctx, d_out_stage, out_ld);
  if (rc != BRACE_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int n = ctx->n, f = ctx->f;
  brace_attack dev_attack;
  const bool do_attack = attack && attack->kind != BRACE_ATTACK_NONE && f > 0;
  if (do_attack) {
    dev_attack = *attack;
    const bool supplied = attack->draws == BRACE_DRAWS_SUPPLIED;
    const bool needs_noise =
        supplied && (attack->kind == BRACE_ATTACK_GAUSSIAN || attack->kind == BRACE_ATTACK_SPARSE_NOISE);
    const bool needs_unif = supplied && attack->kind == BRACE_ATTACK_SPARSE_NOISE;
    if (needs_noise && (!attack->noise || !d_noise_stage || attack->noise_ld < ctx->d)) return BRACE_ERR_INVALID_ARG;
    if (needs_unif && (!attack->uniform || !d_uniform_stage || attack->uniform_ld < ctx->d))
      return BRACE_ERR_INVALID_ARG;
    if (needs_noise) {
      cudaError_t err = cudaMemcpyAsync(d_noise_stage, attack->noise, (size_t)f * attack->noise_ld * sizeof(float),
                                        cudaMemcpyHostToDevice, st);
      if (err != cudaSuccess) return cuda_fail(ctx, err);
      dev_attack.noise = d_noise_stage;
    }
    if (needs_unif) {
      cudaError_t err = cudaMemcpyAsync(d_uniform_stage, attack->uniform,
                                        (size_t)f * attack->uniform_ld * sizeof(float), cudaMemcpyHostToDevice, st);
      if (err != cudaSuccess) return cuda_fail(ctx, err);
      dev_attack.uniform = d_uniform_stage;
    }
  }
  cudaError_t err = cudaMemcpyAsync(d_updates_stage, h_updates, (size_t)n * ld * sizeof(float),
                                    cudaMemcpyHostToDevice, st);
  if (err != cudaSuccess) return cuda_fail(ctx, err);
  if (do_attack) {
    rc = inject_impl(ctx, &dev_attack, d_updates_stage, ld, d_updates_stage, ld, st);
    if (rc != BRACE_OK) return rc;
  }
  rc = aggregate_impl(ctx, d_updates_stage, ld, d_out_stage, out_ld, st);
  if (rc != BRACE_OK) return rc;
  err = cudaMemcpyAsync(h_out, d_out_stage, (size_t)n * out_ld * 4, cudaMemcpyDeviceToHost, st);
  if (err != cudaSuccess) return cuda_fail(ctx, err);
  return BRACE_OK;
}

int brace_debug_mailbox(const brace_ctx* ctx, int32_t client, int32_t hops_back, const void** d_ptr, int64_t* len,
                        int32_t* segment, int32_t* entry_bytes) {
  if (!ctx || !d_ptr || !len || client < 0 || client >= ctx->n || hops_back < 0 || hops_back > 1)
    return BRACE_ERR_INVALID_ARG;
  if (!ctx->ws) return BRACE_ERR_WORKSPACE;
  if (ctx->rs_done < 1 + hops_back) return BRACE_ERR_BAD_STEP;
  const int s = ctx->rs_done - 1 - hops_back;  // the hop asked for
  const int set = (s + 1) & 1;
  int j = (client - 1 - s) % ctx->n;
  if (j < 0) j += ctx->n;
  *d_ptr = ctx->mail[set] + (size_t)client * ctx->seg_pad * ctx->entry_bytes;
  *len = seg_end(ctx->pt, j) - ctx->pt.begin(j);
  if (segment) *segment = j;
  if (entry_bytes) *entry_bytes = ctx->entry_bytes;
  return BRACE_OK;
}

int brace_minmax_rate_probe(int32_t blocks, int32_t iters, float* d_out, int64_t* ops, brace_stream_t stream) {
  if (blocks < 1 || iters < 1 || !d_out || !ops) return BRACE_ERR_INVALID_ARG;
  brace_ctx ctx;
  ctx.no_ctx_call = true;
  minmax_rate_kernel<<<(unsigned)blocks, kThreads, 0, static_cast<cudaStream_t>(stream)>>>(d_out, iters);
  *ops = (int64_t)blocks * kThreads * (int64_t)iters * 64;
  return check_launch(&ctx);
}

int brace_debug_status(int32_t* h_code) {
  if (!h_code) return BRACE_ERR_INVALID_ARG;
  *h_code = 0;
#ifdef BRACE_DEBUG
  int code = 0;
  const int zero = 0;
  cudaError_t err = cudaMemcpyFromSymbol(&code, g_debug_status, sizeof(int));     // waits for the device
  if (err == cudaSuccess) err = cudaMemcpyToSymbol(g_debug_status, &zero, sizeof(int));
  if (err != cudaSuccess) {
    g_last_cuda_no_ctx = (int)err;
    return BRACE_ERR_CUDA;
  }
  *h_code = code;
  return BRACE_OK;
#else
  return BRACE_ERR_UNSUPPORTED;
#endif
}

int brace_aggregate_static(int32_t n, int64_t d, const brace_params* params, const float* d_updates, int64_t ld,
                           void* d_out, int64_t out_ld, brace_stream_t stream) {
  if (n < 2 || d < 1 || !params_ok(params)) return BRACE_ERR_INVALID_ARG;
  const int eb = entry_bytes_for(n, params->rule);
  if (eb == 0) return BRACE_ERR_UNSUPPORTED;
  // size check first: a request that cannot fit is refused before any CUDA call
  const Part pt = make_part(n, d, params->granule);
  const int64_t seg_max = longest_segment(pt);
  const int64_t seg_pad = round_up(seg_max > 0 ? seg_max : 1, kMailAlign);
  const size_t one_set = (size_t)round_up((int64_t)n * seg_pad * eb, 256);
  if (2 * one_set > kStaticScratchBytes) return BRACE_ERR_WORKSPACE;

  brace_ctx ctx;                       // host stack only; its vectors stay empty
  ctx.no_ctx_call = true;
  ctx.n = n;
  ctx.f = 0;
  ctx.d = d;
  ctx.p = *params;
  ctx.pt = pt;
  consensus_thresholds(params, n, &ctx.lam_i, &ctx.lam_lo);
  ctx.entry_bytes = eb;
  ctx.seg_max = seg_max;
  ctx.seg_pad = seg_pad;
  int rc = check_updates(&ctx, d_updates, ld);
  if (rc != BRACE_OK) return rc;
  rc = check_out(&ctx, d_out, out_ld);
  if (rc != BRACE_OK) return rc;
  if (!fused_layout_ok(&ctx, d_updates, ld, d_out, out_ld)) return BRACE_ERR_UNSUPPORTED;
  void* scratch = nullptr;
  cudaError_t err = cudaGetSymbolAddress(&scratch, g_static_scratch);
  if (err != cudaSuccess) return cuda_fail(&ctx, err);
  if (!scratch || (reinterpret_cast<uintptr_t>(scratch) & 255u) != 0) return cuda_fail(&ctx, cudaErrorInvalidSymbol);
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) == cudaSuccess &&
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && sms > 0)
    ctx.sm_count = sms;
  ctx.ws = static_cast<char*>(scratch);
  ctx.ws_bytes = kStaticScratchBytes;
  ctx.mail[0] = ctx.ws;
  ctx.mail[1] = ctx.ws + one_set;
  // nothing in the scratch has to start at zero: the fused kernel only writes the
  // mailboxes (the partial sums travel in registers), so stale contents are harmless
  return launch_fused(&ctx, d_updates, ld, d_out, out_ld, static_cast<cudaStream_t>(stream));
}

}  // extern "C"
