// Host side of the C ABI declared in include/idkm.h: argument checks, workspace layout, tile
// tables and the launch sequences.  Every step of the path runs in the kernels of
// idkm_kernels.cuh; nothing here computes on the data.
#include <nvtx3/nvToolsExt.h>
#include "idkm_kernels.cuh"

#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <new>

#include "../../include/idkm.h"

namespace idkm {

extern const KernelEntry k_table_step[3][N_FAMILY];
extern const KernelEntry k_table_final[3][N_FAMILY];
extern const KernelEntry k_table_grad[3][N_FAMILY];
extern const KernelEntry k_table_adj[3][N_FAMILY];
extern const KernelEntry k_table_scatter[3][N_FAMILY];
extern const KernelEntry k_table_step_sq[3][N_FAMILY];
extern const KernelEntry k_table_final_sq[3][N_FAMILY];
extern const KernelEntry k_table_grad_sq[3][N_FAMILY];
extern const KernelEntry k_table_adj_sq[3][N_FAMILY];
extern const KernelEntry k_table_scatter_sq[3][N_FAMILY];
extern const KernelEntry k_table_step_precise[3][N_FAMILY];
extern const KernelEntry k_table_jacobian[3][N_FAMILY];
extern const SmallLoopEntry k_table_small[3][N_SMALL_FAMILY];
extern const DualEntry k_table_dual[3][2];
extern const DualEntry k_table_dual_delta[3][2];
extern const KernelEntry k_table_step_delta[3][N_FAMILY];
extern const KernelEntry k_table_step_bulk[3][N_FAMILY];

// Initialise the per-layer state and copy C0 into the working centroids.
__global__ void idkm_init_forward(LayerState* st, int n_layers, const float* C0, float* C, int n_coord, int k, int d,
                                  double inv_tau, unsigned int* gtickets, int n_groups, unsigned int* sync,
                                  unsigned int* gtickets64, int n_groups64, int squared) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  for (int o = i; o < n_groups; o += gridDim.x * blockDim.x) gtickets[o] = 0u;
  for (int o = i; o < n_groups64; o += gridDim.x * blockDim.x) gtickets64[o] = 0u;
  if (i < 4) sync[i] = 0u;
  if (i < n_layers) {
    LayerState s;
    s.fwd_done = 0; s.fwd_iters = 0; s.fwd_res = 0.f; s.dead = 0;
    s.adj_done = 0; s.adj_iters = 0; s.adj_res = 0.f; s.status = ST_OK;
    s.ticket = 0u; s.adj_up = 0; s.adj_prev = 3.0e38f;
    s.g_norm = 0.f;
    for (int q = 0; q < 2; ++q) s.pad[q] = 0;
    // bounding box of the starting centroids decides which step kernel takes the layer first
    double box2 = 0.0;
    for (int a = 0; a < d; ++a) {
      double lo = 1e300, hi = -1e300;
      for (int j = 0; j < k; ++j) {
        const double v = (double)C0[((size_t)i * k + j) * d + a];
        lo = fmin(lo, v);
        hi = fmax(hi, v);
      }
      box2 += (hi - lo) * (hi - lo);
    }
    s.precise[0] = s.precise[1] = (!squared && sqrt(box2) * inv_tau <= PRECISE_SPAN) ? 1 : 0;
    st[i] = s;
  }
  if (C0 != C)
    for (int o = i; o < n_coord; o += gridDim.x * blockDim.x) C[o] = C0[o];
}

static int d_index(int d) { return d == 1 ? 0 : (d == 2 ? 1 : (d == 4 ? 2 : -1)); }

// The squared-distance variant of a fused pass (same layouts, same tile and partial sizes as kernel_entry's).
static const KernelEntry* kernel_entry_sq(int mode, int d, int family) {
  const int di = d_index(d);
  if (di < 0 || family < 0 || family >= N_FAMILY) return nullptr;
  switch (mode) {
    case STEP: return &k_table_step_sq[di][family];
    case FINAL: return &k_table_final_sq[di][family];
    case GRAD: return &k_table_grad_sq[di][family];
    case ADJ: return &k_table_adj_sq[di][family];
    case SCATTER: return &k_table_scatter_sq[di][family];
  }
  return nullptr;
}

const KernelEntry* kernel_entry(int mode, int d, int family) {
  const int di = d_index(d);
  if (di < 0 || family < 0 || family >= N_FAMILY) return nullptr;
  switch (mode) {
    case STEP: return &k_table_step[di][family];
    case FINAL: return &k_table_final[di][family];
    case GRAD: return &k_table_grad[di][family];
    case ADJ: return &k_table_adj[di][family];
    case SCATTER: return &k_table_scatter[di][family];
    case STEP_PRECISE: return &k_table_step_precise[di][family];
    case STEP_DELTA: return &k_table_step_delta[di][family];
    case JACOBIAN: return &k_table_jacobian[di][family];
  }
  return nullptr;
}

// Tuning override for experiments: IDKM_FORCE_FAMILY="<mode>:<family>[,<mode>:<family>...]" forces the codebook
// layout of a pass (used only if that layout can hold k centroids).
static int forced_family(int mode) {
  static int table[N_MODES];
  static bool parsed = false;
  if (!parsed) {
    for (int i = 0; i < N_MODES; ++i) table[i] = -1;
    const char* e = getenv("IDKM_FORCE_FAMILY");
    while (e && *e) {
      int m = -1, f = -1;
      if (sscanf(e, "%d:%d", &m, &f) == 2 && m >= 0 && m < N_MODES && f >= 0 && f < N_FAMILY) table[m] = f;
      e = strchr(e, ',');
      if (e) ++e;
    }
    parsed = true;
  }
  return table[mode];
}

int pick_family(int mode, int d, int k) {
  const int forced = forced_family(mode);
  if (forced >= 0) {
    const KernelEntry* e = kernel_entry(mode, d, forced);
    if (e && e->launch && e->kpl * e->lpw >= k) return forced;
  }
  // forward step with more than 128 centroids: for d <= 2 the 8-centroids-per-lane, full-warp layout at two blocks
  // per SM is faster than 16 centroids per lane on half-warps (m = 2^22, k = 256: d = 1 0.46 against 0.54 ms, d = 2
  // 0.71 against 0.77 ms); for d = 4 the half-warp layout wins (0.90 against 0.95 ms)
  if (mode == STEP && k > 128 && d < 4) return FAM_WIDE;
  // adjoint step with more than 128 centroids at d = 4: 16 centroids per lane on half-warps (m = 2^22, k = 256:
  // 1.22 against 1.29 ms for 8 per lane on full warps)
  if (mode == ADJ && k > 128 && d == 4) return FAM_WIDE;
  // forward step with 9..16 centroids at d >= 2: 8 centroids per lane on lane pairs at two blocks per SM instead of 16
  // per thread at one (m = 2^24, k = 16: d = 4 0.28 against 0.50 ms, d = 2 0.19 against 0.22 ms; d = 1 0.13 against 0.12)
  if (mode == STEP && k > 8 && k <= 16 && d >= 2) return FAM_8x2;
  for (int f = 0; f <= FAM_WIDE; ++f) {
    const KernelEntry* e = kernel_entry(mode, d, f);
    if (e && e->launch && e->kpl * e->lpw >= k) return f;
  }
  return -1;
}

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// The explicit-Jacobian pass comes in two kinds: k d <= 8 (matrix in a thread's registers, at most 64 entries) and
// the tiled kind for k d <= 64, whose partials are whole matrices and which therefore runs two blocks per SM.
constexpr int JAC_SMALL_PLEN_MAX = 64;
constexpr int JAC_TILE_BLOCKS_PER_SM = 2;
// Steps of the adjoint iteration from which the tiled kind (one pass of about ten fused passes' cost) is used.
constexpr int JAC_TILE_MIN_ITERS = 16;

// The dual step kernel of (d, k), or null: it exists for the layouts (2,1) and (4,1) where the fp32 and the fp64 step
// pick the same layout and register budget.
static const DualEntry* dual_entry(int d, int k, bool delta = true) {
  const int di = d == 1 ? 0 : (d == 2 ? 1 : (d == 4 ? 2 : -1));
  const int f = pick_family(STEP, d, k);
  if (di < 0 || f < 0 || f > 1 || pick_family(STEP_PRECISE, d, k) != f || pick_family(STEP_DELTA, d, k) != f) return nullptr;
  const DualEntry* e = delta ? &k_table_dual_delta[di][f] : &k_table_dual[di][f];
  return e->launch ? e : nullptr;
}

struct WorkspaceLayout {
  size_t off_state, off_S, off_F, off_g, off_u, off_partials, off_gpartials, off_gtickets, off_sync, total;
  size_t off_hist_fwd, off_hist_adj;
  size_t off_rowstat;   // two floats per weight-vector, or NO_ROWSTAT
  size_t off_partials64, off_gpartials64, off_gtickets64;   // second set for the fp64 half of the dual step kernel
  int max_slots, max_groups, max_groups64;
};

constexpr size_t NO_ROWSTAT = ~(size_t)0;

static int device_sm_count() {
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
      sms <= 0) {
    (void)cudaGetLastError();
    return 148;
  }
  return sms;
}

static bool make_layout(int64_t m_total, int d, int k, int n_layers, int sms, WorkspaceLayout* out) {
  if (d_index(d) < 0 || k < 1 || k > IDKM_MAX_K || n_layers < 1 || n_layers > IDKM_MAX_LAYERS) return false;
  int plen_max = 1;
  size_t jac_tile_doubles = 0;   // the tiled explicit-Jacobian pass: k d x k d partials, but only two blocks per SM
  for (int mode = STEP; mode < N_MODES; ++mode) {
    const int f = pick_family(mode, d, k);
    if (f < 0 && mode == JACOBIAN) continue;   // only small codebooks have the explicit-Jacobian pass
    if (f < 0) return false;
    const int pl = kernel_entry(mode, d, f)->plen;
    if (mode == JACOBIAN && pl > JAC_SMALL_PLEN_MAX) {
      jac_tile_doubles = (size_t)(sms * JAC_TILE_BLOCKS_PER_SM + n_layers) * pl;
      continue;
    }
    if (pl > plen_max) plen_max = pl;
  }
  WorkspaceLayout w;
  size_t o = 0;
  w.off_state = o; o = align_up(o + sizeof(LayerState) * (size_t)n_layers, 256);
  w.off_S = o;     o = align_up(o + sizeof(float) * (size_t)n_layers * k, 256);
  w.off_F = o;     o = align_up(o + sizeof(float) * (size_t)n_layers * k * d, 256);
  w.off_g = o;     o = align_up(o + sizeof(float) * (size_t)n_layers * k * d, 256);
  w.off_u = o;     o = align_up(o + sizeof(float) * (size_t)n_layers * k * d, 256);
  w.max_slots = sms * MAX_BLOCKS_PER_SM + n_layers;
  size_t partial_doubles = (size_t)w.max_slots * plen_max;
  if (jac_tile_doubles > partial_doubles) partial_doubles = jac_tile_doubles;
  w.off_partials = o; o = align_up(o + sizeof(double) * partial_doubles, 256);
  w.max_groups = w.max_slots / RED_GROUP + n_layers + 2;
  w.off_gpartials = o; o = align_up(o + sizeof(double) * (size_t)w.max_groups * plen_max, 256);
  w.off_gtickets = o;  o = align_up(o + sizeof(unsigned int) * (size_t)w.max_groups, 256);
  w.off_sync = o;      o = align_up(o + 4 * sizeof(unsigned int), 256);   // barrier words of the single-launch loop
  w.off_hist_fwd = o;  o = align_up(o + sizeof(float) * (size_t)n_layers * HIST_CAP, 256);
  w.off_hist_adj = o;  o = align_up(o + sizeof(float) * (size_t)n_layers * HIST_CAP, 256);
  // second set of partial buffers for the kernel that steps the fp32 and the collapsing layers in one launch
  const bool de = dual_entry(d, k) != nullptr;
  // (the second half is the fp64 step or the fp32 increment-form step: room for the larger partial)
  const int plen64 = de ? kernel_entry(STEP_DELTA, d, pick_family(STEP_DELTA, d, k))->plen : 0;
  w.max_groups64 = de ? w.max_groups : 0;
  w.off_partials64 = o;  o = align_up(o + sizeof(double) * (size_t)w.max_slots * plen64, 256);
  w.off_gpartials64 = o; o = align_up(o + sizeof(double) * (size_t)w.max_groups64 * plen64, 256);
  w.off_gtickets64 = o;  o = align_up(o + sizeof(unsigned int) * (size_t)w.max_groups64, 256);
  // Most group-per-weight adjoint layouts read each row's softmax reference and normaliser, written by the
  // codebook-gradient pass, instead of recomputing the row minimum and the row sum in every adjoint step.  The two
  // passes must agree on the layout kind, which they do unless a tuning override forces them apart.
  const int f_adj = pick_family(ADJ, d, k), f_grad = pick_family(GRAD, d, k);
  w.off_rowstat = NO_ROWSTAT;
  if (f_adj >= 0 && f_grad >= 0) {
    const bool rd = row_cache_layout(d, kernel_entry(ADJ, d, f_adj)->lpw);
    const bool wr = row_cache_layout(d, kernel_entry(GRAD, d, f_grad)->lpw);
    if (rd && !wr) return false;
    if (rd || wr) {
      w.off_rowstat = o;
      o = align_up(o + sizeof(float2) * (size_t)m_total, 256);
    }
  }
  w.total = o;
  *out = w;
  return true;
}

}  // namespace idkm

using namespace idkm;

struct idkm_ctx {
  int device;
  int sms;
  int64_t launches;
  // last forward
  bool have_forward;
  const float* W;
  float* C;
  void* workspace;
  int64_t m_total;
  int d, k, n_layers;
  float tau;
  long long row_off[MAX_LAYERS + 1];
  cudaStream_t stream;
  int occupancy[2][N_MODES][3][N_FAMILY];   // cached blocks/SM per kernel ([1]: squared-distance variants), 0 = not queried
  // device buffers, streams and events of the host-pointer entry point
  void* hbuf;
  size_t hbuf_bytes;
  bool host_streams_ok;
  cudaStream_t hs_compute, hs_copy;
  cudaEvent_t hev[4];
  // optional phase timing (CUDA events on the call's stream)
  bool timing;
  bool ev_ok;
  bool ev_fwd_set, ev_bwd_set;
  int squared;          // 1: squared-distance variant (idkm_set_distance)
  int wq_dtype;         // element type of Wq_out: 0 fp32, 1 bf16, 2 fp16 (idkm_set_wq_dtype)
  int collapse_step;    // 0: collapsing layers step in the fp32 increment form; 1: in fp64 (idkm_set_collapse_step)
  int adjoint_method;   // 0: explicit Jacobian where k d <= 8, fused passes otherwise; 1: always fused passes
  int forward_loop;     // 0: small layers and batches of them run the whole forward loop in one cooperative launch; 1: never;
                        // 2: never, and the fp32 and fp64 steps of an iteration are always two launches
  int hook_missing_arrivals;      // host-side fault injection for the timeout path (idkm_set_test_hooks); 0 at rest
  long long hook_spin_limit;      // 0: the default bound
  int small_blocks[3][N_SMALL_FAMILY];   // cached co-resident grid of the single-launch loop kernels (0 = not queried)
  // bounded run-ahead of the tolerance-mode loops: a pinned host word the device sets when all layers are done
  int* h_flag;
  int* d_flag;
  int call_id;
  cudaEvent_t chunk_ev[2];
  bool chunk_ev_ok;
  cudaEvent_t ev[8];   // fwd: 0 start, 1 after init, 2 after steps, 3 after final; bwd: 4 start, 5 grad, 6 adj, 7 scatter
};

static void mark(idkm_ctx* ctx, int i) {
  if (ctx->timing && ctx->ev_ok) cudaEventRecord(ctx->ev[i], ctx->stream);
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// The kernel that runs a pass for this ctx: the squared-distance variant of the fused passes when the ctx asks for it.
static const KernelEntry* ctx_entry(const idkm_ctx* ctx, int mode, int family) {
  if (ctx->squared && mode <= SCATTER) return kernel_entry_sq(mode, ctx->d, family);
  return kernel_entry(mode, ctx->d, family);
}

static int blocks_per_sm(idkm_ctx* ctx, int mode, int d, int family) {
  const bool sq = ctx->squared && mode <= SCATTER;
  int& slot = ctx->occupancy[sq ? 1 : 0][mode][d_index(d)][family];
  if (slot == 0) {
    int n = 0;
    const KernelEntry* e = sq ? kernel_entry_sq(mode, d, family) : kernel_entry(mode, d, family);
    // static + dynamic shared memory can exceed the 48 KB default: raise the limit before asking for the occupancy
    if (e->dyn_smem > 0) (void)cudaFuncSetAttribute(e->func, cudaFuncAttributeMaxDynamicSharedMemorySize, e->dyn_smem);
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, e->func, BLOCK, e->dyn_smem) != cudaSuccess || n < 1) {
      (void)cudaGetLastError();
      n = 1;
    }
    slot = n > MAX_BLOCKS_PER_SM ? MAX_BLOCKS_PER_SM : n;
  }
  return slot;
}

// Tile table of one pass: tiles never span layers; blocks get contiguous tile ranges.
static int build_table(idkm_ctx* ctx, int mode, int family, LayerTable* lt) {
  const KernelEntry* e = kernel_entry(mode, ctx->d, family);
  lt->n_layers = ctx->n_layers;
  long long tiles = 0;
  for (int l = 0; l < ctx->n_layers; ++l) {
    lt->row_off[l] = ctx->row_off[l];
    lt->tile_off[l] = (int)tiles;
    const long long rows = ctx->row_off[l + 1] - ctx->row_off[l];
    tiles += (rows + e->tile - 1) / e->tile;
    if (tiles > 0x7fffffffLL / 2) return IDKM_ERR_SHAPE;
  }
  lt->row_off[ctx->n_layers] = ctx->row_off[ctx->n_layers];
  lt->tile_off[ctx->n_layers] = (int)tiles;
  for (int l = ctx->n_layers + 1; l <= MAX_LAYERS; ++l) {
    lt->row_off[l] = lt->row_off[ctx->n_layers];
    lt->tile_off[l] = 0x7fffffff;
  }
  lt->tiles_total = (int)tiles;
  long long nb = (long long)ctx->sms * blocks_per_sm(ctx, mode, ctx->d, family);
  if (mode == JACOBIAN && e->plen > JAC_SMALL_PLEN_MAX && nb > (long long)ctx->sms * JAC_TILE_BLOCKS_PER_SM)
    nb = (long long)ctx->sms * JAC_TILE_BLOCKS_PER_SM;   // the workspace holds this many matrix partials
  // (Batched loops too get one resident wave of blocks.  More blocks than fit at a time -- so that the scheduler could
  // backfill the slots of layers that have dropped out of the loop -- measured slower in every case tried: the
  // ResNet-18-shaped batch 38.5 -> 31.9 us per iteration, a tolerance-mode batch of eight layers 1.52 -> 1.36 ms; what a
  // block costs before and after its rows outweighs the idle slots.)
  if (nb > tiles) nb = tiles;
  lt->n_blocks = (int)nb;
  lt->pad = 0;
  return IDKM_OK;
}

static void fill_params(idkm_ctx* ctx, const WorkspaceLayout& wl, PassParams* p) {
  memset(p, 0, sizeof(*p));
  char* ws = static_cast<char*>(ctx->workspace);
  p->W = ctx->W;
  p->C = ctx->C;
  p->S = reinterpret_cast<float*>(ws + wl.off_S);
  p->F = reinterpret_cast<float*>(ws + wl.off_F);
  p->gvec = reinterpret_cast<float*>(ws + wl.off_g);
  p->u = reinterpret_cast<float*>(ws + wl.off_u);
  p->partials = reinterpret_cast<double*>(ws + wl.off_partials);
  p->gpartials = reinterpret_cast<double*>(ws + wl.off_gpartials);
  p->gtickets = reinterpret_cast<unsigned int*>(ws + wl.off_gtickets);
  p->hist_fwd = reinterpret_cast<float*>(ws + wl.off_hist_fwd);
  p->hist_adj = reinterpret_cast<float*>(ws + wl.off_hist_adj);
  p->st = reinterpret_cast<LayerState*>(ws + wl.off_state);
  p->rowstat = (wl.off_rowstat == NO_ROWSTAT) ? nullptr : reinterpret_cast<float2*>(ws + wl.off_rowstat);
  p->inv_tau = (float)(1.0 / (double)ctx->tau);
  p->inv_tau_d = 1.0 / (double)ctx->tau;
  p->scale = (float)(1.4426950408889634 / (double)ctx->tau);
  p->alpha = 1.f;
  p->k = ctx->k;
  p->squared = ctx->squared;
  p->wq_dtype = ctx->wq_dtype;
}

// Loops with a tolerance are queued in chunks of RUN_CHUNK iterations.  After each chunk the host peeks at the pinned
// word the device sets once every layer's loop has ended, and it waits for the chunk before the previous one, so it
// is never more than two chunks ahead of the device: a loop that converges early leaves at most 2 * RUN_CHUNK launches
// that return at once instead of (cap - iterations).  The convergence decision itself stays on the device; with
// tol = 0 everything is queued without any wait.
constexpr int RUN_CHUNK = 16;

struct RunAhead {
  idkm_ctx* ctx;
  bool on;
  int chunks;
  void begin(idkm_ctx* c, PassParams* p, bool tol_mode) {
    ctx = c;
    on = tol_mode && c->h_flag != nullptr && c->chunk_ev_ok;
    chunks = 0;
    p->host_flag = on ? c->d_flag : nullptr;
    p->call_id = on ? ++c->call_id : 0;
    if (on && c->call_id == 0x7fffffff) c->call_id = 0;
  }
  // call after iteration `it` (0-based) has been queued; true = stop queueing
  bool after(int it) {
    if (!on || (it + 1) % RUN_CHUNK != 0) return false;
    cudaEventRecord(ctx->chunk_ev[chunks & 1], ctx->stream);
    ++chunks;
    if (*reinterpret_cast<volatile int*>(ctx->h_flag) == ctx->call_id) return true;
    if (chunks >= 2) {
      cudaEventSynchronize(ctx->chunk_ev[chunks & 1]);   // the chunk before the one just queued
      if (*reinterpret_cast<volatile int*>(ctx->h_flag) == ctx->call_id) return true;
    }
    return false;
  }
};

// The forward loop: every iteration launches the fp32 step and the fp64 step; each layer is taken by exactly one
// of them (LayerState::precise), the other returns at once for it.
static int launch_step_loop(idkm_ctx* ctx, const WorkspaceLayout& wl, PassParams* p, int repeat) {
  // the step of the collapsing layers: fp32 in the increment form, or fp64
  const int mode64 = ctx->collapse_step == 0 ? STEP_DELTA : STEP_PRECISE;
  const int f32 = pick_family(STEP, ctx->d, ctx->k), f64 = pick_family(mode64, ctx->d, ctx->k);
  const KernelEntry* e32 = ctx_entry(ctx, STEP, f32);
  // forward-loop method 3: the bulk-copy variant of the fp32 step where it exists (thread-per-weight layouts)
  int bulk_per_sm = 0;
  if (ctx->forward_loop == 3 && !ctx->squared && k_table_step_bulk[d_index(ctx->d)][f32].launch) {
    e32 = &k_table_step_bulk[d_index(ctx->d)][f32];
    (void)cudaFuncSetAttribute(e32->func, cudaFuncAttributeMaxDynamicSharedMemorySize, e32->dyn_smem);
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&bulk_per_sm, e32->func, BLOCK, e32->dyn_smem) != cudaSuccess || bulk_per_sm < 1) {
      (void)cudaGetLastError();
      bulk_per_sm = 1;
    }
  }
  const KernelEntry* e64 = kernel_entry(mode64, ctx->d, f64);
  static const bool dual_off = (getenv("IDKM_NO_DUAL") != nullptr);   // tuning knob: always two launches per iteration
  const DualEntry* de = (dual_off || ctx->forward_loop >= 2 || ctx->squared) ? nullptr
                                                                             : dual_entry(ctx->d, ctx->k, mode64 == STEP_DELTA);
  PassParams q = *p;
  int rc = build_table(ctx, STEP, f32, &p->lt);
  if (rc != IDKM_OK) return rc;
  if (bulk_per_sm > 0 && ctx->n_layers == 1) {   // the stages take shared memory: fewer blocks may fit than the table assumed
    const long long nbb = (long long)ctx->sms * (bulk_per_sm > MAX_BLOCKS_PER_SM ? MAX_BLOCKS_PER_SM : bulk_per_sm);
    if (p->lt.n_blocks > nbb) p->lt.n_blocks = (int)nbb;
  }
  rc = build_table(ctx, mode64, f64, &q.lt);
  if (rc != IDKM_OK) return rc;
  int dual_grid = 0;
  if (de) {
    // one grid runs both halves: each half's table may use at most that many blocks
    char* ws = static_cast<char*>(ctx->workspace);
    q.partials = reinterpret_cast<double*>(ws + wl.off_partials64);
    q.gpartials = reinterpret_cast<double*>(ws + wl.off_gpartials64);
    q.gtickets = reinterpret_cast<unsigned int*>(ws + wl.off_gtickets64);
    dual_grid = p->lt.n_blocks > q.lt.n_blocks ? p->lt.n_blocks : q.lt.n_blocks;
  }
  RunAhead ra;
  ra.begin(ctx, p, p->tol > 0.f);
  q.host_flag = p->host_flag;
  q.call_id = p->call_id;
  for (int it = 0; it < repeat; ++it) {
    p->iter = q.iter = it;
    if (de) {
      DualParams dp;
      dp.p = *p;
      dp.q = q;
      if (de->launch(dp, dual_grid, ctx->stream) != cudaSuccess) return IDKM_ERR_CUDA;
      ctx->launches += 1;
    } else {
      if (e32->launch(*p, p->lt.n_blocks, ctx->stream) != cudaSuccess) return IDKM_ERR_CUDA;
      ctx->launches += 1;
      if (!ctx->squared) {   // (the squared-distance variant never hands a layer to the fp64 step)
        if (e64->launch(q, q.lt.n_blocks, ctx->stream) != cudaSuccess) return IDKM_ERR_CUDA;
        ctx->launches += 1;
      }
    }
    if (ra.after(it)) break;
  }
  p->host_flag = nullptr;
  return IDKM_OK;
}

// The single-launch loop of idkm_small_loop.cu takes layers with k <= 16 (k <= 8 for d = 4): a single layer whose rows
// fit SMALL_ROWS_PER_THREAD per thread of the co-resident grid -- about 9.7 million rows on a 148-SM part, 4.8 million at
// d = 4 (measured against a launch per iteration at m = 5 .. 9.5 million: 11.6 against 17.4 us at d = 1, k = 2, m = 5 M;
// 22.8 against 24.4 us at d = 1, k = 4, m = 9.5 M; d = 4, k = 8, collapsing, m = 5 M: 85 against 66 us, hence the lower
// limit there) -- or a batch of up to as many layers as the grid has blocks, with up to SMALL_BATCH_ROWS_PER_THREAD rows
// per thread; either way at most SMALL_MAX_FLOATS weights in all (a batch pays more per iteration on the tiled path:
// every block there walks several layers, each with its own chain of block sums and tickets).  The blocks are dealt out
// to the layers in proportion to their rows, at least one each, and at least SMALL_MIN_ROWS_PER_THREAD rows per thread:
// tiny layers use few blocks, which keeps the cross-block sum short.
constexpr int SMALL_ROWS_PER_THREAD = 128;      // a single layer, d <= 2
constexpr int SMALL_ROWS_PER_THREAD_D4 = 64;    // a single layer, d = 4 (one row per 128-bit load)
constexpr int SMALL_BATCH_ROWS_PER_THREAD = 256;
constexpr long long SMALL_MAX_FLOATS = 20LL << 20;   // 80 MB of weights: they stay in the 126 MB L2 across iterations
constexpr int SMALL_CHUNK_ROWS = 32;   // threads with more rows than this move their fp32 sums out every 32 rows
constexpr int SMALL_MIN_ROWS_PER_THREAD = 4;
constexpr long long SMALL_SOLO_ROWS = 4096;   // a single layer up to this size runs on one block ...
constexpr long long SMALL_SOLO_WORK = 32768;  // ... if rows x centroids x d stays below this (d = 4, k = 8: 1024 rows)
constexpr long long SMALL_SPIN_LIMIT = 2000000000LL;   // about a second of SM clock ticks per barrier wait

// Returns IDKM_OK after queueing the loop, 1 if this problem should take the launch-per-iteration path.
static int try_small_loop(idkm_ctx* ctx, const WorkspaceLayout& wl, const PassParams& p, int max_iter) {
  static const bool env_off = (getenv("IDKM_NO_COOP") != nullptr);   // tuning knob: always a launch per iteration
  // (the loop kernel steps a collapsing layer in the fp32 increment form; the fp64 step exists as launches only)
  if (env_off || ctx->forward_loop != 0 || max_iter < 2 || ctx->squared || ctx->collapse_step != 0)
    return 1;
  const int di = d_index(ctx->d);
  int f = -1;
  for (int q = 0; q < N_SMALL_FAMILY; ++q)
    if (k_table_small[di][q].launch && k_table_small[di][q].kpl >= ctx->k) { f = q; break; }
  if (f < 0) return 1;
  const SmallLoopEntry* se = &k_table_small[di][f];
  int& nb = ctx->small_blocks[di][f];
  if (nb == 0) {
    int coop = 0, per_sm = 0;
    nb = -1;
    if (cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, ctx->device) == cudaSuccess && coop &&
        cudaFuncSetAttribute(se->func, cudaFuncAttributeMaxDynamicSharedMemorySize, se->dyn_smem) == cudaSuccess &&
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, se->func, BLOCK, se->dyn_smem) == cudaSuccess && per_sm >= 1)
      nb = ctx->sms * (per_sm > 2 ? 2 : per_sm);
    (void)cudaGetLastError();
  }
  if (nb <= 0) return 1;
  const int L = ctx->n_layers;
  const long long m = ctx->m_total;
  if (L > nb || L > MAX_LAYERS) return 1;
  const int per_thread = L > 1 ? SMALL_BATCH_ROWS_PER_THREAD : (ctx->d == 4 ? SMALL_ROWS_PER_THREAD_D4 : SMALL_ROWS_PER_THREAD);
  if (m > (long long)per_thread * nb * BLOCK) return 1;
  // (weights that do not stay in L2 are faster by a launch per iteration, whose kernels keep more loads in flight:
  // 16 x 1 M rows at d = 2, k = 2: 68 against 38 us per iteration; 8 x 1 M at d = 4, k = 2: 65 against 41 us)
  if (m * ctx->d > SMALL_MAX_FLOATS) return 1;
  long long grid = (m + (long long)SMALL_MIN_ROWS_PER_THREAD * BLOCK - 1) / ((long long)SMALL_MIN_ROWS_PER_THREAD * BLOCK);
  if (grid > nb) grid = nb;
  // a single layer of a few thousand weights: one block, which then skips the partial buffers and the barrier
  // (m = 4096, d = 1, k = 4: 2.6 against 4.7 us per iteration on four blocks; d = 4, k = 8 at that size is faster spread out)
  if (L == 1 && m <= SMALL_SOLO_ROWS && m * ctx->k * ctx->d <= SMALL_SOLO_WORK) grid = 1;
  if (grid < L) grid = L;
  if (2 * grid > wl.max_slots) return 1;   // the two partial buffers live in the partial-slot region
  SmallLoopParams sp;
  memset(&sp, 0, sizeof(sp));
  sp.W = ctx->W;
  sp.n_layers = L;
  // blocks per layer: one each, the rest in proportion to the rows (largest remainders first)
  int cnt[MAX_LAYERS];
  long long rem[MAX_LAYERS];
  int given = 0;
  const long long spare = grid - L;
  for (int l = 0; l < L; ++l) {
    const long long rows = ctx->row_off[l + 1] - ctx->row_off[l];
    const long long share = (m > 0) ? spare * rows / m : 0;
    cnt[l] = 1 + (int)share;
    rem[l] = (m > 0) ? spare * rows % m : 0;
    given += cnt[l];
    sp.row_off[l] = ctx->row_off[l];
  }
  sp.row_off[L] = ctx->row_off[L];
  while (given < grid) {
    int best = 0;
    for (int l = 1; l < L; ++l)
      if (rem[l] > rem[best]) best = l;
    ++cnt[best];
    rem[best] = -1;
    ++given;
  }
  long long max_rows_per_thread = 0;
  sp.blk_first[0] = 0;
  for (int l = 0; l < L; ++l) {
    sp.blk_first[l + 1] = sp.blk_first[l] + cnt[l];
    const long long rows = ctx->row_off[l + 1] - ctx->row_off[l];
    const long long per = (rows + (long long)cnt[l] * BLOCK - 1) / ((long long)cnt[l] * BLOCK);
    if (per > max_rows_per_thread) max_rows_per_thread = per;
  }
  for (int l = L + 1; l <= MAX_LAYERS; ++l) {
    sp.blk_first[l] = sp.blk_first[L];
    sp.row_off[l] = sp.row_off[L];
  }
  sp.C = ctx->C;
  sp.st = p.st;
  sp.partials = p.partials;
  sp.sync = reinterpret_cast<unsigned int*>(static_cast<char*>(ctx->workspace) + wl.off_sync);
  sp.k = ctx->k;
  sp.scale = p.scale;
  sp.tol = p.tol;
  sp.inv_tau_d = p.inv_tau_d;
  sp.max_iter = max_iter;
  sp.hist = p.hist_fwd;
  sp.chunked = (max_rows_per_thread > SMALL_CHUNK_ROWS) ? 1 : 0;
  sp.spin_limit = SMALL_SPIN_LIMIT;
  // Host-side fault injection for tests of the timeout path (idkm_set_test_hooks; no GPU fault involved: the waits
  // are bounded and the kernel returns)
  sp.missing_arrivals = ctx->hook_missing_arrivals;
  if (ctx->hook_spin_limit > 0 && ctx->hook_spin_limit < SMALL_SPIN_LIMIT) sp.spin_limit = ctx->hook_spin_limit;
  if (se->launch(sp, (int)grid, ctx->stream) != cudaSuccess) {
    (void)cudaGetLastError();
    return 1;   // nothing was queued: take the launch-per-iteration path
  }
  ++ctx->launches;
  return IDKM_OK;
}

static int launch_pass(idkm_ctx* ctx, int mode, PassParams* p, int repeat) {
  const int f = pick_family(mode, ctx->d, ctx->k);
  const KernelEntry* e = ctx_entry(ctx, mode, f);
  const int rc = build_table(ctx, mode, f, &p->lt);
  if (rc != IDKM_OK) return rc;
  RunAhead ra;
  ra.begin(ctx, p, mode == ADJ && p->tol > 0.f && repeat > 1);
  for (int it = 0; it < repeat; ++it) {
    if (e->launch(*p, p->lt.n_blocks, ctx->stream) != cudaSuccess) return IDKM_ERR_CUDA;
    ++ctx->launches;
    if (ra.after(it)) break;
  }
  p->host_flag = nullptr;
  return IDKM_OK;
}

// The last phase of a backward: the pass that writes dL/dW from the adjoint u in the workspace, and the copy of u.
static int backward_outputs(idkm_ctx* ctx, PassParams* p, float* dW_out, float* dC_out) {
  if (dW_out) {
    p->dW = dW_out;
    nvtxRangePushA("idkm dL/dW pass");
    const int rc = launch_pass(ctx, SCATTER, p, 1);
    nvtxRangePop();
    if (rc != IDKM_OK) return rc;
  }
  mark(ctx, 7);
  ctx->ev_bwd_set = ctx->timing && ctx->ev_ok;
  if (dC_out) {
    if (cudaMemcpyAsync(dC_out, p->u, sizeof(float) * (size_t)ctx->n_layers * ctx->k * ctx->d, cudaMemcpyDeviceToDevice,
                        ctx->stream) != cudaSuccess)
      return IDKM_ERR_CUDA;
  }
  return IDKM_OK;
}

extern "C" {

int idkm_create(idkm_ctx** out) {
  if (!out) return IDKM_ERR_NULL;
  idkm_ctx* c = new (std::nothrow) idkm_ctx;
  if (!c) return IDKM_ERR_CUDA;
  memset(c, 0, sizeof(*c));
  if (cudaGetDevice(&c->device) != cudaSuccess ||
      cudaDeviceGetAttribute(&c->sms, cudaDevAttrMultiProcessorCount, c->device) != cudaSuccess || c->sms < 1) {
    (void)cudaGetLastError();
    delete c;
    return IDKM_ERR_CUDA;
  }
  // optional: without mapped pinned memory the tolerance-mode loops simply queue every iteration
  if (cudaHostAlloc(reinterpret_cast<void**>(&c->h_flag), sizeof(int), cudaHostAllocMapped) == cudaSuccess) {
    *c->h_flag = 0;
    if (cudaHostGetDevicePointer(reinterpret_cast<void**>(&c->d_flag), c->h_flag, 0) != cudaSuccess) {
      cudaFreeHost(c->h_flag);
      c->h_flag = c->d_flag = nullptr;
    }
  } else {
    c->h_flag = c->d_flag = nullptr;
  }
  (void)cudaGetLastError();
  if (c->h_flag && cudaEventCreateWithFlags(&c->chunk_ev[0], cudaEventDisableTiming) == cudaSuccess) {
    if (cudaEventCreateWithFlags(&c->chunk_ev[1], cudaEventDisableTiming) == cudaSuccess) c->chunk_ev_ok = true;
    else cudaEventDestroy(c->chunk_ev[0]);
  }
  (void)cudaGetLastError();
  *out = c;
  return IDKM_OK;
}

void idkm_destroy(idkm_ctx* ctx) {
  if (!ctx) return;
  if (ctx->hbuf) cudaFree(ctx->hbuf);
  if (ctx->host_streams_ok) {
    for (int i = 0; i < 4; ++i) cudaEventDestroy(ctx->hev[i]);
    cudaStreamDestroy(ctx->hs_compute);
    cudaStreamDestroy(ctx->hs_copy);
  }
  if (ctx->chunk_ev_ok) {
    cudaEventDestroy(ctx->chunk_ev[0]);
    cudaEventDestroy(ctx->chunk_ev[1]);
  }
  if (ctx->h_flag) cudaFreeHost(ctx->h_flag);
  if (ctx->ev_ok)
    for (int i = 0; i < 8; ++i) cudaEventDestroy(ctx->ev[i]);
  delete ctx;
}

size_t idkm_workspace_bytes(int64_t m_total, int d, int k, int n_layers) {
  WorkspaceLayout wl;
  if (m_total < 1 || !make_layout(m_total, d, k, n_layers, device_sm_count(), &wl)) return 0;
  return wl.total;
}

int idkm_forward_batched(idkm_ctx* ctx, const float* W_cat, const int64_t* layer_offsets, int n_layers, int d,
                         const float* C0, int k, float tau, float tol, int max_iter, float* C_out, float* A_out,
                         float* Wq_out, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!ctx || !W_cat || !layer_offsets || !C0 || !C_out || !workspace) return IDKM_ERR_NULL;
  if (d_index(d) < 0 || k < 1 || k > IDKM_MAX_K) return IDKM_ERR_UNSUPPORTED;
  if (n_layers < 1 || n_layers > IDKM_MAX_LAYERS) return IDKM_ERR_SHAPE;
  if (layer_offsets[0] != 0) return IDKM_ERR_SHAPE;
  for (int l = 0; l < n_layers; ++l)
    if (layer_offsets[l + 1] <= layer_offsets[l]) return IDKM_ERR_SHAPE;
  const int64_t m_total = layer_offsets[n_layers];
  if (m_total < 1 || m_total > (1LL << 40) / (k > d ? k : d)) return IDKM_ERR_SHAPE;
  if (!(tau > 0.f) || !isfinite(tau) || !(tol >= 0.f) || !isfinite(tol) || max_iter < 0) return IDKM_ERR_PARAM;
  if (!aligned16(W_cat) || !aligned16(C0) || !aligned16(C_out) || !aligned16(workspace) ||
      (A_out && !aligned16(A_out)) || (Wq_out && !aligned16(Wq_out)))
    return IDKM_ERR_ALIGN;
  WorkspaceLayout wl;
  if (!make_layout(m_total, d, k, n_layers, ctx->sms, &wl)) return IDKM_ERR_UNSUPPORTED;
  if (workspace_bytes < wl.total) return IDKM_ERR_WORKSPACE;

  ctx->have_forward = false;
  ctx->W = W_cat;
  ctx->C = C_out;
  ctx->workspace = workspace;
  ctx->m_total = m_total;
  ctx->d = d;
  ctx->k = k;
  ctx->n_layers = n_layers;
  ctx->tau = tau;
  ctx->stream = static_cast<cudaStream_t>(cuda_stream);
  for (int l = 0; l <= n_layers; ++l) ctx->row_off[l] = layer_offsets[l];

  PassParams p;
  fill_params(ctx, wl, &p);
  p.tol = tol;
  p.max_iter = max_iter;

  ctx->ev_fwd_set = ctx->ev_bwd_set = false;
  mark(ctx, 0);
  const int n_coord = n_layers * k * d;
  const int init_threads = n_coord > n_layers ? n_coord : n_layers;
  idkm_init_forward<<<(init_threads + 255) / 256, 256, 0, ctx->stream>>>(p.st, n_layers, C0, C_out, n_coord, k, d,
                                                                                     p.inv_tau_d, p.gtickets, wl.max_groups,
                                                                                     reinterpret_cast<unsigned int*>(static_cast<char*>(workspace) + wl.off_sync),
                                                                                     reinterpret_cast<unsigned int*>(static_cast<char*>(workspace) + wl.off_gtickets64),
                                                                                     wl.max_groups64, ctx->squared);
  if (cudaGetLastError() != cudaSuccess) return IDKM_ERR_CUDA;
  ++ctx->launches;
  mark(ctx, 1);

  nvtxRangePushA("idkm forward loop");
  int rc = try_small_loop(ctx, wl, p, max_iter);
  if (rc == 1) rc = launch_step_loop(ctx, wl, &p, max_iter);
  nvtxRangePop();
  if (rc != IDKM_OK) return rc;
  mark(ctx, 2);
  p.Wq = Wq_out;
  p.A = A_out;
  nvtxRangePushA("idkm final pass");
  rc = launch_pass(ctx, FINAL, &p, 1);
  nvtxRangePop();
  if (rc != IDKM_OK) return rc;
  mark(ctx, 3);
  ctx->ev_fwd_set = ctx->timing && ctx->ev_ok;
  ctx->have_forward = true;
  return IDKM_OK;
}

int idkm_forward(idkm_ctx* ctx, const float* W, int64_t m, int d, const float* C0, int k, float tau, float tol,
                 int max_iter, float* C_out, float* A_out, float* Wq_out, void* workspace, size_t workspace_bytes,
                 void* cuda_stream) {
  if (m < 1) return ctx ? IDKM_ERR_SHAPE : IDKM_ERR_NULL;
  const int64_t offs[2] = {0, m};
  return idkm_forward_batched(ctx, W, offs, 1, d, C0, k, tau, tol, max_iter, C_out, A_out, Wq_out, workspace,
                              workspace_bytes, cuda_stream);
}

int idkm_backward(idkm_ctx* ctx, const float* dWq, idkm_mode mode, float adj_tol, int adj_max_iter, float alpha,
                  float* dW_out, float* dC_out, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!ctx || !dWq || !workspace) return IDKM_ERR_NULL;
  if (!ctx->have_forward) return IDKM_ERR_ORDER;
  if (workspace != ctx->workspace) return IDKM_ERR_ORDER;
  if (mode != IDKM_IMPLICIT && mode != IDKM_JFB) return IDKM_ERR_PARAM;
  if (!(adj_tol >= 0.f) || !isfinite(adj_tol) || adj_max_iter < 0 || !(alpha > 0.f) || !(alpha <= 1.f))
    return IDKM_ERR_PARAM;
  if (!aligned16(dWq) || (dW_out && !aligned16(dW_out)) || (dC_out && !aligned16(dC_out))) return IDKM_ERR_ALIGN;
  if (dW_out && (dW_out == dWq || dW_out == ctx->W)) return IDKM_ERR_PARAM;
  WorkspaceLayout wl;
  if (!make_layout(ctx->m_total, ctx->d, ctx->k, ctx->n_layers, ctx->sms, &wl)) return IDKM_ERR_UNSUPPORTED;
  if (workspace_bytes < wl.total) return IDKM_ERR_WORKSPACE;
  ctx->stream = static_cast<cudaStream_t>(cuda_stream);

  PassParams p;
  fill_params(ctx, wl, &p);
  p.G = dWq;
  p.tol = adj_tol;
  p.max_iter = adj_max_iter;
  p.alpha = alpha;
  ctx->ev_bwd_set = false;
  const bool solve = (mode == IDKM_IMPLICIT && adj_max_iter > 0);
  const int fj = pick_family(JACOBIAN, ctx->d, ctx->k);
  const bool jac_tile = fj >= 0 && kernel_entry(JACOBIAN, ctx->d, fj)->plen > JAC_SMALL_PLEN_MAX;
  // (the explicit-Jacobian kernels are written for the Euclidean distance: the squared variant takes the fused passes)
  const bool exact = ctx->adjoint_method == 2 && !ctx->squared && fj >= 0;   // solve on the explicit matrix
  const bool explicit_jac = exact || (ctx->adjoint_method == 0 && !ctx->squared && fj >= 0 &&
                                      (!jac_tile || adj_max_iter >= JAC_TILE_MIN_ITERS));
  // the per-row softmax reference and normaliser are kept only if fused adjoint passes follow
  if (!solve || explicit_jac) p.rowstat = nullptr;
  mark(ctx, 4);
  nvtxRangePushA("idkm codebook gradient");
  int rc = launch_pass(ctx, GRAD, &p, 1);
  nvtxRangePop();
  if (rc != IDKM_OK) return rc;
  mark(ctx, 5);
  if (solve) {
    nvtxRangePushA("idkm adjoint solve");
    if (explicit_jac) {
      if (exact) p.max_iter = -1;                  // the epilogue solves (I - J^T) u = g instead of iterating
      rc = launch_pass(ctx, JACOBIAN, &p, 1);      // one pass forms J_C; the whole iteration runs on it in the epilogue
      p.max_iter = adj_max_iter;
    } else {
      rc = launch_pass(ctx, ADJ, &p, adj_max_iter);
    }
    nvtxRangePop();
    if (rc != IDKM_OK) return rc;
  }
  mark(ctx, 6);
  return backward_outputs(ctx, &p, dW_out, dC_out);
}

int idkm_backward_restart(idkm_ctx* ctx, const float* dWq, float adj_tol, int adj_max_iter, float alpha0,
                          int max_halvings, float* dW_out, float* dC_out, void* workspace, size_t workspace_bytes,
                          void* cuda_stream, float* alpha_used_out, int* attempts_out) {
  if (!ctx || !dWq || !workspace) return IDKM_ERR_NULL;
  if (max_halvings < 0 || max_halvings > 30) return IDKM_ERR_PARAM;
  if (dW_out && (!aligned16(dW_out) || dW_out == dWq || dW_out == ctx->W)) return dW_out == dWq || dW_out == ctx->W ? IDKM_ERR_PARAM : IDKM_ERR_ALIGN;
  if (dC_out && !aligned16(dC_out)) return IDKM_ERR_ALIGN;
  float alpha = alpha0;
  int attempts = 0;
  for (;;) {
    // codebook gradient and adjoint solve only: the dL/dW pass waits for an iteration that did not diverge
    int rc = idkm_backward(ctx, dWq, IDKM_IMPLICIT, adj_tol, adj_max_iter, alpha, nullptr, nullptr, workspace,
                           workspace_bytes, cuda_stream);
    if (rc != IDKM_OK) return rc;
    ++attempts;
    idkm_info info[MAX_LAYERS];
    rc = idkm_get_info(ctx, info);   // waits for the stream: the decision to start over is the host's
    if (rc != IDKM_OK) return rc;
    bool diverged = false;
    for (int l = 0; l < ctx->n_layers; ++l) diverged = diverged || (info[l].status == IDKM_ERR_DIVERGED);
    if (!diverged || attempts > max_halvings) break;
    alpha *= 0.5f;
  }
  if (alpha_used_out) *alpha_used_out = alpha;
  if (attempts_out) *attempts_out = attempts;
  WorkspaceLayout wl;
  if (!make_layout(ctx->m_total, ctx->d, ctx->k, ctx->n_layers, ctx->sms, &wl)) return IDKM_ERR_UNSUPPORTED;
  PassParams p;
  fill_params(ctx, wl, &p);
  p.G = dWq;
  p.alpha = alpha;
  return backward_outputs(ctx, &p, dW_out, dC_out);
}

int idkm_get_info(idkm_ctx* ctx, idkm_info* info_out) {
  if (!ctx || !info_out) return IDKM_ERR_NULL;
  if (!ctx->have_forward) return IDKM_ERR_ORDER;
  WorkspaceLayout wl;
  if (!make_layout(ctx->m_total, ctx->d, ctx->k, ctx->n_layers, ctx->sms, &wl)) return IDKM_ERR_UNSUPPORTED;
  LayerState host[MAX_LAYERS];
  if (cudaStreamSynchronize(ctx->stream) != cudaSuccess) return IDKM_ERR_CUDA;
  if (cudaMemcpy(host, static_cast<char*>(ctx->workspace) + wl.off_state, sizeof(LayerState) * (size_t)ctx->n_layers,
                 cudaMemcpyDeviceToHost) != cudaSuccess)
    return IDKM_ERR_CUDA;
  for (int l = 0; l < ctx->n_layers; ++l) {
    info_out[l].status = host[l].status;
    info_out[l].fwd_iters = host[l].fwd_iters;
    info_out[l].fwd_residual = host[l].fwd_res;
    info_out[l].dead_clusters = host[l].dead;
    info_out[l].adj_iters = host[l].adj_iters;
    info_out[l].adj_residual = host[l].adj_res;
  }
  return IDKM_OK;
}

int idkm_quantize_host_ex(idkm_ctx* ctx, const float* W_host, const int64_t* layer_offsets, int n_layers, int d,
                          const float* C0_host, int k, float tau, float tol, int max_iter, const float* dWq_host,
                          idkm_mode mode, float adj_tol, int adj_max_iter, float alpha, float* C_out_host,
                          float* Wq_out_host, float* dW_out_host, float* dC_out_host, float* dW_jfb_out_host,
                          float* dC_jfb_out_host, idkm_info* info_out) {
  if (!ctx || !W_host || !layer_offsets || !C0_host || !dWq_host || !C_out_host) return IDKM_ERR_NULL;
  if (d_index(d) < 0 || k < 1 || k > IDKM_MAX_K) return IDKM_ERR_UNSUPPORTED;
  if (n_layers < 1 || n_layers > IDKM_MAX_LAYERS || layer_offsets[0] != 0) return IDKM_ERR_SHAPE;
  const int64_t m = layer_offsets[n_layers];
  if (m < 1) return IDKM_ERR_SHAPE;
  const size_t ws_bytes = idkm_workspace_bytes(m, d, k, n_layers);
  if (ws_bytes == 0) return IDKM_ERR_UNSUPPORTED;
  const bool also_jfb = (dW_jfb_out_host != nullptr || dC_jfb_out_host != nullptr) && mode == IDKM_IMPLICIT;
  const size_t wbytes = align_up(sizeof(float) * (size_t)m * d, 256);
  const size_t cbytes = align_up(sizeof(float) * (size_t)n_layers * k * d, 256);
  // W, G, Wq, dW, dW (Jacobian-free) | C0, C, dC, dC (Jacobian-free) | workspace
  const size_t need = 5 * wbytes + 4 * cbytes + align_up(ws_bytes, 256);
  if (need > ctx->hbuf_bytes) {
    if (ctx->hbuf) cudaFree(ctx->hbuf);
    ctx->hbuf = nullptr;
    ctx->hbuf_bytes = 0;
    if (cudaMalloc(&ctx->hbuf, need) != cudaSuccess) {
      (void)cudaGetLastError();
      return IDKM_ERR_CUDA;
    }
    ctx->hbuf_bytes = need;
  }
  // two streams of the ctx's own: the kernels run on one, the copies that can overlap them on the other
  if (!ctx->host_streams_ok) {
    if (cudaStreamCreateWithFlags(&ctx->hs_compute, cudaStreamNonBlocking) != cudaSuccess) return IDKM_ERR_CUDA;
    if (cudaStreamCreateWithFlags(&ctx->hs_copy, cudaStreamNonBlocking) != cudaSuccess) {
      cudaStreamDestroy(ctx->hs_compute);
      return IDKM_ERR_CUDA;
    }
    for (int i = 0; i < 4; ++i)
      if (cudaEventCreateWithFlags(&ctx->hev[i], cudaEventDisableTiming) != cudaSuccess) {
        for (int q = 0; q < i; ++q) cudaEventDestroy(ctx->hev[q]);
        cudaStreamDestroy(ctx->hs_compute);
        cudaStreamDestroy(ctx->hs_copy);
        return IDKM_ERR_CUDA;
      }
    ctx->host_streams_ok = true;
  }
  char* base = static_cast<char*>(ctx->hbuf);
  float* dW_ = reinterpret_cast<float*>(base);
  float* dG = reinterpret_cast<float*>(base + wbytes);
  float* dWq = reinterpret_cast<float*>(base + 2 * wbytes);
  float* ddW = reinterpret_cast<float*>(base + 3 * wbytes);
  float* ddWj = reinterpret_cast<float*>(base + 4 * wbytes);
  float* dC0 = reinterpret_cast<float*>(base + 5 * wbytes);
  float* dC = reinterpret_cast<float*>(base + 5 * wbytes + cbytes);
  float* ddC = reinterpret_cast<float*>(base + 5 * wbytes + 2 * cbytes);
  float* ddCj = reinterpret_cast<float*>(base + 5 * wbytes + 3 * cbytes);
  void* ws = base + 5 * wbytes + 4 * cbytes;
  cudaStream_t s = ctx->hs_compute, sc = ctx->hs_copy;
  const size_t wn = sizeof(float) * (size_t)m * d, cn = sizeof(float) * (size_t)n_layers * k * d;
#define IDKM_TRY(call) do { if ((call) != cudaSuccess) { (void)cudaGetLastError(); cudaStreamSynchronize(s); cudaStreamSynchronize(sc); return IDKM_ERR_CUDA; } } while (0)
  // W and C0 go first on the compute stream; the upstream gradient is uploaded on the copy stream while the forward
  // loop runs (it is first read by the backward)
  IDKM_TRY(cudaMemcpyAsync(dW_, W_host, wn, cudaMemcpyHostToDevice, s));
  IDKM_TRY(cudaMemcpyAsync(dC0, C0_host, cn, cudaMemcpyHostToDevice, s));
  IDKM_TRY(cudaMemcpyAsync(dG, dWq_host, wn, cudaMemcpyHostToDevice, sc));
  IDKM_TRY(cudaEventRecord(ctx->hev[0], sc));
  const int wq_dtype_saved = ctx->wq_dtype;
  ctx->wq_dtype = 0;   // the host buffers of this entry point are fp32
  int rc = idkm_forward_batched(ctx, dW_, layer_offsets, n_layers, d, dC0, k, tau, tol, max_iter, dC, nullptr,
                                Wq_out_host ? dWq : nullptr, ws, ws_bytes, s);
  ctx->wq_dtype = wq_dtype_saved;
  if (rc != IDKM_OK) { cudaStreamSynchronize(s); cudaStreamSynchronize(sc); return rc; }
  // C and Wq go back on the copy stream while the backward runs
  IDKM_TRY(cudaEventRecord(ctx->hev[1], s));
  IDKM_TRY(cudaStreamWaitEvent(sc, ctx->hev[1], 0));
  IDKM_TRY(cudaMemcpyAsync(C_out_host, dC, cn, cudaMemcpyDeviceToHost, sc));
  if (Wq_out_host) IDKM_TRY(cudaMemcpyAsync(Wq_out_host, dWq, wn, cudaMemcpyDeviceToHost, sc));
  IDKM_TRY(cudaStreamWaitEvent(s, ctx->hev[0], 0));
  if (also_jfb) {
    rc = idkm_backward(ctx, dG, IDKM_JFB, 0.f, 0, 1.f, dW_jfb_out_host ? ddWj : nullptr, dC_jfb_out_host ? ddCj : nullptr,
                       ws, ws_bytes, s);
    if (rc != IDKM_OK) { cudaStreamSynchronize(s); cudaStreamSynchronize(sc); return rc; }
    IDKM_TRY(cudaEventRecord(ctx->hev[2], s));
    IDKM_TRY(cudaStreamWaitEvent(sc, ctx->hev[2], 0));
    if (dW_jfb_out_host) IDKM_TRY(cudaMemcpyAsync(dW_jfb_out_host, ddWj, wn, cudaMemcpyDeviceToHost, sc));
    if (dC_jfb_out_host) IDKM_TRY(cudaMemcpyAsync(dC_jfb_out_host, ddCj, cn, cudaMemcpyDeviceToHost, sc));
  }
  rc = idkm_backward(ctx, dG, mode, adj_tol, adj_max_iter, alpha, dW_out_host ? ddW : nullptr,
                     dC_out_host ? ddC : nullptr, ws, ws_bytes, s);
  if (rc != IDKM_OK) { cudaStreamSynchronize(s); cudaStreamSynchronize(sc); return rc; }
  if (dW_out_host) IDKM_TRY(cudaMemcpyAsync(dW_out_host, ddW, wn, cudaMemcpyDeviceToHost, s));
  if (dC_out_host) IDKM_TRY(cudaMemcpyAsync(dC_out_host, ddC, cn, cudaMemcpyDeviceToHost, s));
#undef IDKM_TRY
  if (cudaStreamSynchronize(sc) != cudaSuccess || cudaStreamSynchronize(s) != cudaSuccess) return IDKM_ERR_CUDA;
  if (info_out) return idkm_get_info(ctx, info_out);
  return IDKM_OK;
}

int idkm_quantize_host(idkm_ctx* ctx, const float* W_host, const int64_t* layer_offsets, int n_layers, int d,
                       const float* C0_host, int k, float tau, float tol, int max_iter, const float* dWq_host,
                       idkm_mode mode, float adj_tol, int adj_max_iter, float alpha, float* C_out_host,
                       float* Wq_out_host, float* dW_out_host, float* dC_out_host, idkm_info* info_out) {
  return idkm_quantize_host_ex(ctx, W_host, layer_offsets, n_layers, d, C0_host, k, tau, tol, max_iter, dWq_host, mode,
                               adj_tol, adj_max_iter, alpha, C_out_host, Wq_out_host, dW_out_host, dC_out_host, nullptr,
                               nullptr, info_out);
}

int idkm_set_timing(idkm_ctx* ctx, int enable) {
  if (!ctx) return IDKM_ERR_NULL;
  if (enable && !ctx->ev_ok) {
    for (int i = 0; i < 8; ++i)
      if (cudaEventCreate(&ctx->ev[i]) != cudaSuccess) {
        for (int q = 0; q < i; ++q) cudaEventDestroy(ctx->ev[q]);
        (void)cudaGetLastError();
        return IDKM_ERR_CUDA;
      }
    ctx->ev_ok = true;
  }
  ctx->timing = enable != 0;
  ctx->ev_fwd_set = ctx->ev_bwd_set = false;
  return IDKM_OK;
}

int idkm_get_phase_ms(idkm_ctx* ctx, float* ms_out) {
  if (!ctx || !ms_out) return IDKM_ERR_NULL;
  for (int i = 0; i < 6; ++i) ms_out[i] = -1.f;
  if (ctx->ev_fwd_set) {
    if (cudaEventSynchronize(ctx->ev[3]) != cudaSuccess) return IDKM_ERR_CUDA;
    for (int i = 0; i < 3; ++i)
      if (cudaEventElapsedTime(&ms_out[i], ctx->ev[i], ctx->ev[i + 1]) != cudaSuccess) return IDKM_ERR_CUDA;
  }
  if (ctx->ev_bwd_set) {
    if (cudaEventSynchronize(ctx->ev[7]) != cudaSuccess) return IDKM_ERR_CUDA;
    for (int i = 0; i < 3; ++i)
      if (cudaEventElapsedTime(&ms_out[3 + i], ctx->ev[4 + i], ctx->ev[5 + i]) != cudaSuccess) return IDKM_ERR_CUDA;
  }
  return IDKM_OK;
}

int idkm_set_adjoint_method(idkm_ctx* ctx, int method) {
  if (!ctx) return IDKM_ERR_NULL;
  if (method < 0 || method > 2) return IDKM_ERR_PARAM;
  ctx->adjoint_method = method;
  return IDKM_OK;
}

int idkm_get_history(idkm_ctx* ctx, int which, int layer, float* host_out, int capacity, int* n_out) {
  if (!ctx || !host_out || !n_out) return IDKM_ERR_NULL;
  if (!ctx->have_forward) return IDKM_ERR_ORDER;
  if ((which != 0 && which != 1) || layer < 0 || layer >= ctx->n_layers || capacity < 0) return IDKM_ERR_PARAM;
  WorkspaceLayout wl;
  if (!make_layout(ctx->m_total, ctx->d, ctx->k, ctx->n_layers, ctx->sms, &wl)) return IDKM_ERR_UNSUPPORTED;
  if (cudaStreamSynchronize(ctx->stream) != cudaSuccess) return IDKM_ERR_CUDA;
  LayerState st;
  const char* ws = static_cast<const char*>(ctx->workspace);
  if (cudaMemcpy(&st, ws + wl.off_state + sizeof(LayerState) * (size_t)layer, sizeof(st), cudaMemcpyDeviceToHost) != cudaSuccess)
    return IDKM_ERR_CUDA;
  int n = which == 0 ? st.fwd_iters : st.adj_iters;
  if (n > HIST_CAP) n = HIST_CAP;
  if (n > capacity) n = capacity;
  if (n < 0) n = 0;
  const size_t off = (which == 0 ? wl.off_hist_fwd : wl.off_hist_adj) + sizeof(float) * (size_t)layer * HIST_CAP;
  if (n > 0 && cudaMemcpy(host_out, ws + off, sizeof(float) * (size_t)n, cudaMemcpyDeviceToHost) != cudaSuccess)
    return IDKM_ERR_CUDA;
  *n_out = n;
  return IDKM_OK;
}

int idkm_set_distance(idkm_ctx* ctx, int squared) {
  if (!ctx) return IDKM_ERR_NULL;
  if (squared != 0 && squared != 1) return IDKM_ERR_PARAM;
  if (ctx->squared != squared) ctx->have_forward = false;   // a backward must follow a forward of the same variant
  ctx->squared = squared;
  return IDKM_OK;
}

int idkm_set_wq_dtype(idkm_ctx* ctx, int dtype) {
  if (!ctx) return IDKM_ERR_NULL;
  if (dtype < 0 || dtype > 2) return IDKM_ERR_PARAM;
  ctx->wq_dtype = dtype;
  return IDKM_OK;
}

int idkm_set_collapse_step(idkm_ctx* ctx, int method) {
  if (!ctx) return IDKM_ERR_NULL;
  if (method != 0 && method != 1) return IDKM_ERR_PARAM;
  ctx->collapse_step = method;
  return IDKM_OK;
}

int idkm_set_forward_loop(idkm_ctx* ctx, int method) {
  if (!ctx) return IDKM_ERR_NULL;
  if (method < 0 || method > 3) return IDKM_ERR_PARAM;
  ctx->forward_loop = method;
  return IDKM_OK;
}

int idkm_set_test_hooks(idkm_ctx* ctx, int missing_arrivals, int64_t spin_limit_ticks) {
  if (!ctx) return IDKM_ERR_NULL;
  if (missing_arrivals < 0 || spin_limit_ticks < 0) return IDKM_ERR_PARAM;
  ctx->hook_missing_arrivals = missing_arrivals;
  ctx->hook_spin_limit = spin_limit_ticks;
  return IDKM_OK;
}

int idkm_count_busy_tickets(idkm_ctx* ctx, int* count_out) {
  if (!ctx || !count_out) return IDKM_ERR_NULL;
  if (!ctx->have_forward) return IDKM_ERR_ORDER;
  WorkspaceLayout wl;
  if (!make_layout(ctx->m_total, ctx->d, ctx->k, ctx->n_layers, ctx->sms, &wl)) return IDKM_ERR_UNSUPPORTED;
  if (cudaStreamSynchronize(ctx->stream) != cudaSuccess) return IDKM_ERR_CUDA;
  const char* ws = static_cast<const char*>(ctx->workspace);
  int busy = 0;
  LayerState host[MAX_LAYERS];
  if (cudaMemcpy(host, ws + wl.off_state, sizeof(LayerState) * (size_t)ctx->n_layers, cudaMemcpyDeviceToHost) != cudaSuccess)
    return IDKM_ERR_CUDA;
  for (int l = 0; l < ctx->n_layers; ++l) busy += (host[l].ticket != 0u);
  const size_t offs[2] = {wl.off_gtickets, wl.off_gtickets64};
  const int counts[2] = {wl.max_groups, wl.max_groups64};
  for (int s = 0; s < 2; ++s) {
    if (counts[s] <= 0) continue;
    unsigned int* t = new (std::nothrow) unsigned int[counts[s]];
    if (!t) return IDKM_ERR_CUDA;
    const cudaError_t rc = cudaMemcpy(t, ws + offs[s], sizeof(unsigned int) * (size_t)counts[s], cudaMemcpyDeviceToHost);
    if (rc == cudaSuccess)
      for (int i = 0; i < counts[s]; ++i) busy += (t[i] != 0u);
    delete[] t;
    if (rc != cudaSuccess) return IDKM_ERR_CUDA;
  }
  *count_out = busy;
  return IDKM_OK;
}

int64_t idkm_launch_count(const idkm_ctx* ctx) { return ctx ? ctx->launches : 0; }

int idkm_describe_path(int d, int k, int adj_max_iter, int adjoint_method, int* out) {
  if (!out) return IDKM_ERR_NULL;
  if (d_index(d) < 0 || k < 1 || k > IDKM_MAX_K) return IDKM_ERR_UNSUPPORTED;
  const int fs = pick_family(STEP, d, k), fa = pick_family(ADJ, d, k), fj = pick_family(JACOBIAN, d, k);
  if (fs < 0 || fa < 0) return IDKM_ERR_UNSUPPORTED;
  out[0] = kernel_entry(STEP, d, fs)->kpl;
  out[1] = kernel_entry(STEP, d, fs)->lpw;
  out[2] = kernel_entry(ADJ, d, fa)->kpl;
  out[3] = kernel_entry(ADJ, d, fa)->lpw;
  const bool jac_tile = fj >= 0 && kernel_entry(JACOBIAN, d, fj)->plen > JAC_SMALL_PLEN_MAX;
  const bool explicit_jac = adjoint_method == 0 && fj >= 0 && (!jac_tile || adj_max_iter >= JAC_TILE_MIN_ITERS);
  out[4] = (adj_max_iter <= 0) ? 0 : ((adjoint_method == 2 && fj >= 0) ? 3 : (explicit_jac ? (jac_tile ? 2 : 1) : 0));
  return IDKM_OK;
}

const char* idkm_status_string(int status) {
  switch (status) {
    case IDKM_OK: return "ok";
    case IDKM_MAXITER: return "iteration cap reached before the tolerance";
    case IDKM_ERR_NULL: return "required pointer is NULL";
    case IDKM_ERR_ALIGN: return "pointer is not 16-byte aligned";
    case IDKM_ERR_SHAPE: return "bad shape or layer offsets";
    case IDKM_ERR_UNSUPPORTED: return "unsupported d or k";
    case IDKM_ERR_PARAM: return "parameter out of range";
    case IDKM_ERR_WORKSPACE: return "workspace too small";
    case IDKM_ERR_ORDER: return "backward without a matching forward";
    case IDKM_ERR_CUDA: return "CUDA runtime error";
    case IDKM_ERR_NONFINITE: return "non-finite value met on the device";
    case IDKM_ERR_DIVERGED: return "adjoint iteration diverged";
    case IDKM_ERR_NOALLOC_TOO_LARGE: return "problem needs more than the library's built-in scratch";
    case IDKM_ERR_TIMEOUT: return "a grid-wide wait of the single-launch forward loop ran out";
  }
  return "unknown status";
}

}  // extern "C"
