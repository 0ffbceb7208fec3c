// Fused passes of the IDKM hot path (sm_100a).
//
// One kernel template serves the five passes over W.  A "group" of LPW lanes handles one
// weight-vector at a time; each lane of the group owns KPL centroids in registers, so the
// k x (d+1) sums of the M-step live in registers and the m x k attention matrix is never
// stored (Algorithm 1, steps 3-5, fused).  LPW == 1 is the thread-per-weight layout for
// small codebooks, with 128-bit loads of 4/d weight-vectors per thread.
//
// Blocks are persistent and own a fixed, contiguous range of tiles; tiles never span layers.
// Sums are reduced lane -> warp -> block in a fixed order, written as one fp64 partial per
// (block, layer), and the last block to finish a layer adds the partials in slot order in
// fp64 and applies the pass's epilogue (M-step and stop test; adjoint update; ...).  Results
// are therefore bit-reproducible from run to run.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <type_traits>

namespace idkm {

constexpr int BLOCK = 256;
constexpr int NWARP = BLOCK / 32;
constexpr int MAX_LAYERS = 64;
constexpr float PAD_COORD = 1e18f;   // coordinate of a padding centroid: exp underflows to exactly 0
constexpr double S_MIN = 1e-20;      // column sums below this mark a dead cluster
constexpr float S_MIN_F = 1e-20f;
constexpr int MAX_BLOCKS_PER_SM = 8;
constexpr int HIST_CAP = 1024;       // iterations of residual history kept per layer and loop
// Blocks whose partials one block adds up in the first stage of the cross-block reduction (see finish_layer).
constexpr int RED_GROUP = 16;
// Up to this many partials one block adds them all: the extra stage costs a few microseconds of latency, which only
// pays off once the single stage would read hundreds of rows.
constexpr int RED_SINGLE_MAX = 64;
// When the bounding box of a layer's centroids is smaller than PRECISE_SPAN * tau, all softmax logits of a
// weight differ by less than PRECISE_SPAN and the centroid update is decided by attention differences far below
// fp32 resolution (w - c_j rounds away the differences between the c_j).  Such layers step in fp64.
constexpr double PRECISE_SPAN = 0.0625;
// A converging adjoint iteration u <- alpha (J^T u + g) + (1 - alpha) u stays below ||g|| / (1 - rho); once ||u|| has
// grown past this multiple of ||g|| the iteration is reported as diverged (Section 4.2: "if we see the iteration
// diverge, we start over and divide alpha by 2").  A residual that grows 10 steps running, or a non-finite u, counts
// as well; a spiralling (complex-eigenvalue) divergence shows only in the norm.
constexpr double ADJ_GROWTH_LIMIT = 1e6;

enum Mode { STEP = 0, FINAL = 1, GRAD = 2, ADJ = 3, SCATTER = 4, STEP_PRECISE = 5, JACOBIAN = 6, STEP_DELTA = 7 };
constexpr int N_MODES = 8;

// status values mirrored from idkm.h (device side needs only these)
constexpr int ST_OK = 0, ST_MAXITER = 1, ST_NONFINITE = -9, ST_DIVERGED = -10, ST_TIMEOUT = -12;

struct LayerState {   // 64 bytes, one per layer, in the workspace
  int fwd_done, fwd_iters;   // fwd_done: 0 while the loop runs, else the number of iterations after which it ended
  float fwd_res;
  int dead;
  int adj_done, adj_iters;
  float adj_res;
  int status;
  unsigned int ticket;
  int adj_up;        // consecutive adjoint steps whose residual grew
  float adj_prev;
  int precise[2];    // [t & 1] routes forward iteration t.  1: the layer's centroids lie within PRECISE_SPAN * tau of
                     // each other (collapsing) and the step runs in the fp64 kernel.  The epilogue of iteration t
                     // writes entry (t + 1) & 1 only, so nothing a launch routes by changes while it runs: the fp32
                     // and the fp64 half of the dual step kernel, whose blocks are not ordered against each other,
                     // can never both take (or both skip) a layer.
  float g_norm;      // ||g||_2 of the last codebook-gradient pass: the adjoint iteration counts as diverged once
                     // ||u||_2 exceeds ADJ_GROWTH_LIMIT times it
  int pad[2];
};
static_assert(sizeof(LayerState) == 64, "LayerState layout");

struct LayerTable {
  int n_layers;
  int tiles_total;
  int n_blocks;                       // grid size the table was built for
  int pad;
  long long row_off[MAX_LAYERS + 1];  // first row of each layer
  int tile_off[MAX_LAYERS + 1];       // first tile of each layer
};

struct PassParams {
  const float* W;
  const float* G;     // upstream gradient dL/dWq (GRAD, SCATTER)
  void* Wq;           // FINAL (may be null); element type wq_dtype
  float* A;           // FINAL (may be null)
  float* dW;          // SCATTER
  float* C;           // [L][k][d] centroids, updated in place by STEP
  float* S;           // [L][k]   column sums at the returned centroids (FINAL writes)
  float* F;           // [L][k][d] F(C_T, W) (FINAL writes)
  float* gvec;        // [L][k][d] direct codebook gradient (GRAD writes)
  float* u;           // [L][k][d] adjoint (GRAD initialises, ADJ updates)
  float* hist_fwd;    // [L][HIST_CAP]: relative change of C after each forward iteration (first HIST_CAP of them)
  float* hist_adj;    // [L][HIST_CAP]: relative change of u after each adjoint iteration
  double* partials;   // [(n_blocks + L)][PLEN]
  double* gpartials;  // [(n_blocks + L) / RED_GROUP + L + 2][PLEN]: sums over groups of RED_GROUP partials
  unsigned int* gtickets;   // one arrival counter per group, zero at rest
  float2* rowstat;    // [rows] or null: per row the softmax reference (scale * min_j D_ij) and 1 / sum_j exp, as the
                      // codebook-gradient pass computed them; read by the adjoint layouts of row_cache_layout()
  LayerState* st;
  float inv_tau;      // 1 / tau
  float scale;        // log2(e) / tau
  float tol;          // stop tolerance of the loop this pass belongs to
  float alpha;        // averaging weight of the adjoint iteration
  double inv_tau_d;   // 1 / tau in double (fp64 step)
  int k;
  int max_iter;       // iteration cap of the loop (for the advisory status)
  int* host_flag;     // device view of a pinned host word, or null: set to call_id once every layer's loop has ended
  int call_id;
  int wq_dtype;       // element type of Wq (FINAL): 0 fp32, 1 bf16, 2 fp16 (round to nearest even of the fp32 result)
  int squared;        // 1: squared-distance variant; its layers always step in the fp32 kernel (the fp64 step's
                      // short exponential series is derived for the Euclidean distance)
  int iter;           // index of this forward iteration: a layer is stepped only while fwd_iters == iter, so that
                      // the fp32 and the fp64 step launched for the same iteration never both take it
  LayerTable lt;
};

// ---- configuration shared by host and device -------------------------------------------------
template <int MODE, int D, int KPL, int LPW>
struct PassCfg {
  static constexpr int KP = KPL * LPW;
  static constexpr int NACC = (MODE == STEP || MODE == FINAL) ? D + 1 : (MODE == SCATTER ? 0 : D);
  static constexpr int PLEN = KP * (NACC > 0 ? NACC : 1);
  static constexpr int GROUPS = BLOCK / LPW;
  static constexpr int VEC = (LPW == 1) ? 4 / D : 1;              // weight-vectors per 128-bit load
  // 128-bit loads in flight per thread (thread-per-weight layouts): small codebooks are bound by memory latency
  static constexpr int UNROLL = (LPW == 1) ? ((KPL * D >= 32) ? 1 : ((KPL * D >= 16) ? 2 : 4)) : 1;
  // weight-vectors per group per tile (bounded so that the staging buffers stay a few KB)
  // (thread-per-weight: one 128-bit load per thread per tile; a block takes up to UNROLL consecutive tiles at once,
  // so small layers still spread over many blocks)
  static constexpr int WPG = (LPW == 1) ? VEC : (LPW >= 16 ? 16 : (LPW == 8 ? 8 : 4));
  static constexpr int TILE = GROUPS * WPG;
  // Each thread's sums are moved out of its registers into a private fp32 slot in (dynamic) shared memory every
  // SPILL_TILES tiles, i.e. after about 64 weight-vectors.  A long-running fp32 accumulator silently drops the
  // many terms that are smaller than half its ulp (the attention of far-away weights), a one-sided loss that was
  // measured to grow in proportion to the number of terms; 64-term chunks keep it below 3e-8 relative.
  static constexpr int SPILL_TILES = (64 / WPG) > 0 ? (64 / WPG) : 1;
  static constexpr int DYN_SMEM = (NACC > 0) ? BLOCK * KPL * NACC * 4 : 0;
  // resident blocks per SM the register budget is sized for (the 32-lane layouts hold 8 centroids per lane)
  // (thread-per-weight: estimated from the registers that hold centroids, per-centroid constants and sums)
  static constexpr int REGS_EST = KPL * ((MODE == STEP || MODE == FINAL) ? 2 * D + 1 : 3 * D + 1) + 40;
  // (the two 16-centroid group layouts: three resp. two blocks, their centroids and sums need 36 resp. 72 registers)
  static constexpr int MIN_BLOCKS =
      (LPW == 32) ? 2
      : (KPL == 4 && LPW == 4) ? 3
      : (KPL == 8 && LPW == 2 && (MODE == STEP || MODE == FINAL)) ? 2
      : ((LPW > 1) ? 1 : ((256 / REGS_EST) > 4 ? 4 : ((256 / REGS_EST) < 1 ? 1 : (256 / REGS_EST))));
};

// Layouts whose adjoint step reads each row's softmax reference and normaliser from the workspace instead of
// recomputing them: the group-per-weight layouts, except the full-warp layout at d = 4, whose register budget is
// full (there the two extra values per row in flight made the step spill and run 8 % slower).
__host__ __device__ constexpr bool row_cache_layout(int d, int lpw) { return lpw > 1; }

// ---- special-function-unit wrappers ------------------------------------------------------------
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float sqrt_approx(float x) {
  float y;
  asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float rsqrt_approx(float x) {
  float y;
  asm("rsqrt.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float rcp_approx(float x) {
  float y;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Pairwise (tree) sum (OP 0) or minimum (OP 1) of a register array: log2(N) dependent steps instead of N.
template <int N, int OP>
__device__ __forceinline__ float tree_reduce(const float (&x)[N]) {
  float t[N];
#pragma unroll
  for (int i = 0; i < N; ++i) t[i] = x[i];
#pragma unroll
  for (int s = 1; s < N; s <<= 1)
#pragma unroll
    for (int i = 0; i + s < N; i += 2 * s) t[i] = (OP == 0) ? t[i] + t[i + s] : fminf(t[i], t[i + s]);
  return t[0];
}

// Programmatic dependent launch: wait until the kernels this one depends on have completed (and their writes are
// visible), then let the next kernel in the stream be scheduled early.  Must run before the first global read.
__device__ __forceinline__ void grid_dependency_sync() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
}
// Called by every block once its share of the rows is done, before the reduction epilogue: the next kernel's blocks
// may then take the SMs that fall idle during the epilogue (they still wait for this grid to complete).  Releasing
// them at the start of the kernel instead measured slower on the batched workload.
__device__ __forceinline__ void grid_release_dependents() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

template <int LPW>
__device__ __forceinline__ float group_sum(float v) {
#pragma unroll
  for (int o = LPW / 2; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
// Minimum over the lanes of a group of a NON-NEGATIVE float.  Non-negative IEEE floats order like their bit
// patterns read as unsigned integers, so a full warp does it with one integer warp-reduce instruction; with
// sub-warp masks that instruction measured slower than the shuffles, so smaller groups shuffle.
template <int LPW>
__device__ __forceinline__ float group_min(float v) {
  if constexpr (LPW == 32) {
    return __uint_as_float(__reduce_min_sync(0xffffffffu, __float_as_uint(v)));
  } else {
#pragma unroll
    for (int o = LPW / 2; o > 0; o >>= 1) v = fminf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
  }
}

// block that owns tile t when n_tiles are dealt contiguously to n_blocks blocks:
// block b owns [b*T/NB, (b+1)*T/NB)
__host__ __device__ inline int tile_begin(int b, int n_tiles, int n_blocks) {
  return (int)(((long long)b * n_tiles) / n_blocks);
}
__host__ __device__ inline int block_of_tile(int t, int n_tiles, int n_blocks) {
  return (int)((((long long)t + 1) * n_blocks - 1) / n_tiles);
}

// Fixed-order block reduction of one double per thread (OP: 0 sum, 1 min, 2 max); result valid in every thread.
template <int OP>
__device__ __forceinline__ double block_reduce_double(double v, double* scratch /* BLOCK doubles */) {
  const int tid = threadIdx.x;
  __syncthreads();
  scratch[tid] = v;
  __syncthreads();
#pragma unroll
  for (int s = BLOCK / 2; s > 0; s >>= 1) {
    if (tid < s) {
      const double a = scratch[tid], b = scratch[tid + s];
      scratch[tid] = (OP == 0) ? a + b : ((OP == 1) ? fmin(a, b) : fmax(a, b));
    }
    __syncthreads();
  }
  double r = scratch[0];
  __syncthreads();
  return r;
}
__device__ __forceinline__ double block_sum_double(double v, double* scratch) { return block_reduce_double<0>(v, scratch); }

// After a block has written its partial of layer l, the partials are added up in two stages so that no block
// ever reads more than RED_GROUP + (blocks / RED_GROUP) of them: the contributing blocks form groups of RED_GROUP
// consecutive blocks; the last block to arrive in a group adds the group's partials in slot order (fp64) into a
// group partial; the last group to finish adds the group partials in group order and applies the epilogue of the
// pass.  Grouping and order depend on block indices only, so the result is reproducible.  Layers with at most
// RED_SINGLE_MAX contributing blocks skip the first stage.  Called by all threads of the block.
// smem_raw must hold (PLEN + BLOCK) doubles.
// DELTA (forward step of a collapsing layer in the increment form, see delta_body): the totals are
// dS_j = sum_i (A_ij - 1/k), dN_j = sum_i (A_ij - 1/k) (w_i - c_0) and, in the last D entries, sum_i w_i; with
// U = sum_i w_i - m c_0 the M-step is C+_j = c_0 + (U / k + dN_j) / (m / k + dS_j).
template <int MODE, int D, int PLEN, int NA, bool DELTA = false>
__device__ __forceinline__ void finish_layer(const PassParams& p, int l, int b, unsigned char* smem_raw, int* s_flag) {
  const int tid = threadIdx.x;
  const int k = p.k;
  const int nb = p.lt.n_blocks;
  __threadfence();
  __syncthreads();
  const int first_b = block_of_tile(p.lt.tile_off[l], p.lt.tiles_total, nb);
  const int last_b = block_of_tile(p.lt.tile_off[l + 1] - 1, p.lt.tiles_total, nb);
  const int n_contrib = last_b - first_b + 1;
  const double* base = p.partials + (size_t)(first_b + l) * PLEN;   // rows the last stage adds
  int n_terms = n_contrib;
  if (n_contrib > RED_SINGLE_MAX) {
    // ---- first stage: one group of RED_GROUP consecutive slots ----
    const int g = (b - first_b) / RED_GROUP;
    const int gsize = (n_contrib - g * RED_GROUP < RED_GROUP) ? n_contrib - g * RED_GROUP : RED_GROUP;
    // group rows of layer l start at (first slot / RED_GROUP) + l: distinct layers get distinct rows because a
    // layer with n slots has at most n / RED_GROUP + 1 groups
    const int grow0 = (first_b + l) / RED_GROUP + l;
    if (tid == 0) {
      const unsigned int prev = atomicAdd(&p.gtickets[grow0 + g], 1u);
      *s_flag = (prev == (unsigned int)(gsize - 1));
    }
    __syncthreads();
    if (!*s_flag) return;
    __threadfence();
    const double* gb = base + (size_t)g * RED_GROUP * PLEN;
    double* gout = p.gpartials + (size_t)(grow0 + g) * PLEN;
    for (int o = tid; o < PLEN; o += BLOCK) {
      double v[RED_GROUP];
#pragma unroll
      for (int q = 0; q < RED_GROUP; ++q) v[q] = (q < gsize) ? __ldcg(gb + (size_t)q * PLEN + o) : 0.0;
      double s = 0.0;
#pragma unroll
      for (int q = 0; q < RED_GROUP; ++q) s += v[q];
      gout[o] = s;
    }
    if (tid == 0) p.gtickets[grow0 + g] = 0u;
    __threadfence();
    __syncthreads();
    base = p.gpartials + (size_t)grow0 * PLEN;
    n_terms = (n_contrib + RED_GROUP - 1) / RED_GROUP;
  }
  // ---- last stage: the last arrival (block, or group) adds the remaining rows ----
  if (tid == 0) {
    const unsigned int prev = atomicAdd(&p.st[l].ticket, 1u);
    *s_flag = (prev == (unsigned int)(n_terms - 1));
  }
  __syncthreads();
  if (!*s_flag) return;
  __threadfence();
  double* tot = reinterpret_cast<double*>(smem_raw);   // [PLEN]
  double* scratch = tot + PLEN;                          // [BLOCK]
  if constexpr (PLEN >= BLOCK) {
    for (int o = tid; o < PLEN; o += BLOCK) {
      double s = 0.0;
#pragma unroll 8
      for (int q = 0; q < n_terms; ++q) s += __ldcg(base + (size_t)q * PLEN + o);
      tot[o] = s;
    }
    __syncthreads();
  } else {
    constexpr int NCH = BLOCK / PLEN;   // PLEN is a power of two times (d+1); BLOCK % PLEN may be nonzero
    const int ch = tid / PLEN, o = tid % PLEN;
    double s = 0.0;
    if (ch < NCH)
      for (int q = ch; q < n_terms; q += NCH) s += __ldcg(base + (size_t)q * PLEN + o);
    scratch[tid] = s;
    __syncthreads();
    if (tid < PLEN) {
      double r2 = 0.0;
#pragma unroll 1
      for (int c2 = 0; c2 < NCH; ++c2) r2 += scratch[c2 * PLEN + tid];
      tot[tid] = r2;
    }
    __syncthreads();
  }
  // ---- epilogue on the layer totals ----
  LayerState* st = p.st + l;
  double num = 0.0, den = 0.0, bad = 0.0, dead = 0.0;
  double cmin[D], cmax[D];
#pragma unroll
  for (int a = 0; a < D; ++a) {
    cmin[a] = 1e300;
    cmax[a] = -1e300;
  }
  if constexpr (MODE == STEP) {
    float* Cl = p.C + (size_t)l * k * D;
    double c0[D], ubar[D], mk = 0.0;
    (void)c0; (void)ubar; (void)mk;
    if constexpr (DELTA) {
      constexpr int NEXTRA = (D == 1) ? 4 : 0;
      const double mrows = (double)(p.lt.row_off[l + 1] - p.lt.row_off[l]);
      mk = mrows / (double)k;
      double wsum[D];
#pragma unroll
      for (int a = 0; a < D; ++a) {
        c0[a] = (double)Cl[a];                       // centroid 0 before anybody overwrites it
        wsum[a] = tot[PLEN - NEXTRA - D + a];
      }
      if constexpr (D == 1) {
        // Scalar weights outside the centroids see the logits +-delta_j / tau, whatever their own value: their
        // attention increments take two values per centroid, a+_j for w > c and a-_j for w < c, and the row loop only
        // counted them (cp, cm) and added their weights up (sp, sm).  Their share of dS_j and dN_j is added here.
        const double cp = tot[PLEN - 4], sp = tot[PLEN - 3], cm = tot[PLEN - 2], sm = tot[PLEN - 1];
        wsum[0] += sp + sm;
        // (k <= BLOCK: one centroid per thread; fixed-order block sums for the two means)
        double tpj = 0.0, tmj = 0.0;
        if (tid < k) {
          const double dj = ((double)Cl[tid] - c0[0]) * p.inv_tau_d;
          tpj = expm1(dj);
          tmj = expm1(-dj);
        }
        const double tbp = block_sum_double(tpj, scratch) / (double)k;
        const double tbm = block_sum_double(tmj, scratch) / (double)k;
        if (tid < k) {
          const double ap = (tpj - tbp) / ((double)k * (1.0 + tbp));
          const double am = (tmj - tbm) / ((double)k * (1.0 + tbm));
          tot[tid * NA] += ap * cp + am * cm;
          tot[tid * NA + 1] += ap * (sp - cp * c0[0]) + am * (sm - cm * c0[0]);
        }
      }
#pragma unroll
      for (int a = 0; a < D; ++a) ubar[a] = (wsum[a] - mrows * c0[a]) / (double)k;
      __syncthreads();
    }
    for (int j = tid; j < k; j += BLOCK) {
      const double s = DELTA ? mk + tot[j * NA] : tot[j * NA];
      const bool alive = (s >= S_MIN);
      if (!alive) dead += 1.0;
      if (!(s == s) || s > 1e300) bad += 1.0;
#pragma unroll
      for (int a = 0; a < D; ++a) {
        const double cold = (double)Cl[j * D + a];
        const double cnew = alive ? (DELTA ? c0[a] + (ubar[a] + tot[j * NA + 1 + a]) / s : tot[j * NA + 1 + a] / s) : cold;
        if (!(cnew == cnew) || fabs(cnew) > 1e300) bad += 1.0;
        num += (cnew - cold) * (cnew - cold);
        den += cnew * cnew;
        Cl[j * D + a] = (float)cnew;
        cmin[a] = fmin(cmin[a], (double)(float)cnew);
        cmax[a] = fmax(cmax[a], (double)(float)cnew);
      }
    }
  } else if constexpr (MODE == FINAL) {
    for (int j = tid; j < k; j += BLOCK) {
      const double s = tot[j * NA];
      const bool alive = (s >= S_MIN);
      if (!(s == s) || s > 1e300) bad += 1.0;
      p.S[(size_t)l * k + j] = alive ? (float)s : 0.f;
#pragma unroll
      for (int a = 0; a < D; ++a) {
        const double f = alive ? tot[j * NA + 1 + a] / s : (double)p.C[((size_t)l * k + j) * D + a];
        if (!(f == f)) bad += 1.0;
        p.F[((size_t)l * k + j) * D + a] = (float)f;
      }
    }
  } else if constexpr (MODE == GRAD) {
    for (int o = tid; o < k * D; o += BLOCK) {
      const double gv = tot[o];
      if (!(gv == gv) || fabs(gv) > 1e300) bad += 1.0;
      den += gv * gv;
      p.gvec[(size_t)l * k * D + o] = (float)gv;
      p.u[(size_t)l * k * D + o] = (float)gv;
    }
  } else if constexpr (MODE == ADJ) {
    for (int o = tid; o < k * D; o += BLOCK) {
      const double uold = (double)p.u[(size_t)l * k * D + o];
      const double gv = (double)p.gvec[(size_t)l * k * D + o];
      const double al = (double)p.alpha;
      const double unew = al * (tot[o] + gv) + (1.0 - al) * uold;
      if (!(unew == unew) || fabs(unew) > 1e300) bad += 1.0;
      num += (unew - uold) * (unew - uold);
      den += unew * unew;
      p.u[(size_t)l * k * D + o] = (float)unew;
    }
  }
  // All block-wide reductions of the epilogue in one go (two barriers): warp trees by shuffle, then the NWARP warp
  // results combined in warp order by every thread.  Slots: bad, num, den, dead (sums), cmin[D] (min), cmax[D] (max).
  double box2 = 0.0;
  {
    constexpr int NV = 4 + 2 * D;
    double v[NV];
    v[0] = bad; v[1] = num; v[2] = den; v[3] = dead;
#pragma unroll
    for (int a = 0; a < D; ++a) {
      v[4 + a] = cmin[a];
      v[4 + D + a] = cmax[a];
    }
#pragma unroll
    for (int i = 0; i < NV; ++i) {
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const double other = __shfl_xor_sync(0xffffffffu, v[i], o);
        v[i] = (i < 4) ? v[i] + other : ((i < 4 + D) ? fmin(v[i], other) : fmax(v[i], other));
      }
    }
    __syncthreads();
    if ((tid & 31) == 0) {
#pragma unroll
      for (int i = 0; i < NV; ++i) scratch[(tid >> 5) * NV + i] = v[i];
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < NV; ++i) {
      double r = scratch[i];
      for (int wv = 1; wv < NWARP; ++wv) {
        const double other = scratch[wv * NV + i];
        r = (i < 4) ? r + other : ((i < 4 + D) ? fmin(r, other) : fmax(r, other));
      }
      v[i] = r;
    }
    bad = v[0]; num = v[1]; den = v[2]; dead = v[3];
    if constexpr (MODE == STEP) {
#pragma unroll
      for (int a = 0; a < D; ++a) box2 += (v[4 + D + a] - v[4 + a]) * (v[4 + D + a] - v[4 + a]);
    }
  }
  if (tid == 0) {
    st->ticket = 0u;
    if constexpr (MODE == STEP) {
      st->precise[(p.iter + 1) & 1] = (!p.squared && sqrt(box2) * p.inv_tau_d <= PRECISE_SPAN) ? 1 : 0;
      double dn = sqrt(den);
      if (dn < 1e-300) dn = 1e-300;
      const float res = (float)(sqrt(num) / dn);
      const int it = st->fwd_iters + 1;
      st->fwd_iters = it;
      st->fwd_res = res;
      if (it <= HIST_CAP) p.hist_fwd[(size_t)l * HIST_CAP + it - 1] = res;
      st->dead = (int)dead;
      if (bad > 0.0) {
        st->status = ST_NONFINITE;
        st->fwd_done = it;
      } else if (p.tol > 0.f && res < p.tol) {
        st->fwd_done = it;
        st->status = ST_OK;
      } else if (p.tol > 0.f && it >= p.max_iter) {
        st->status = ST_MAXITER;
      }
    } else if constexpr (MODE == FINAL) {
      if (bad > 0.0) st->status = ST_NONFINITE;
    } else if constexpr (MODE == GRAD) {
      st->adj_done = (bad > 0.0) ? 1 : 0;
      st->adj_iters = 0;
      st->adj_res = 0.f;
      st->adj_up = 0;
      st->adj_prev = 3.0e38f;
      st->g_norm = (float)sqrt(den);
      if (bad > 0.0) st->status = ST_NONFINITE;
      else if (st->status == ST_DIVERGED) st->status = ST_OK;
    } else if constexpr (MODE == ADJ) {
      double dn = sqrt(den);
      if (dn < 1e-300) dn = 1e-300;
      const float res = (float)(sqrt(num) / dn);
      const int it = st->adj_iters + 1;
      st->adj_iters = it;
      st->adj_res = res;
      if (it <= HIST_CAP) p.hist_adj[(size_t)l * HIST_CAP + it - 1] = res;
      const int up = (res > st->adj_prev) ? st->adj_up + 1 : 0;
      st->adj_up = up;
      st->adj_prev = res;
      if (bad > 0.0 || up >= 10 || sqrt(den) > ADJ_GROWTH_LIMIT * (double)st->g_norm) {
        st->status = ST_DIVERGED;
        st->adj_done = 1;
      } else if (p.tol > 0.f && res < p.tol) {
        st->adj_done = 1;
      } else if (p.tol > 0.f && it >= p.max_iter && st->status == ST_OK) {
        st->status = ST_MAXITER;
      }
    }
    // Tell the host (it only peeks, it never waits on this) when the loops of ALL layers have ended, so that it can
    // stop queueing iterations that would return at once.  Whichever epilogue sees every flag set writes the word.
    if constexpr (MODE == STEP || MODE == ADJ) {
      if (p.host_flag != nullptr && ((MODE == STEP) ? st->fwd_done : st->adj_done)) {
        __threadfence();
        bool all = true;
        for (int q = 0; q < p.lt.n_layers; ++q) {
          const volatile LayerState* sq = p.st + q;
          all = all && (((MODE == STEP) ? sq->fwd_done : sq->adj_done) != 0);
        }
        if (all) {
          *reinterpret_cast<volatile int*>(p.host_flag) = p.call_id;
          __threadfence_system();
        }
      }
    }
  }
  __syncthreads();
}

// Stores N consecutive elements of the soft-quantised weights, starting at element index `elem` of Wq, in the element
// type the caller asked for (bf16 / fp16: the fp32 result rounded to nearest even).  `vec`: the N elements may go out
// as one store (their byte offset is a multiple of the store width).
// (The two-byte types go through a function of their own that is not inlined: with their conversions inlined into the
// row loop the fp32 final pass of the largest codebook ran 12 % slower.)
template <int N>
__device__ __noinline__ void store_wq_half(void* base, long long elem, float v0, float v1, float v2, float v3, int dtype, bool vec) {
  const float v[4] = {v0, v1, v2, v3};
  unsigned short h[4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
    h[i] = (dtype == 1) ? __bfloat16_as_ushort(__float2bfloat16_rn(v[i])) : __half_as_ushort(__float2half_rn(v[i]));
  unsigned short* dst = static_cast<unsigned short*>(base) + elem;
  if (vec && N == 4) {
    *reinterpret_cast<uint2*>(dst) = make_uint2((unsigned)h[0] | ((unsigned)h[1] << 16), (unsigned)h[2] | ((unsigned)h[3] << 16));
  } else if (vec && N == 2) {
    *reinterpret_cast<unsigned*>(dst) = (unsigned)h[0] | ((unsigned)h[1] << 16);
  } else {
#pragma unroll
    for (int i = 0; i < N; ++i) dst[i] = h[i];
  }
}
template <int N>
__device__ __forceinline__ void store_wq(void* base, long long elem, const float (&v)[N], int dtype, bool vec) {
  if (dtype == 0) {
    float* dst = static_cast<float*>(base) + elem;
    if (vec && N == 4) *reinterpret_cast<float4*>(dst) = make_float4(v[0], v[N > 1 ? 1 : 0], v[N > 2 ? 2 : 0], v[N > 3 ? 3 : 0]);
    else if (vec && N == 2) *reinterpret_cast<float2*>(dst) = make_float2(v[0], v[N > 1 ? 1 : 0]);
    else {
#pragma unroll
      for (int i = 0; i < N; ++i) dst[i] = v[i];
    }
    return;
  }
  store_wq_half<N>(base, elem, v[0], v[N > 1 ? 1 : 0], v[N > 2 ? 2 : 0], v[N > 3 ? 3 : 0], dtype, vec);
}

// ---- bulk asynchronous copies into shared memory, completion on an mbarrier --------------------------------------
constexpr int BULK_STAGES = 3;
constexpr int BULK_WAIT_POLLS = 1 << 22;   // polls of one wait before the block gives up (each poll may itself block
                                           // for a hardware-defined slice): seconds, against microseconds of copy
__device__ __forceinline__ unsigned smem_addr(const void* ptr) { return (unsigned)__cvta_generic_to_shared(ptr); }
__device__ __forceinline__ void mbar_init(unsigned long long* bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_init_fence() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void mbar_arrive_expect_tx(unsigned long long* bar, unsigned bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned long long* bar, unsigned parity) {
  unsigned ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_addr(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// dst: shared memory, 16-byte aligned; src: global memory, 16-byte aligned; bytes: a multiple of 16
__device__ __forceinline__ void bulk_copy_g2s(void* dst, const void* src, unsigned bytes, unsigned long long* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(smem_addr(dst)),
               "l"(src), "r"(bytes), "r"(smem_addr(bar))
               : "memory");
}

// ---- the pass ------------------------------------------------------------------------------------
// RELEASE: let the next kernel of the stream be scheduled once this block's rows are done (the caller has already
// waited for the previous kernel).  The dual step kernel runs this body with RELEASE = false and releases after its
// second body.
// SQ: the squared-distance variant, D_ij = ||w_i - c_j||^2 in the softmax (the distance the clustering objectives of
// Sections 3.1 / 3.2 are written in) and n_ij = dD_ij/dw_i = 2 (w_i - c_j): no square root, no reciprocal square
// root, no kink at w_i = c_j.
// BULK (forward step, thread-per-weight layouts): the rows of a trip arrive in shared memory by one bulk
// asynchronous copy per trip (cp.async.bulk, completion on an mbarrier), issued by one thread BULK_STAGES trips ahead
// of the arithmetic, instead of by per-thread 128-bit loads issued at the top of the trip.
template <int MODE, int D, int KPL, int LPW, bool RELEASE, bool SQ = false, bool BULK = false>
__device__ __forceinline__ void pass_body(const PassParams& p) {
  using Cfg = PassCfg<MODE, D, KPL, LPW>;
  constexpr int NACC = Cfg::NACC;
  constexpr int PLEN = Cfg::PLEN;
  constexpr int WPG = Cfg::WPG;
  constexpr int TILE = Cfg::TILE;
  constexpr int VEC = Cfg::VEC;
  constexpr bool FWD = (MODE == STEP || MODE == FINAL);
  constexpr bool NEED_G = (MODE == GRAD || MODE == SCATTER);
  constexpr bool NEED_U = (MODE == ADJ || MODE == SCATTER);
  constexpr bool ACCUM = (NACC > 0);
  constexpr int NA = ACCUM ? NACC : 1;
  constexpr int KH = KPL / 2;
  // weight-vectors of a group per unrolled loop body: two in the forward passes (more independent work per warp);
  // one in the backward passes, whose register budget is already full (measured: 4 % faster than two)
  constexpr int WUNROLL = FWD ? 2 : 1;
  // thread-per-weight forward step: runs of whole trips in a streamlined inner loop (see the tile loop)
  constexpr bool STREAM_RUNS = (LPW == 1);
  // The adjoint step takes each row's softmax reference and normaliser from p.rowstat (written by the
  // codebook-gradient pass at the same centroids, with the same arithmetic, so the exponentials come out bit-equal):
  // no row minimum, no row sum, no cross-lane reduction before the exponentials and no reciprocal.
  constexpr bool ROWSTAT_R = (MODE == ADJ) && row_cache_layout(D, LPW);
  constexpr bool ROWSTAT_W = (MODE == GRAD) && row_cache_layout(D, LPW);

  // shared: cross-warp reduction buffer (floats), reused by the last block as fp64 scratch
  constexpr int RED_BYTES = ACCUM ? NWARP * PLEN * 4 : 16;
  constexpr int LAST_BYTES = ACCUM ? (PLEN + BLOCK) * 8 : 16;
  constexpr int SMEM_BYTES = RED_BYTES > LAST_BYTES ? RED_BYTES : LAST_BYTES;
  __shared__ __align__(16) unsigned char smem_raw[SMEM_BYTES];
  __shared__ int s_flag;
  // group-per-weight layouts stage each tile's rows in shared memory (one slot per group)
  constexpr int STAGE = (LPW > 1) ? Cfg::GROUPS * WPG * D : 4;
  constexpr int LD = (LPW > 1) ? (WPG + LPW - 1) / LPW : 1;   // rows each lane fetches per tile
  extern __shared__ __align__(16) float slots[];   // [KPL * NA][BLOCK]: second-level sums, one column per thread
  __shared__ __align__(16) float wstage[STAGE];
  __shared__ __align__(16) float gstage[NEED_G ? STAGE : 4];
  __shared__ float2 lstage[ROWSTAT_R ? Cfg::GROUPS * WPG : 1];
  __shared__ float2 ostage[ROWSTAT_W ? Cfg::GROUPS * WPG : 1];
  int stage_slot = 0;   // where the row being processed parks its (reference, 1 / sum)
  (void)ostage; (void)stage_slot;
  (void)wstage; (void)gstage; (void)lstage;

  const int tid = threadIdx.x;
  const int lane = tid & 31;
  const int warp = tid >> 5;
  const int gl = (LPW == 1) ? 0 : (lane % LPW);   // lane index inside its group
  const int grp = tid / LPW;                      // group index inside the block
  const int k = p.k;
  const int nb = p.lt.n_blocks;
  const int b = blockIdx.x;
  const int t_lo = tile_begin(b, p.lt.tiles_total, nb);
  const int t_hi = tile_begin(b + 1, p.lt.tiles_total, nb);
  if (b >= nb || t_lo >= t_hi) return;   // (the dual step kernel's grid can be larger than this pass's table)

  // Centroids and sums are held as float2 pairs of neighbouring centroids (2h, 2h+1); c_(t, a) / acc_(t, a) give
  // the scalar view, which resolves to a register half once the loops are unrolled.  (The packed fp32x2
  // instructions of sm_100 were measured on this layout: they halve the issue slots of the FMAs but run on half of
  // the FMA pipe, and the step came out slower, so the arithmetic below is scalar.)
  float2 c2[KH][D];                // owned centroids
  // u_j / S_j (0 for a dead cluster) and kap_j = (u_j / S_j) . F(C_T, W)_j, so that p_ij = (u_j / S_j) . w_i - kap_j.
  // The full-warp layouts and the 16-centroids-per-lane layout keep them in shared memory ([t][lane] order:
  // conflict-free), the others in registers: with 8 centroids per lane at two blocks per SM, or with 16 per lane, the
  // registers do not hold them without spilling.
  constexpr bool US_SMEM = NEED_U && (LPW == 32 || KPL == 16);
  float us[(NEED_U && !US_SMEM) ? KPL : 1][D];
  float kap[(NEED_U && !US_SMEM) ? KPL : 1];
  __shared__ __align__(16) float us_sm[US_SMEM ? KPL * LPW * D : 4];
  __shared__ float kap_sm[US_SMEM ? KPL * LPW : 1];
  (void)us_sm; (void)kap_sm;
  auto us_ = [&](int t, int a) -> float { return US_SMEM ? us_sm[(t * LPW + gl) * D + a] : us[US_SMEM ? 0 : t][a]; };
  auto kap_ = [&](int t) -> float { return US_SMEM ? kap_sm[t * LPW + gl] : kap[US_SMEM ? 0 : t]; };
  float2 acc2[ACCUM ? KH : 1][NA];
  (void)kap; (void)us; (void)acc2;
  auto c_ = [&](int t, int a) -> float& { return (t & 1) ? c2[t >> 1][a].y : c2[t >> 1][a].x; };
  auto acc_ = [&](int t, int a) -> float& { return (t & 1) ? acc2[t >> 1][a].y : acc2[t >> 1][a].x; };

  int layer = 0;
  while (p.lt.tile_off[layer + 1] <= t_lo) ++layer;
  int cur_layer = -1;
  bool layer_active = false;

  auto load_layer = [&](int l) {
    const float* Cl = p.C + (size_t)l * k * D;
#pragma unroll
    for (int t = 0; t < KPL; ++t) {
      const int j = gl * KPL + t;
#pragma unroll
      for (int a = 0; a < D; ++a) c_(t, a) = (j < k) ? Cl[j * D + a] : PAD_COORD;
      if constexpr (NEED_U) {
        const float s = (j < k) ? p.S[(size_t)l * k + j] : 0.f;
        const float inv = (s >= S_MIN_F) ? 1.f / s : 0.f;
        float kp = 0.f;
#pragma unroll
        for (int a = 0; a < D; ++a) {
          const float f = (j < k) ? p.F[((size_t)l * k + j) * D + a] : 0.f;
          const float uv = (j < k) ? p.u[((size_t)l * k + j) * D + a] * inv : 0.f;
          kp = fmaf(uv, f, kp);
          if constexpr (US_SMEM) {
            if (grp == 0) us_sm[(t * LPW + gl) * D + a] = uv;
          } else {
            us[t][a] = uv;
          }
        }
        if constexpr (US_SMEM) {
          if (grp == 0) kap_sm[t * LPW + gl] = kp;
        } else {
          kap[t] = kp;
        }
      }
      if constexpr (ACCUM) {
#pragma unroll
        for (int a = 0; a < NA; ++a) {
          acc_(t, a) = 0.f;
          slots[(t * NA + a) * BLOCK + tid] = 0.f;
        }
      }
    }
  };
  int since_spill = 0;
  auto spill = [&]() {
    if constexpr (ACCUM) {
#pragma unroll
      for (int t = 0; t < KPL; ++t)
#pragma unroll
        for (int a = 0; a < NA; ++a) {
          slots[(t * NA + a) * BLOCK + tid] += acc_(t, a);
          acc_(t, a) = 0.f;
        }
    }
  };

  // ---- per weight-vector work: returns through the accumulators / writes row outputs ----------
  auto process = [&](const float (&w)[D], const float (&gi)[D], bool valid, long long row, float (&out)[D], float2 rstat) {
    if constexpr (ROWSTAT_R) {
      // Adjoint step with the row's reference and normaliser at hand: nothing separates a pair's distance from its
      // exponential, so each centroid is taken from distance to eps_ij / (p_ij - pbar_i) in one go and only two
      // values per centroid (that product's left factor and p_ij) stay live for the second loop.
      float ers[KPL], z[KPL];
      float lzp[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int t = 0; t < KPL; ++t) {
        // keeps the shared-memory reads of the second half of the centroids (u_j / S_j, kappa_j) from being hoisted
        // above the first half's arithmetic, which cost more registers than the full-warp layout at d = 4 has
        if (US_SMEM && D == 4 && t == KPL / 2) __syncwarp();
        float dist_t, rs_t = 1.f;
        if constexpr (SQ) {
          float sq = 0.f;
#pragma unroll
          for (int a = 0; a < D; ++a) {
            const float df = w[a] - c_(t, a);
            sq = fmaf(df, df, sq);
          }
          dist_t = sq;
        } else if constexpr (D == 1) {
          dist_t = fabsf(w[0] - c_(t, 0));
        } else {
          float sq = 1e-30f;   // rsqrt stays finite when w == c (n_ij = 0 then)
#pragma unroll
          for (int a = 0; a < D; ++a) {
            const float df = w[a] - c_(t, a);
            sq = fmaf(df, df, sq);
          }
          rs_t = rsqrt_approx(sq);
          dist_t = sq * rs_t;
        }
        const float et0 = ex2_approx(fmaf(-p.scale, dist_t, rstat.x));
        float v = -kap_(t);
#pragma unroll
        for (int a = 0; a < D; ++a) v = fmaf(us_(t, a), w[a], v);
        z[t] = v;
        lzp[t & 3] = fmaf(et0, v, lzp[t & 3]);
        ers[t] = (D > 1 && !SQ) ? et0 * rs_t : et0;
      }
      const float rr = rstat.y;
      const float zbar = group_sum<LPW>((lzp[0] + lzp[1]) + (lzp[2] + lzp[3])) * rr;
      const float rt = rr * (SQ ? 2.f * p.inv_tau : p.inv_tau);   // squared distance: n_ij = 2 (w_i - c_j)
      const float nzr = -zbar * rt;
#pragma unroll
      for (int t = 0; t < KPL; ++t) {
        const float et = ers[t] * fmaf(z[t], rt, nzr);   // e_ij(p) / (tau D_ij)
#pragma unroll
        for (int a = 0; a < D; ++a) {
          const float df = w[a] - c_(t, a);
          float n;
          if constexpr (D == 1 && !SQ) n = (df > 0.f) ? 1.f : ((df < 0.f) ? -1.f : 0.f);
          else n = df;
          acc_(t, a) = fmaf(et, n, acc_(t, a));
        }
      }
      return;
    }
    float dist[KPL];
    float rs[(D > 1 && !FWD && !SQ) ? KPL : 1];
    (void)rs; (void)dist;
    float e[KPL];
    float lmin = 3.0e38f;
    float lsum = 0.f;
    float gsum, r;
    {
#pragma unroll
      for (int t = 0; t < KPL; ++t) {
        if constexpr (SQ) {
          float sq = 0.f;
#pragma unroll
          for (int a = 0; a < D; ++a) {
            const float df = w[a] - c_(t, a);
            sq = fmaf(df, df, sq);
          }
          dist[t] = sq;
        } else if constexpr (D == 1) {
          dist[t] = fabsf(w[0] - c_(t, 0));
        } else {
          // the backward passes start the square at 1e-30 so that rsqrt stays finite when w == c (n_ij = 0 then)
          float sq = FWD ? 0.f : 1e-30f;
#pragma unroll
          for (int a = 0; a < D; ++a) {
            const float df = w[a] - c_(t, a);
            sq = fmaf(df, df, sq);
          }
          if constexpr (FWD) {
            dist[t] = sqrt_approx(sq);
          } else {
            rs[t] = rsqrt_approx(sq);
            dist[t] = sq * rs[t];
          }
        }
      }
      {
        lmin = tree_reduce<KPL, 1>(dist);
        const float gmin = group_min<LPW>(lmin);
        const float mref = gmin * p.scale;
#pragma unroll
        for (int t = 0; t < KPL; ++t) {
          e[t] = ex2_approx(fmaf(-p.scale, dist[t], mref));
        }
        lsum = tree_reduce<KPL, 0>(e);
        gsum = group_sum<LPW>(lsum);
        r = valid ? rcp_approx(gsum) : 0.f;
        if constexpr (ROWSTAT_W) {
          if (gl == 0) ostage[stage_slot] = make_float2(mref, r);   // stored to the workspace once per tile
        }
      }
    }

    if constexpr (MODE == STEP || MODE == FINAL) {
      float rw[D];
#pragma unroll
      for (int a = 0; a < D; ++a) rw[a] = r * w[a];
#pragma unroll
      for (int t = 0; t < KPL; ++t) {
        acc_(t, 0) = fmaf(e[t], r, acc_(t, 0));
#pragma unroll
        for (int a = 0; a < D; ++a) acc_(t, 1 + a) = fmaf(e[t], rw[a], acc_(t, 1 + a));
      }
      if constexpr (MODE == FINAL) {
        if (p.Wq != nullptr) {
#pragma unroll
          for (int a = 0; a < D; ++a) {
            float sp[2] = {0.f, 0.f};
#pragma unroll
            for (int t = 0; t < KPL; ++t) sp[t & 1] = fmaf(e[t], (gl * KPL + t < k) ? c_(t, a) : 0.f, sp[t & 1]);
            out[a] = group_sum<LPW>(sp[0] + sp[1]) * r;
          }
        }
        if (p.A != nullptr && valid) {
          float* Arow = p.A + (size_t)row * k;
#pragma unroll
          for (int t = 0; t < KPL; ++t) {
            const int j = gl * KPL + t;
            if (j < k) Arow[j] = e[t] * r;
          }
        }
      }
    } else {
      // z_ij: what the softmax Jacobian is contracted with (q for GRAD, p for ADJ, q + p for SCATTER)
      float z[KPL];
      float lzp[4] = {0.f, 0.f, 0.f, 0.f};   // four interleaved partial sums keep the dependent chain short
#pragma unroll
      for (int t = 0; t < KPL; ++t) {
        float v = 0.f;
        if constexpr (NEED_U) {
          v = -kap_(t);
#pragma unroll
          for (int a = 0; a < D; ++a) v = fmaf(us_(t, a), w[a], v);
        }
        if constexpr (NEED_G) {
#pragma unroll
          for (int a = 0; a < D; ++a) v = fmaf(gi[a], (gl * KPL + t < k) ? c_(t, a) : 0.f, v);
        }
        z[t] = v;
        lzp[t & 3] = fmaf(e[t], v, lzp[t & 3]);
      }
      const float zbar = group_sum<LPW>((lzp[0] + lzp[1]) + (lzp[2] + lzp[3])) * r;
      const float rt = r * (SQ ? 2.f * p.inv_tau : p.inv_tau);   // squared distance: n_ij = 2 (w_i - c_j)
      const float nzr = -zbar * rt;
      float dwl[D];
#pragma unroll
      for (int a = 0; a < D; ++a) dwl[a] = 0.f;
#pragma unroll
      for (int t = 0; t < KPL; ++t) {
        const float at = e[t] * r;                    // A_ij
        float et = e[t] * fmaf(z[t], rt, nzr);        // e_ij(z) / tau = A_ij (z_ij - zbar_i) / tau
        if constexpr (D > 1 && !SQ) et *= rs[t];      // ... / D_ij, so that et * (w - c) = e_ij(z) n_ij / tau
#pragma unroll
        for (int a = 0; a < D; ++a) {
          const float df = w[a] - c_(t, a);
          float n;
          if constexpr (D == 1 && !SQ) n = (df > 0.f) ? 1.f : ((df < 0.f) ? -1.f : 0.f);
          else n = df;
          if constexpr (MODE == GRAD) acc_(t, a) = fmaf(at, gi[a], fmaf(et, n, acc_(t, a)));
          if constexpr (MODE == ADJ) acc_(t, a) = fmaf(et, n, acc_(t, a));
          if constexpr (MODE == SCATTER) dwl[a] = fmaf(at, us_(t, a), fmaf(-et, n, dwl[a]));
        }
      }
      if constexpr (MODE == SCATTER) {
#pragma unroll
        for (int a = 0; a < D; ++a) out[a] = group_sum<LPW>(dwl[a]);
      }
    }
  };

  // ---- flush: block-reduce the accumulators of the current layer and maybe finish the layer ----
  auto flush = [&](int l) {
    if constexpr (!ACCUM) {
      return;
    } else {
      float* red = reinterpret_cast<float*>(smem_raw);
      // across the groups of a warp (lanes with equal gl); the thread's own two levels are joined first
#pragma unroll
      for (int t = 0; t < KPL; ++t)
#pragma unroll
        for (int a = 0; a < NA; ++a) {
          float v = acc_(t, a) + slots[(t * NA + a) * BLOCK + tid];
#pragma unroll
          for (int o = LPW; o < 32; o <<= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
          acc_(t, a) = v;
        }
      __syncthreads();
      if (lane < LPW) {
#pragma unroll
        for (int t = 0; t < KPL; ++t)
#pragma unroll
          for (int a = 0; a < NA; ++a) red[warp * PLEN + (gl * KPL + t) * NA + a] = acc_(t, a);
      }
      __syncthreads();
      const int slot = b + l;
      double* mine = p.partials + (size_t)slot * PLEN;
      for (int o = tid; o < PLEN; o += BLOCK) {
        double s = 0.0;
#pragma unroll
        for (int wv = 0; wv < NWARP; ++wv) s += (double)red[wv * PLEN + o];
        mine[o] = s;
      }
      finish_layer<MODE, D, PLEN, NA>(p, l, b, smem_raw, &s_flag);
    }
  };

  // rows fetched one tile ahead by this lane (group-per-weight layouts)
  float pw[LD][D], pg[NEED_G ? LD : 1][D], pl2[ROWSTAT_R ? LD : 1][2];
  (void)pw; (void)pg; (void)pl2;
  auto fetch = [&](int tl, int ly) {
    if constexpr (LPW > 1) {
      const long long r0 = p.lt.row_off[ly];
      const long long rws = p.lt.row_off[ly + 1] - r0;
      const long long gb = (long long)(tl - p.lt.tile_off[ly]) * TILE + (long long)grp * WPG;
#pragma unroll
      for (int q = 0; q < LD; ++q) {
        const int idx = gl + q * LPW;
        if (idx < WPG) {
          const long long loc = gb + idx;
          const long long grow = r0 + ((loc < rws) ? loc : 0);
          if constexpr (D == 4) {
            const float4 x = __ldg(reinterpret_cast<const float4*>(p.W + grow * 4));
            pw[q][0] = x.x; pw[q][1] = x.y; pw[q][2] = x.z; pw[q][3] = x.w;
          } else if constexpr (D == 2) {
            const float2 x = __ldg(reinterpret_cast<const float2*>(p.W + grow * 2));
            pw[q][0] = x.x; pw[q][1] = x.y;
          } else {
            pw[q][0] = __ldg(p.W + grow);
          }
          if constexpr (ROWSTAT_R) {
            const float2 y = __ldg(p.rowstat + grow);
            pl2[q][0] = y.x; pl2[q][1] = y.y;
          }
          if constexpr (NEED_G) {
            if constexpr (D == 4) {
              const float4 y = __ldg(reinterpret_cast<const float4*>(p.G + grow * 4));
              pg[q][0] = y.x; pg[q][1] = y.y; pg[q][2] = y.z; pg[q][3] = y.w;
            } else if constexpr (D == 2) {
              const float2 y = __ldg(reinterpret_cast<const float2*>(p.G + grow * 2));
              pg[q][0] = y.x; pg[q][1] = y.y;
            } else {
              pg[q][0] = __ldg(p.G + grow);
            }
          }
        }
      }
    }
  };
  fetch(t_lo, layer);

  // ---- bulk-copy pipeline (see BULK above): stages after the second-level sums in dynamic shared memory ----------
  constexpr bool BULK_ON = BULK && (LPW == 1) && (MODE == STEP);
  constexpr int STAGE_FLOATS = BULK_ON ? Cfg::UNROLL * BLOCK * 4 : 4;
  __shared__ __align__(8) unsigned long long bfull[BULK_ON ? BULK_STAGES : 1];
  float* bstage = slots + (ACCUM ? BLOCK * KPL * NA : 0);
  int ptile = t_lo, player = layer;   // producer cursor (used by thread 0)
  int cons_n = 0;                      // bulk trips consumed so far
  (void)bfull; (void)bstage; (void)ptile; (void)player; (void)cons_n;
  // The next trip at or after the producer cursor whose layer steps in this launch and whose rows start on a 16-byte
  // boundary is copied into stage n % BULK_STAGES (trips of other layers are skipped; unaligned layers keep the
  // per-thread loads).  The routing flags do not change while a launch runs, so producer and consumer agree.
  auto bulk_issue = [&](int n) {
    if constexpr (BULK_ON) {
      while (ptile < t_hi) {
        while (p.lt.tile_off[player + 1] <= ptile) ++player;
        const int lim = (t_hi < p.lt.tile_off[player + 1]) ? t_hi : p.lt.tile_off[player + 1];
        const int a = (lim - ptile < Cfg::UNROLL) ? lim - ptile : Cfg::UNROLL;
        const int tl = ptile;
        ptile += a;
        const bool act = (p.st[player].fwd_done == 0) && (p.st[player].precise[p.iter & 1] == 0) &&
                         (p.st[player].fwd_iters == p.iter);
        const long long r0 = p.lt.row_off[player];
        if (!act || (r0 * D) % 4 != 0) continue;
        const long long rws = p.lt.row_off[player + 1] - r0;
        const long long tb = (long long)(tl - p.lt.tile_off[player]) * TILE;
        long long nrows = (long long)a * TILE;
        if (nrows > rws - tb) nrows = rws - tb;
        const unsigned bytes = (unsigned)(nrows * D * 4);
        const unsigned ab = bytes & ~15u;
        float* dst = bstage + (n % BULK_STAGES) * STAGE_FLOATS;
        const float* src = p.W + (r0 + tb) * D;
        for (unsigned q = ab / 4; q < bytes / 4; ++q) dst[q] = __ldg(src + q);   // at most three trailing floats
        mbar_arrive_expect_tx(&bfull[n % BULK_STAGES], ab);
        if (ab > 0) bulk_copy_g2s(dst, src, ab, &bfull[n % BULK_STAGES]);
        return;
      }
    }
  };
  if constexpr (BULK_ON) {
    if (tid == 0) {
#pragma unroll
      for (int q = 0; q < BULK_STAGES; ++q) mbar_init(&bfull[q], 1);
      mbar_init_fence();
    }
    __syncthreads();
    if (tid == 0) {
#pragma unroll
      for (int q = 0; q < BULK_STAGES; ++q) bulk_issue(q);
    }
  }

  // ---- persistent loop over this block's tiles -------------------------------------------------
  int adv = 1;   // tiles consumed per trip: 1, or up to UNROLL consecutive tiles of one layer (thread-per-weight)
  for (int tile = t_lo; tile < t_hi; tile += adv) {
    while (p.lt.tile_off[layer + 1] <= tile) ++layer;
    if constexpr (LPW == 1) {
      const int lim = (t_hi < p.lt.tile_off[layer + 1]) ? t_hi : p.lt.tile_off[layer + 1];
      adv = (lim - tile < Cfg::UNROLL) ? lim - tile : Cfg::UNROLL;
    }
    if (layer != cur_layer) {
      if (cur_layer >= 0 && layer_active) flush(cur_layer);
      cur_layer = layer;
      if constexpr (MODE == STEP)
        layer_active = (p.st[layer].fwd_done == 0) && (p.st[layer].precise[p.iter & 1] == 0) && (p.st[layer].fwd_iters == p.iter);
      else if constexpr (MODE == ADJ) layer_active = (p.st[layer].adj_done == 0);
      else layer_active = true;
      if constexpr (US_SMEM) __syncthreads();   // the previous layer's table is no longer read
      if (layer_active) load_layer(layer);
      if constexpr (US_SMEM) __syncthreads();   // table written by the first group, read by all
      since_spill = 0;
    }
    if constexpr (LPW > 1) {
      // park the rows fetched for this tile, then fetch the next tile's while this one is processed
      __syncwarp();
#pragma unroll
      for (int q = 0; q < LD; ++q) {
        const int idx = gl + q * LPW;
        if (idx < WPG) {
#pragma unroll
          for (int a = 0; a < D; ++a) {
            wstage[(grp * WPG + idx) * D + a] = pw[q][a];
            if constexpr (NEED_G) gstage[(grp * WPG + idx) * D + a] = pg[q][a];
          }
          if constexpr (ROWSTAT_R) lstage[grp * WPG + idx] = make_float2(pl2[q][0], pl2[q][1]);
        }
      }
      __syncwarp();
      if (tile + 1 < t_hi) {
        int ly2 = layer;
        while (p.lt.tile_off[ly2 + 1] <= tile + 1) ++ly2;
        fetch(tile + 1, ly2);
      }
    }
    if (!layer_active) continue;
    const long long row0 = p.lt.row_off[layer];
    const long long rows = p.lt.row_off[layer + 1] - row0;
    const long long tbase = (long long)(tile - p.lt.tile_off[layer]) * TILE;   // first row of the tile in the layer

    if constexpr (LPW == 1) {
      const bool vec_ok = ((row0 * D) % 4 == 0);
      constexpr int UN = Cfg::UNROLL;
      // Forward step: a run of whole trips inside one layer (every row exists, rows start on a 16-byte boundary) is
      // taken in one inner loop with a running pointer -- no tile, layer or range arithmetic per trip -- and the
      // 128-bit loads of the next trip are issued before the arithmetic of the current one.
      if constexpr (MODE == STEP && !BULK_ON && STREAM_RUNS) {
        const int lim_r = (t_hi < p.lt.tile_off[layer + 1]) ? t_hi : p.lt.tile_off[layer + 1];
        const long long by_rows = (rows - tbase) / ((long long)UN * TILE);
        const int by_tiles = (lim_r - tile) / UN;
        const int nfull = vec_ok ? (by_rows < (long long)by_tiles ? (int)by_rows : by_tiles) : 0;
        if (nfull > 0) {
          const float4* wp = reinterpret_cast<const float4*>(p.W + (row0 + tbase) * D) + tid;
          float4 cur[UN], nxt[UN];
#pragma unroll
          for (int un = 0; un < UN; ++un) nxt[un] = cur[un] = __ldg(wp + un * BLOCK);
#pragma unroll 1
          for (int s = 0; s < nfull; ++s) {
            wp += UN * BLOCK;
            if (s + 1 < nfull) {
#pragma unroll
              for (int un = 0; un < UN; ++un) nxt[un] = __ldg(wp + un * BLOCK);
            }
#pragma unroll
            for (int un = 0; un < UN; ++un) {
              const float xs[4] = {cur[un].x, cur[un].y, cur[un].z, cur[un].w};
#pragma unroll
              for (int v = 0; v < VEC; ++v) {
                float w1[D], g0[D], o0[D];
#pragma unroll
                for (int a = 0; a < D; ++a) {
                  w1[a] = xs[v * D + a];
                  g0[a] = 0.f;
                }
                process(w1, g0, true, 0, o0, make_float2(0.f, 0.f));
              }
            }
            since_spill += UN;
            if (since_spill >= Cfg::SPILL_TILES) {
              spill();
              since_spill = 0;
            }
#pragma unroll
            for (int un = 0; un < UN; ++un) cur[un] = nxt[un];
          }
          adv = nfull * UN;
          continue;
        }
      }
      float wv[UN][VEC][D];
      float gv[UN][VEC][D];
      (void)gv;
      long long first[UN];
      bool from_stage = false;
      if constexpr (BULK_ON) {
        if (vec_ok) {
          // this trip's rows were copied to a stage: wait for the copy (bounded), take this thread's rows, hand the
          // stage back and let thread 0 start the copy of the trip BULK_STAGES ahead
          from_stage = true;
          unsigned long long* bar = &bfull[cons_n % BULK_STAGES];
          const unsigned parity = (unsigned)((cons_n / BULK_STAGES) & 1);
          bool arrived = false;
          for (int poll = 0; poll < BULK_WAIT_POLLS && !arrived; ++poll) arrived = mbar_try_wait(bar, parity);
          const float* stg = bstage + (cons_n % BULK_STAGES) * STAGE_FLOATS;
#pragma unroll
          for (int un = 0; un < UN; ++un) {
            const long long loc = (un < adv) ? tbase + (long long)(un * BLOCK + tid) * VEC : rows;
            first[un] = loc;
            const float4 x = *reinterpret_cast<const float4*>(stg + (un * BLOCK + tid) * 4);
            const float xs[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
            for (int v = 0; v < VEC; ++v)
#pragma unroll
              for (int a = 0; a < D; ++a) wv[un][v][a] = (arrived && loc + v < rows) ? xs[v * D + a] : 0.f;
          }
          if (__syncthreads_or(arrived ? 0 : 1)) {
            // a copy never arrived: report it and leave (the layer's reduction is not completed, the layer stops)
            if (tid == 0) p.st[layer].status = ST_TIMEOUT;
            return;
          }
          if (tid == 0) bulk_issue(cons_n + BULK_STAGES);
          ++cons_n;
        }
      }
      // A trip of UNROLL whole tiles on a 16-byte boundary (all but a layer's last trip, as a rule) takes the same
      // code with every row known to exist: no per-row range test, no select on the normaliser.
      auto trip = [&](auto full_c) {
      constexpr bool FULL = decltype(full_c)::value;
      // issue all loads of the tile first
#pragma unroll
      for (int un = 0; un < UN; ++un) {
        if (from_stage) break;
        // trips shorter than UNROLL tiles mark the missing tiles as out of range
        const long long loc = (FULL || un < adv) ? tbase + (long long)(un * BLOCK + tid) * VEC : rows;
        first[un] = loc;
        const long long grow = row0 + loc;
        if (FULL || (vec_ok && loc + VEC <= rows)) {
          const float4 x = __ldg(reinterpret_cast<const float4*>(p.W + grow * D));
          const float xs[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
          for (int v = 0; v < VEC; ++v)
#pragma unroll
            for (int a = 0; a < D; ++a) wv[un][v][a] = xs[v * D + a];
          if constexpr (NEED_G) {
            const float4 y = __ldg(reinterpret_cast<const float4*>(p.G + grow * D));
            const float ys[4] = {y.x, y.y, y.z, y.w};
#pragma unroll
            for (int v = 0; v < VEC; ++v)
#pragma unroll
              for (int a = 0; a < D; ++a) gv[un][v][a] = ys[v * D + a];
          }
        } else {
#pragma unroll
          for (int v = 0; v < VEC; ++v) {
            const bool ok = (loc + v < rows);
#pragma unroll
            for (int a = 0; a < D; ++a) {
              wv[un][v][a] = ok ? __ldg(p.W + (grow + v) * D + a) : 0.f;
              if constexpr (NEED_G) gv[un][v][a] = ok ? __ldg(p.G + (grow + v) * D + a) : 0.f;
            }
          }
        }
      }
#pragma unroll
      for (int un = 0; un < UN; ++un) {
        const long long loc = first[un];
        const long long grow = row0 + loc;
        float outv[VEC][D];
#pragma unroll
        for (int v = 0; v < VEC; ++v) {
          float gdummy[D];
#pragma unroll
          for (int a = 0; a < D; ++a) gdummy[a] = 0.f;
          if constexpr (NEED_G) process(wv[un][v], gv[un][v], FULL || loc + v < rows, grow + v, outv[v], make_float2(0.f, 0.f));
          else process(wv[un][v], gdummy, FULL || loc + v < rows, grow + v, outv[v], make_float2(0.f, 0.f));
        }
        if constexpr (MODE == FINAL || MODE == SCATTER) {
          float* dst = (MODE == FINAL) ? static_cast<float*>(p.Wq) : p.dW;
          if (dst != nullptr) {
            if (FULL || (vec_ok && loc + VEC <= rows)) {
              float os[4];
#pragma unroll
              for (int v = 0; v < VEC; ++v)
#pragma unroll
                for (int a = 0; a < D; ++a) os[v * D + a] = outv[v][a];
              if constexpr (MODE == FINAL) store_wq<4>(p.Wq, grow * D, os, p.wq_dtype, true);
              else *reinterpret_cast<float4*>(dst + grow * D) = make_float4(os[0], os[1], os[2], os[3]);
            } else {
#pragma unroll
              for (int v = 0; v < VEC; ++v)
                if (loc + v < rows)
#pragma unroll
                  for (int a = 0; a < D; ++a) {
                    if constexpr (MODE == FINAL) {
                      const float one[1] = {outv[v][a]};
                      store_wq<1>(p.Wq, (grow + v) * D + a, one, p.wq_dtype, false);
                    } else {
                      dst[(grow + v) * D + a] = outv[v][a];
                    }
                  }
            }
          }
        }
      }
      };
      // (layouts with one load per trip measured 5 % slower with the second copy of the body: d = 4, k = 8)
      if (UN > 1 && !from_stage && vec_ok && adv == UN && tbase + (long long)UN * TILE <= rows) trip(std::true_type{});
      else trip(std::false_type{});
    } else {
      // group-per-weight: the group reads one staged row at a time (a shared-memory broadcast)
      const long long gbase = tbase + (long long)grp * WPG;
      // rows of this group's share of the tile that exist (the last tile of a layer may be ragged): one 32-bit
      // count per tile, so that the row loop carries no 64-bit arithmetic (the backward kernels sit at their
      // register limit and would otherwise recompute row indices and staging addresses for every row)
      const long long left = rows - gbase;
      const int nvalid = left >= WPG ? WPG : (left > 0 ? (int)left : 0);
      auto one_row = [&](int t, bool ok, const float* ws, const float* gs, const float2* ls) {
        float w[D], gi[D], outv[D];
        if constexpr (D == 4) {
          const float4 x = *reinterpret_cast<const float4*>(ws);
          w[0] = x.x; w[1] = x.y; w[2] = x.z; w[3] = x.w;
        } else if constexpr (D == 2) {
          const float2 x = *reinterpret_cast<const float2*>(ws);
          w[0] = x.x; w[1] = x.y;
        } else {
          w[0] = ws[0];
        }
#pragma unroll
        for (int a = 0; a < D; ++a) gi[a] = 0.f;
        if constexpr (NEED_G) {
          if constexpr (D == 4) {
            const float4 y = *reinterpret_cast<const float4*>(gs);
            gi[0] = y.x; gi[1] = y.y; gi[2] = y.z; gi[3] = y.w;
          } else if constexpr (D == 2) {
            const float2 y = *reinterpret_cast<const float2*>(gs);
            gi[0] = y.x; gi[1] = y.y;
          } else {
            gi[0] = gs[0];
          }
        }
        float2 rstat = make_float2(0.f, 0.f);
        if constexpr (ROWSTAT_R) {
          rstat = *ls;
          if (!ok) rstat.y = 0.f;      // a zero normaliser switches the row off
        }
        if constexpr (ROWSTAT_W) stage_slot = grp * WPG + t;
        long long grow = 0;
        if constexpr (MODE == FINAL || MODE == SCATTER) grow = row0 + gbase + (ok ? t : 0);
        process(w, gi, ok, grow, outv, rstat);
        if constexpr (MODE == FINAL || MODE == SCATTER) {
          float* dst = (MODE == FINAL) ? static_cast<float*>(p.Wq) : p.dW;
          if (dst != nullptr && ok && gl == 0) {
            if constexpr (MODE == FINAL) store_wq<D>(p.Wq, grow * D, outv, p.wq_dtype, true);
            else if constexpr (D == 4) *reinterpret_cast<float4*>(dst + grow * 4) = make_float4(outv[0], outv[1], outv[2], outv[3]);
            else if constexpr (D == 2) *reinterpret_cast<float2*>(dst + grow * 2) = make_float2(outv[0], outv[1]);
            else dst[grow] = outv[0];
          }
        }
      };
      if constexpr (MODE == STEP) {
        // the forward step measured 10 % slower with the loop below (two rows in flight interleave less well)
#pragma unroll WUNROLL
        for (int t = 0; t < WPG; ++t)
          one_row(t, gbase + t < rows, wstage + (grp * WPG + t) * D, gstage + (NEED_G ? (grp * WPG + t) * D : 0), lstage + (ROWSTAT_R ? grp * WPG + t : 0));
      } else {
        // running pointers: one add per staged array and row
        const float* ws = wstage + grp * (WPG * D);
        const float* gs = gstage + (NEED_G ? grp * (WPG * D) : 0);
        const float2* ls = lstage + (ROWSTAT_R ? grp * WPG : 0);
#pragma unroll WUNROLL
        for (int t = 0; t < WPG; ++t) {
          one_row(t, t < nvalid, ws, gs, ls);
          ws += D;
          if constexpr (NEED_G) gs += D;
          if constexpr (ROWSTAT_R) ls += 1;
        }
      }
      if constexpr (ROWSTAT_W) {
        // the tile's (reference, 1 / sum) pairs go to the workspace together, one row per lane
        __syncwarp();
        if (p.rowstat != nullptr) {
#pragma unroll
          for (int q = 0; q < LD; ++q) {
            const int idx = gl + q * LPW;
            if (idx < WPG && gbase + idx < rows) p.rowstat[row0 + gbase + idx] = ostage[grp * WPG + idx];
          }
        }
        __syncwarp();
      }
    }
    if constexpr (ACCUM) {
      since_spill += adv;
      if (since_spill >= Cfg::SPILL_TILES) {
        spill();
        since_spill = 0;
      }
    }
  }
  if constexpr (RELEASE) grid_release_dependents();
  if (cur_layer >= 0 && layer_active) flush(cur_layer);
}

template <int MODE, int D, int KPL, int LPW, bool SQ = false, bool BULK = false>
__global__ void __launch_bounds__(BLOCK, PassCfg<MODE, D, KPL, LPW>::MIN_BLOCKS)
idkm_pass(const __grid_constant__ PassParams p) {
  grid_dependency_sync();
  pass_body<MODE, D, KPL, LPW, true, SQ, BULK>(p);
}


// ---- fp64 forward step for collapsing layers ------------------------------------------------------------
// Same sums as the STEP pass, for the layers flagged `precise`.  There every logit difference is below
// PRECISE_SPAN, so exp is a short Taylor series, and everything from w - c to the accumulation is fp64.
template <int D, int KPL, int LPW>
struct PreciseCfg {
  static constexpr int KP = KPL * LPW;
  static constexpr int NA = D + 1;
  static constexpr int PLEN = KP * NA;
  static constexpr int WPG = (LPW == 1) ? 4 : 16;   // small tiles in the thread-per-weight layouts spread small layers
  static constexpr int TILE = (BLOCK / LPW) * WPG;
  // small codebooks in the thread-per-weight layout: four resident blocks per SM (64 registers) hide the latency of
  // the dependent fp64 chains better than two blocks with more rows in flight each
  static constexpr int MIN_BLOCKS = (LPW == 1 && KPL * (D + 1) <= 8) ? 4 : 1;
};

// exp(z / tau) for |z / tau| <= PRECISE_SPAN by the Taylor series to the sixth power (truncation error
// y^7/5040 < 8e-13 relative), with 1 / tau folded into the coefficients ec[n] = (1/tau)^(n+1) / (n+1)!: six fused
// multiply-adds and no separate scaling.  (1/tau)^6 is finite for every positive float tau.
__device__ __forceinline__ void exp_scaled_coeffs(double inv_tau, double (&ec)[6]) {
  const double f[6] = {1.0, 0.5, 1.0 / 6.0, 1.0 / 24.0, 1.0 / 120.0, 1.0 / 720.0};
  double pw = inv_tau;
#pragma unroll
  for (int n = 0; n < 6; ++n) {
    ec[n] = pw * f[n];
    pw *= inv_tau;
  }
}
__device__ __forceinline__ double exp_scaled(double z, const double (&ec)[6]) {
  double s = ec[5];
  s = fma(s, z, ec[4]);
  s = fma(s, z, ec[3]);
  s = fma(s, z, ec[2]);
  s = fma(s, z, ec[1]);
  s = fma(s, z, ec[0]);
  return fma(s, z, 1.0);
}

template <int LPW>
__device__ __forceinline__ double group_sum_d(double v) {
#pragma unroll
  for (int o = LPW / 2; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

template <int D, int KPL, int LPW>
__device__ __forceinline__ void precise_body(const PassParams& p) {
  using Cfg = PreciseCfg<D, KPL, LPW>;
  constexpr int NA = Cfg::NA;
  constexpr int PLEN = Cfg::PLEN;
  constexpr int WPG = Cfg::WPG;
  constexpr int TILE = Cfg::TILE;
  constexpr int RED_BYTES = NWARP * LPW * NA * 8;
  constexpr int LAST_BYTES = (PLEN + BLOCK) * 8;
  constexpr int SMEM_BYTES = RED_BYTES > LAST_BYTES ? RED_BYTES : LAST_BYTES;
  __shared__ __align__(16) unsigned char smem_raw[SMEM_BYTES];
  __shared__ int s_flag;

  const int tid = threadIdx.x;
  const int lane = tid & 31;
  const int warp = tid >> 5;
  const int gl = (LPW == 1) ? 0 : (lane % LPW);
  const int grp = tid / LPW;
  const int k = p.k;
  const int nb = p.lt.n_blocks;
  const int b = blockIdx.x;
  const int t_lo = tile_begin(b, p.lt.tiles_total, nb);
  const int t_hi = tile_begin(b + 1, p.lt.tiles_total, nb);
  if (b >= nb || t_lo >= t_hi) return;   // (the dual step kernel's grid can be larger than this pass's table)

  double c[KPL][D];
  double acc[KPL][NA];
  double ec[6];
  exp_scaled_coeffs(p.inv_tau_d, ec);
  int layer = 0;
  while (p.lt.tile_off[layer + 1] <= t_lo) ++layer;
  int cur_layer = -1;
  bool layer_active = false;

  auto flush = [&](int l) {
    double* red = reinterpret_cast<double*>(smem_raw);
#pragma unroll
    for (int t = 0; t < KPL; ++t)
#pragma unroll
      for (int a = 0; a < NA; ++a) {
        double v = acc[t][a];
#pragma unroll
        for (int o = LPW; o < 32; o <<= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        acc[t][a] = v;
      }
    double* mine = p.partials + (size_t)(b + l) * PLEN;
#pragma unroll
    for (int t = 0; t < KPL; ++t) {
      __syncthreads();
      if (lane < LPW) {
#pragma unroll
        for (int a = 0; a < NA; ++a) red[warp * (LPW * NA) + gl * NA + a] = acc[t][a];
      }
      __syncthreads();
      for (int o = tid; o < LPW * NA; o += BLOCK) {
        double s = 0.0;
#pragma unroll
        for (int wv = 0; wv < NWARP; ++wv) s += red[wv * (LPW * NA) + o];
        mine[((o / NA) * KPL + t) * NA + (o % NA)] = s;
      }
    }
    finish_layer<STEP, D, PLEN, NA>(p, l, b, smem_raw, &s_flag);
  };

  for (int tile = t_lo; tile < t_hi; ++tile) {
    while (p.lt.tile_off[layer + 1] <= tile) ++layer;
    if (layer != cur_layer) {
      if (cur_layer >= 0 && layer_active) flush(cur_layer);
      cur_layer = layer;
      layer_active = (p.st[layer].fwd_done == 0) && (p.st[layer].precise[p.iter & 1] != 0) && (p.st[layer].fwd_iters == p.iter);
      if (layer_active) {
        const float* Cl = p.C + (size_t)layer * k * D;
#pragma unroll
        for (int t = 0; t < KPL; ++t) {
          const int j = gl * KPL + t;
#pragma unroll
          for (int a = 0; a < D; ++a) c[t][a] = (j < k) ? (double)Cl[j * D + a] : 0.0;
#pragma unroll
          for (int a = 0; a < NA; ++a) acc[t][a] = 0.0;
        }
      }
    }
    if (!layer_active) continue;
    const long long row0 = p.lt.row_off[layer];
    const long long rows = p.lt.row_off[layer + 1] - row0;
    // thread-per-weight (LPW == 1): consecutive threads take consecutive rows (coalesced); otherwise a group walks
    // its own WPG consecutive rows
    const long long tb = (long long)(tile - p.lt.tile_off[layer]) * TILE;
    // all rows of the trip are fetched first (thread-per-weight layouts: 4 loads in flight per thread)
    constexpr int QB = (LPW == 1 && Cfg::MIN_BLOCKS == 1) ? WPG : 2;   // rows per fully unrolled batch
    // one body for codebooks that fill every centroid slot of the layout (no per-centroid validity tests) and one
    // for padded codebooks
    auto rows_of_tile = [&](auto full_tag) {
      constexpr bool FULL = decltype(full_tag)::value;
#pragma unroll 1
      for (int q0 = 0; q0 < WPG; q0 += QB) {
        float wf[QB][D];
        bool okq[QB];
#pragma unroll
        for (int qq = 0; qq < QB; ++qq) {
          const int q = q0 + qq;
          const long long loc = (LPW == 1) ? tb + (long long)q * BLOCK + grp : tb + (long long)grp * WPG + q;
          okq[qq] = (loc < rows);
          const long long grow = row0 + (okq[qq] ? loc : 0);
#pragma unroll
          for (int a = 0; a < D; ++a) wf[qq][a] = __ldg(p.W + grow * D + a);
        }
#pragma unroll
        for (int qq = 0; qq < QB; ++qq) {
          double w[D];
#pragma unroll
          for (int a = 0; a < D; ++a) w[a] = (double)wf[qq][a];
          double dist[KPL];
#pragma unroll
          for (int t = 0; t < KPL; ++t) {
            double sq = 0.0;
#pragma unroll
            for (int a = 0; a < D; ++a) {
              const double df = w[a] - c[t][a];
              sq = (D == 1) ? fabs(df) : fma(df, df, sq);
            }
            dist[t] = (D == 1) ? sq : sqrt(sq);
          }
          // Softmax reference: the distance to centroid 0 instead of the row minimum.  All centroids of a `precise`
          // layer lie within PRECISE_SPAN * tau of each other, so by the triangle inequality every
          // (reference - D_ij) / tau stays within +-PRECISE_SPAN, which is all exp_scaled needs.
          double ref = dist[0];
          if constexpr (LPW > 1) ref = __shfl_sync(0xffffffffu, ref, lane - gl);
          double e[KPL];
          double lsum = 0.0;
#pragma unroll
          for (int t = 0; t < KPL; ++t) {
            const double ev = exp_scaled(ref - dist[t], ec);
            e[t] = (FULL || gl * KPL + t < k) ? ev : 0.0;
            lsum += e[t];
          }
          const double gsum = group_sum_d<LPW>(lsum);
          // reciprocal of the row sum (about k): fp32 seed and two Newton steps in fp64 (error ~1e-28 relative
          // to the seed's 1e-7 squared twice), cheaper than a double division
          double r = (double)rcp_approx((float)gsum);
          r = r * (2.0 - gsum * r);
          r = r * (2.0 - gsum * r);
          if (!okq[qq]) r = 0.0;
          double rw[D];
#pragma unroll
          for (int a = 0; a < D; ++a) rw[a] = r * w[a];
#pragma unroll
          for (int t = 0; t < KPL; ++t) {
            acc[t][0] = fma(e[t], r, acc[t][0]);
#pragma unroll
            for (int a = 0; a < D; ++a) acc[t][1 + a] = fma(e[t], rw[a], acc[t][1 + a]);
          }
        }
      }
    };
    if (k == Cfg::KP) rows_of_tile(std::true_type{});
    else rows_of_tile(std::false_type{});
  }
  grid_release_dependents();
  if (cur_layer >= 0 && layer_active) flush(cur_layer);
}

template <int D, int KPL, int LPW>
__global__ void __launch_bounds__(BLOCK, PreciseCfg<D, KPL, LPW>::MIN_BLOCKS)
idkm_step_precise(const __grid_constant__ PassParams p) {
  grid_dependency_sync();
  precise_body<D, KPL, LPW>(p);
}

// ---- fp32 forward step for collapsing layers in the increment form ---------------------------------------------
// The same M-step as the STEP pass for the layers flagged `precise`, without fp64 in the row loop.  In such a layer
// every centroid lies within PRECISE_SPAN * tau of centroid 0, so with u_i = w_i - c_0 and delta_j = c_j - c_0
// (formed in fp64, rounded once):
//   D_ij^2 - D_i0^2 = |delta_j|^2 - 2 delta_j . u_i =: q_ij,      D_ij - D_i0 = q_ij / (D_ij + D_i0)
//   (d = 1: D_ij - D_i0 = |u_i - delta_j| - |u_i| = -sign(u_i) delta_j for every weight outside [c_0, c_j])
//   x_ij = -(D_ij - D_i0) / tau,  |x_ij| <= PRECISE_SPAN,   t_ij = exp(x_ij) - 1 by a fifth-degree series,
//   A_ij - 1/k = (t_ij - tbar_i) / (k (1 + tbar_i)),   tbar_i = mean_j t_ij.
// Every quantity is small and known to fp32 RELATIVE accuracy -- errors scale with delta, not with |w| -- which is
// what the fp32 STEP pass loses (its w - c_j rounds on the grid of w).  Accumulated per centroid:
// dS_j = sum_i (A_ij - 1/k) and dN_j = sum_i (A_ij - 1/k) u_i, and once per layer sum_i w_i (of the weights themselves:
// the fp32 difference w_i - c_0 rounds the same way for every weight of a binade, harmless relative to u_i in dN_j but a
// bias in a plain sum; U = sum_i w_i - m c_0 is formed in fp64); the epilogue forms
// C+_j = c_0 + (U / k + dN_j) / (m / k + dS_j) in fp64 (finish_layer with DELTA).  Sums are two-level like the STEP
// pass (fp32 per about 64 rows, then a private shared-memory slot; fp64 across blocks).
template <int D, int KPL, int LPW>
struct DeltaCfg {
  static constexpr int KP = KPL * LPW;
  static constexpr int NA = D + 1;
  static constexpr int PLENK = KP * NA;
  // after the per-centroid sums: D entries for the sum of the weights and, for scalar weights, the four sums of the
  // rows that need no per-centroid work (see delta_body)
  static constexpr int NEXTRA = (D == 1) ? 4 : 0;
  static constexpr int PLEN = PLENK + D + NEXTRA;
  static constexpr int VEC = 4 / D;                  // rows per 128-bit load (thread-per-weight layouts)
  static constexpr int UN = 4;                       // 128-bit loads in flight per thread and trip
  static constexpr int WPG = (LPW == 1) ? VEC * UN : 16;   // rows per thread (per group) and tile
  static constexpr int TILE = (BLOCK / LPW) * WPG;
  static constexpr int NSLOT = KPL * NA + D + NEXTRA;   // second-level sums per thread
  static constexpr int DYN_SMEM = BLOCK * NSLOT * 4;
  static constexpr int SPILL_TILES = (64 / WPG) > 0 ? (64 / WPG) : 1;
  static constexpr int MIN_BLOCKS = (LPW == 1 && KPL * NA <= 8) ? 4 : ((KPL * NA <= 24) ? 2 : 1);
};

// exp(x) - 1 for |x| <= PRECISE_SPAN: x + x^2 (1/2 + x (1/6 + x (1/24 + x/120))), truncation x^5 / 720 < 2e-9
// relative; five instructions
__device__ __forceinline__ float expm1_small(float x) {
  float s = fmaf(x, 1.f / 120.f, 1.f / 24.f);
  s = fmaf(s, x, 1.f / 6.f);
  s = fmaf(s, x, 0.5f);
  return fmaf(s * x, x, x);
}

template <int D, int KPL, int LPW>
__device__ __forceinline__ void delta_body(const PassParams& p) {
  using Cfg = DeltaCfg<D, KPL, LPW>;
  constexpr int NA = Cfg::NA, PLEN = Cfg::PLEN, PLENK = Cfg::PLENK, WPG = Cfg::WPG, TILE = Cfg::TILE, NSLOT = Cfg::NSLOT;
  constexpr int NEXTRA = Cfg::NEXTRA;
  constexpr int RED_BYTES = NWARP * PLEN * 4;
  constexpr int LAST_BYTES = (PLEN + BLOCK) * 8;
  constexpr int SMEM_BYTES = RED_BYTES > LAST_BYTES ? RED_BYTES : LAST_BYTES;
  __shared__ __align__(16) unsigned char smem_raw[SMEM_BYTES];
  __shared__ int s_flag;
  extern __shared__ __align__(16) float slots[];   // [NSLOT][BLOCK]

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int gl = (LPW == 1) ? 0 : (lane % LPW);
  const int grp = tid / LPW;
  const int k = p.k;
  const int nb = p.lt.n_blocks;
  const int b = blockIdx.x;
  const int t_lo = tile_begin(b, p.lt.tiles_total, nb);
  const int t_hi = tile_begin(b + 1, p.lt.tiles_total, nb);
  if (b >= nb || t_lo >= t_hi) return;

  float dl[KPL][D], dl2[KPL], c0[D];
  float acc[KPL][NA], uacc[D];
  // scalar weights: count and sum of the rows above / below all centroids (cp, sp, cm, sm), which need no
  // per-centroid work (their attention increments take two values per centroid, applied in the epilogue)
  float fx[NEXTRA > 0 ? NEXTRA : 1];
  float dmax2 = 0.f;      // twice the largest |delta_j|: rows farther than this from c_0 are outside the centroids
  (void)fx; (void)dmax2;
  bool cvalid[KPL];
  float inv_k = 0.f;
  int layer = 0;
  while (p.lt.tile_off[layer + 1] <= t_lo) ++layer;
  int cur_layer = -1;
  bool layer_active = false;
  int since_spill = 0;

  auto spill = [&]() {
#pragma unroll
    for (int t = 0; t < KPL; ++t)
#pragma unroll
      for (int a = 0; a < NA; ++a) {
        slots[(t * NA + a) * BLOCK + tid] += acc[t][a];
        acc[t][a] = 0.f;
      }
#pragma unroll
    for (int a = 0; a < D; ++a) {
      slots[(KPL * NA + a) * BLOCK + tid] += uacc[a];
      uacc[a] = 0.f;
    }
#pragma unroll
    for (int q = 0; q < NEXTRA; ++q) {
      slots[(KPL * NA + D + q) * BLOCK + tid] += fx[q];
      fx[q] = 0.f;
    }
  };

  auto flush = [&](int l) {
    float* red = reinterpret_cast<float*>(smem_raw);   // [NWARP][PLEN]
    // per-centroid sums: across the groups of a warp (lanes with equal gl); U: once per group (its lanes hold copies)
#pragma unroll
    for (int t = 0; t < KPL; ++t)
#pragma unroll
      for (int a = 0; a < NA; ++a) {
        float v = acc[t][a] + slots[(t * NA + a) * BLOCK + tid];
#pragma unroll
        for (int o = LPW; o < 32; o <<= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        acc[t][a] = v;
      }
#pragma unroll
    for (int a = 0; a < D; ++a) {
      float v = (gl == 0) ? uacc[a] + slots[(KPL * NA + a) * BLOCK + tid] : 0.f;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
      uacc[a] = v;
    }
    __syncthreads();
    if (lane < LPW) {
#pragma unroll
      for (int t = 0; t < KPL; ++t)
#pragma unroll
        for (int a = 0; a < NA; ++a) red[warp * PLEN + (gl * KPL + t) * NA + a] = acc[t][a];
    }
    float fxs[NEXTRA > 0 ? NEXTRA : 1];
    (void)fxs;
#pragma unroll
    for (int q = 0; q < NEXTRA; ++q) {
      float v = (gl == 0) ? fx[q] + slots[(KPL * NA + D + q) * BLOCK + tid] : 0.f;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
      fxs[q] = v;
    }
    if (lane == 0) {
#pragma unroll
      for (int a = 0; a < D; ++a) red[warp * PLEN + PLENK + a] = uacc[a];
#pragma unroll
      for (int q = 0; q < NEXTRA; ++q) red[warp * PLEN + PLENK + D + q] = fxs[q];
    }
    __syncthreads();
    double* mine = p.partials + (size_t)(b + l) * PLEN;
    for (int o = tid; o < PLEN; o += BLOCK) {
      double sres = 0.0;
#pragma unroll
      for (int wv = 0; wv < NWARP; ++wv) sres += (double)red[wv * PLEN + o];
      mine[o] = sres;
    }
    finish_layer<STEP, D, PLEN, NA, true>(p, l, b, smem_raw, &s_flag);
  };

  // full_tag: the codebook fills every centroid slot of the layout (no per-centroid validity tests)
  auto row = [&](const float (&w)[D], bool ok, auto full_tag) {
    constexpr bool FULL = decltype(full_tag)::value;
    float u[D];
#pragma unroll
    for (int a = 0; a < D; ++a) u[a] = w[a] - c0[a];
    float x[KPL];
    if constexpr (D == 1) {
      // |u - delta| - |u| without forming u - delta (which would round delta on the grid of u): -sign(u) delta when
      // c_0 and c_j lie on the same side of the weight, |delta| - 2 |u| when the weight lies between them
      // (with s = sign(u): -s delta + 2 max(0, s delta - |u|), branch-free)
      const float u0 = u[0], aut = fabsf(u0) * p.inv_tau;
      const float sg = copysignf(p.inv_tau, u0);           // s / tau
#pragma unroll
      for (int t = 0; t < KPL; ++t) {
        const float sd = sg * dl[t][0];                     // s delta / tau
        x[t] = fmaf(-2.f, fmaxf(sd - aut, 0.f), sd);        // -(D_ij - D_i0) / tau
      }
    } else {
      float d0sq = 0.f;
#pragma unroll
      for (int a = 0; a < D; ++a) d0sq = fmaf(u[a], u[a], d0sq);
      const float d0 = sqrt_approx(d0sq);
      float v[D];
#pragma unroll
      for (int a = 0; a < D; ++a) v[a] = -2.f * u[a];
#pragma unroll
      for (int t = 0; t < KPL; ++t) {
        float q = dl2[t];
#pragma unroll
        for (int a = 0; a < D; ++a) q = fmaf(dl[t][a], v[a], q);            // D_ij^2 - D_i0^2
        const float dij = sqrt_approx(fmaxf(d0sq + q, 0.f));
        x[t] = -q * p.inv_tau * rcp_approx(fmaxf(dij + d0, 1e-30f));
      }
    }
    float tt[KPL], lsum = 0.f;
#pragma unroll
    for (int t = 0; t < KPL; ++t) {
      tt[t] = (FULL || cvalid[t]) ? expm1_small(x[t]) : 0.f;
      lsum += tt[t];
    }
    const float tbar = group_sum<LPW>(lsum) * inv_k;
    const float r = ok ? inv_k * rcp_approx(1.f + tbar) : 0.f;
    const float ntr = -tbar * r;
#pragma unroll
    for (int t = 0; t < KPL; ++t) {
      const float aij = (FULL || cvalid[t]) ? fmaf(tt[t], r, ntr) : 0.f;    // A_ij - 1/k = (t_ij - tbar_i) r_i
      acc[t][0] += aij;
#pragma unroll
      for (int a = 0; a < D; ++a) acc[t][1 + a] = fmaf(aij, u[a], acc[t][1 + a]);
    }
#pragma unroll
    for (int a = 0; a < D; ++a) uacc[a] += ok ? w[a] : 0.f;
  };

  // Scalar weights: a row farther than dmax2 from c_0 lies outside all centroids and is only counted; the others
  // (about a fraction dmax2 / spread of the rows) take the general path, under a warp-uniform branch.
  auto row_any = [&](const float (&w)[D], bool ok, auto full_tag) {
    if constexpr (D == 1) {
      const float u0 = w[0] - c0[0];
      const bool fast = ok && (fabsf(u0) > dmax2);
      const bool pos = fast && (u0 > 0.f), neg = fast && !(u0 > 0.f);
      fx[0] += pos ? 1.f : 0.f;
      fx[1] += pos ? w[0] : 0.f;
      fx[2] += neg ? 1.f : 0.f;
      fx[3] += neg ? w[0] : 0.f;
      if (__any_sync(0xffffffffu, ok && !fast)) row(w, ok && !fast, full_tag);
    } else {
      row(w, ok, full_tag);
    }
  };

  auto load_w = [&](long long grow, float (&w)[D]) {
    if constexpr (D == 4) {
      const float4 v4 = __ldg(reinterpret_cast<const float4*>(p.W) + grow);
      w[0] = v4.x; w[1] = v4.y; w[2] = v4.z; w[3] = v4.w;
    } else if constexpr (D == 2) {
      const float2 v2 = __ldg(reinterpret_cast<const float2*>(p.W) + grow);
      w[0] = v2.x; w[1] = v2.y;
    } else {
      w[0] = __ldg(p.W + grow);
    }
  };

  for (int tile = t_lo; tile < t_hi; ++tile) {
    while (p.lt.tile_off[layer + 1] <= tile) ++layer;
    if (layer != cur_layer) {
      if (cur_layer >= 0 && layer_active) flush(cur_layer);
      cur_layer = layer;
      layer_active = (p.st[layer].fwd_done == 0) && (p.st[layer].precise[p.iter & 1] != 0) && (p.st[layer].fwd_iters == p.iter);
      if (layer_active) {
        const float* Cl = p.C + (size_t)layer * k * D;
        inv_k = 1.f / (float)k;
#pragma unroll
        for (int a = 0; a < D; ++a) {
          c0[a] = Cl[a];
          uacc[a] = 0.f;
          slots[(KPL * NA + a) * BLOCK + tid] = 0.f;
        }
        if constexpr (D == 1) {
          float dm = 0.f;
          for (int j = 1; j < k; ++j) dm = fmaxf(dm, fabsf(Cl[j] - c0[0]));
          dmax2 = 2.f * dm;
#pragma unroll
          for (int q = 0; q < NEXTRA; ++q) {
            fx[q] = 0.f;
            slots[(KPL * NA + D + q) * BLOCK + tid] = 0.f;
          }
        }
#pragma unroll
        for (int t = 0; t < KPL; ++t) {
          const int j = gl * KPL + t;
          cvalid[t] = (j < k);
          double d2 = 0.0;
#pragma unroll
          for (int a = 0; a < D; ++a) {
            const double dd = cvalid[t] ? (double)Cl[j * D + a] - (double)c0[a] : 0.0;
            dl[t][a] = (float)dd;
            d2 += dd * dd;
          }
          dl2[t] = (float)d2;
#pragma unroll
          for (int a = 0; a < NA; ++a) {
            acc[t][a] = 0.f;
            slots[(t * NA + a) * BLOCK + tid] = 0.f;
          }
        }
        since_spill = 0;
      }
    }
    if (!layer_active) continue;
    const long long row0 = p.lt.row_off[layer];
    const long long rows = p.lt.row_off[layer + 1] - row0;
    const long long tb = (long long)(tile - p.lt.tile_off[layer]) * TILE;
    const bool full = (k == Cfg::KP);
    if constexpr (LPW == 1) {
      // thread-per-weight: a thread takes VEC consecutive rows per 128-bit load, UN loads per trip, all issued first
      constexpr int VEC = Cfg::VEC, UN = Cfg::UN;
      const bool vec_ok = ((row0 * D) % 4 == 0);
      // a run of whole tiles inside the layer: one inner loop with a running pointer, the next tile's loads issued
      // before the current tile's arithmetic (as in the fp32 forward step)
      {
        const int lim_r = (t_hi < p.lt.tile_off[layer + 1]) ? t_hi : p.lt.tile_off[layer + 1];
        const long long by_rows = (rows - tb) / TILE;
        const int by_tiles = lim_r - tile;
        const int nfull = vec_ok ? (by_rows < (long long)by_tiles ? (int)by_rows : by_tiles) : 0;
        if (nfull > 0) {
          auto run = [&](auto full_tag) {
            const float4* wp = reinterpret_cast<const float4*>(p.W + (row0 + tb) * D) + tid;
            float4 cur[UN], nxt[UN];
#pragma unroll
            for (int un = 0; un < UN; ++un) nxt[un] = cur[un] = __ldg(wp + un * BLOCK);
#pragma unroll 1
            for (int s2 = 0; s2 < nfull; ++s2) {
              wp += UN * BLOCK;
              if (s2 + 1 < nfull) {
#pragma unroll
                for (int un = 0; un < UN; ++un) nxt[un] = __ldg(wp + un * BLOCK);
              }
#pragma unroll
              for (int un = 0; un < UN; ++un) {
                const float xs[4] = {cur[un].x, cur[un].y, cur[un].z, cur[un].w};
#pragma unroll
                for (int v = 0; v < VEC; ++v) {
                  float w1[D];
#pragma unroll
                  for (int a = 0; a < D; ++a) w1[a] = xs[v * D + a];
                  row_any(w1, true, full_tag);
                }
              }
              if (++since_spill >= Cfg::SPILL_TILES) {
                spill();
                since_spill = 0;
              }
#pragma unroll
              for (int un = 0; un < UN; ++un) cur[un] = nxt[un];
            }
          };
          if (full) run(std::true_type{});
          else run(std::false_type{});
          tile += nfull - 1;
          continue;
        }
      }
      float wv[UN][VEC][D];
      int nv[UN];                       // rows of each load that exist (32-bit: the row loop compares against it)
#pragma unroll
      for (int un = 0; un < UN; ++un) {
        const long long loc = tb + (long long)(un * BLOCK + tid) * VEC;
        const long long left = rows - loc;
        nv[un] = left >= VEC ? VEC : (left > 0 ? (int)left : 0);
        const long long grow = row0 + loc;
        if (vec_ok && loc + VEC <= rows) {
          const float4 x4 = __ldg(reinterpret_cast<const float4*>(p.W + grow * D));
          const float xs[4] = {x4.x, x4.y, x4.z, x4.w};
#pragma unroll
          for (int v = 0; v < VEC; ++v)
#pragma unroll
            for (int a = 0; a < D; ++a) wv[un][v][a] = xs[v * D + a];
        } else {
#pragma unroll
          for (int v = 0; v < VEC; ++v)
#pragma unroll
            for (int a = 0; a < D; ++a) wv[un][v][a] = (loc + v < rows) ? __ldg(p.W + (grow + v) * D + a) : 0.f;
        }
      }
      if (full) {
#pragma unroll
        for (int un = 0; un < UN; ++un)
#pragma unroll
          for (int v = 0; v < VEC; ++v) row_any(wv[un][v], v < nv[un], std::true_type{});
      } else {
#pragma unroll
        for (int un = 0; un < UN; ++un)
#pragma unroll
          for (int v = 0; v < VEC; ++v) row_any(wv[un][v], v < nv[un], std::false_type{});
      }
    } else {
      // group-per-weight: a group walks its own WPG consecutive rows, two fetched ahead
      const long long gb = tb + (long long)grp * WPG;
#pragma unroll 1
      for (int q0 = 0; q0 < WPG; q0 += 2) {
        float wv[2][D];
        bool okq[2];
#pragma unroll
        for (int qq = 0; qq < 2; ++qq) {
          const long long loc = gb + q0 + qq;
          okq[qq] = (loc < rows);
          load_w(row0 + (okq[qq] ? loc : 0), wv[qq]);
        }
        if (full) {
#pragma unroll
          for (int qq = 0; qq < 2; ++qq) row_any(wv[qq], okq[qq], std::true_type{});
        } else {
#pragma unroll
          for (int qq = 0; qq < 2; ++qq) row_any(wv[qq], okq[qq], std::false_type{});
        }
      }
    }
    if (++since_spill >= Cfg::SPILL_TILES) {
      spill();
      since_spill = 0;
    }
  }
  grid_release_dependents();
  if (cur_layer >= 0 && layer_active) flush(cur_layer);
}

template <int D, int KPL, int LPW>
__global__ void __launch_bounds__(BLOCK, DeltaCfg<D, KPL, LPW>::MIN_BLOCKS)
idkm_step_delta(const __grid_constant__ PassParams p) {
  grid_dependency_sync();
  delta_body<D, KPL, LPW>(p);
}

// One launch per forward iteration instead of two, for the smallest thread-per-weight layouts, where the fp32 and
// the fp64 step have the same register budget: every block first takes its tiles of the layers that step in fp32,
// then its tiles of the layers that step in fp64 (own tile table, own partial-sum buffers: the two run side by side
// across blocks).  On a batched workload with collapsing layers the two kinds of layers then overlap instead of
// running one kernel after the other.
struct DualParams {
  PassParams p;   // fp32 step
  PassParams q;   // fp64 step
};
// DELTA: the collapsing layers step in the fp32 increment form (delta_body) instead of fp64 (precise_body).
template <int D, int KPL, bool DELTA>
__global__ void __launch_bounds__(BLOCK, PreciseCfg<D, KPL, 1>::MIN_BLOCKS)
idkm_step_dual(const __grid_constant__ DualParams dp) {
  grid_dependency_sync();
  pass_body<STEP, D, KPL, 1, false>(dp.p);
  __syncthreads();
  if constexpr (DELTA) delta_body<D, KPL, 1>(dp.q);
  else precise_body<D, KPL, 1>(dp.q);
}



// Exact solve of (I - J^T) u = g -- the linear system behind M* = (I - dF/dC)^-1 of Section 4.2, contracted with g --
// by ONE warp: the matrix J (n x n, row stride ld, fp64, shared memory) is turned into I - J^T in place, then Gaussian
// elimination with partial pivoting and back substitution.  b holds g on entry and u on exit.  Lanes take columns
// (consecutive addresses: no bank conflicts), rows run in a loop.  Returns false when a pivot vanishes or is not a
// number (J has an eigenvalue 1 to working precision, or the sums were not finite).  n <= 64.
__device__ __forceinline__ bool warp_solve_adjoint(double* J, int ld, double* b, int n, int lane) {
  for (int idx = lane; idx < n * n; idx += 32) {
    const int r = idx / n, c = idx % n;
    if (r < c) {
      const double x = J[r * ld + c], y = J[c * ld + r];
      J[r * ld + c] = -y;
      J[c * ld + r] = -x;
    } else if (r == c) {
      J[r * ld + r] = 1.0 - J[r * ld + r];
    }
  }
  __syncwarp();
  bool ok = true;
  for (int c = 0; c < n; ++c) {
    double best = -1.0;
    int br = c;
    for (int r = c + lane; r < n; r += 32) {
      const double v = fabs(J[r * ld + c]);
      if (v > best) {
        best = v;
        br = r;
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const double ob = __shfl_xor_sync(0xffffffffu, best, o);
      const int orow = __shfl_xor_sync(0xffffffffu, br, o);
      if (ob > best || (ob == best && orow < br)) {
        best = ob;
        br = orow;
      }
    }
    if (!(best > 0.0) || !(best < 1e300)) {
      ok = false;
      break;
    }
    if (br != c) {
      for (int q = lane; q < n; q += 32) {
        const double x = J[c * ld + q];
        J[c * ld + q] = J[br * ld + q];
        J[br * ld + q] = x;
      }
      if (lane == 0) {
        const double x = b[c];
        b[c] = b[br];
        b[br] = x;
      }
    }
    __syncwarp();
    const double inv_piv = 1.0 / J[c * ld + c];
    const double bc = b[c];
    for (int r = c + 1; r < n; ++r) {
      const double f = J[r * ld + c] * inv_piv;
      for (int q = c + 1 + lane; q < n; q += 32) J[r * ld + q] = fma(-f, J[c * ld + q], J[r * ld + q]);
      if (lane == 0) b[r] = fma(-f, bc, b[r]);
    }
    __syncwarp();
  }
  if (!ok) return false;
  for (int r = n - 1; r >= 0; --r) {
    double sres = 0.0;
    for (int q = r + 1 + lane; q < n; q += 32) sres = fma(J[r * ld + q], b[q], sres);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sres += __shfl_xor_sync(0xffffffffu, sres, o);
    if (lane == 0) b[r] = (b[r] - sres) / J[r * ld + r];
    __syncwarp();
  }
  return true;
}

// ---- explicit Jacobian for small codebooks -------------------------------------------------------------------
// When k d <= 8 the matrix J_C = dF/dC (k d x k d, at most 64 entries) fits in a thread's registers.  One pass over
// W accumulates it -- J[(j,a),(l,b)] = sum_i P_ija (delta_jl - A_il) n_ilb with P_ija = A_ij (w_ia - F_ja) / (S_j tau)
// -- and the last block then runs the WHOLE adjoint iteration u <- alpha (J^T u + g) + (1 - alpha) u on that small
// matrix in fp64: the same iterates as one fused pass over W per step, for the cost of one pass.  This is the paper's
// own formulation (it iterates a k x k matrix, Section 4.2) restricted to where the matrix is cheap to form.
template <int D, int KPL>
struct JacCfg {
  static constexpr int KD = KPL * D;
  static constexpr int PLEN = KD * KD;
  static constexpr int VEC = 4 / D;
  static constexpr int TILE = BLOCK * VEC;
};

template <int D, int KPL>
__global__ void __launch_bounds__(BLOCK) idkm_jacobian(const __grid_constant__ PassParams p) {
  using Cfg = JacCfg<D, KPL>;
  constexpr int KD = Cfg::KD;
  constexpr int PLEN = Cfg::PLEN;
  constexpr int VEC = Cfg::VEC;
  constexpr int TILE = Cfg::TILE;
  constexpr int SMEM_DBL = (NWARP * PLEN > PLEN + BLOCK) ? NWARP * PLEN : PLEN + BLOCK;
  __shared__ double sm[SMEM_DBL];
  __shared__ int s_flag;

  grid_dependency_sync();
  const int tid = threadIdx.x;
  const int lane = tid & 31;
  const int warp = tid >> 5;
  const int k = p.k;
  const int nb = p.lt.n_blocks;
  const int b = blockIdx.x;
  const int t_lo = tile_begin(b, p.lt.tiles_total, nb);
  const int t_hi = tile_begin(b + 1, p.lt.tiles_total, nb);
  if (b >= nb || t_lo >= t_hi) return;   // (the dual step kernel's grid can be larger than this pass's table)

  float c[KPL][D], fj[KPL][D], ist[KPL];   // centroids, F(C_T, W)_j, 1 / (S_j tau) (0 for a dead or padding cluster)
  float jac[KD][KD];
  float jac_hi[KD][KD];                     // second level: the running sums are moved here every 64 rows
  int layer = 0;
  while (p.lt.tile_off[layer + 1] <= t_lo) ++layer;
  int cur_layer = -1;
  bool layer_active = false;
  int since = 0;

  auto finish = [&](int l) {
#pragma unroll
    for (int r = 0; r < KD; ++r)
#pragma unroll
      for (int q = 0; q < KD; ++q) {
        double v = (double)jac_hi[r][q] + (double)jac[r][q];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if (lane == 0) sm[warp * PLEN + r * KD + q] = v;
      }
    __syncthreads();
    double* mine = p.partials + (size_t)(b + l) * PLEN;
    for (int o = tid; o < PLEN; o += BLOCK) {
      double s = 0.0;
#pragma unroll
      for (int wv = 0; wv < NWARP; ++wv) s += sm[wv * PLEN + o];
      mine[o] = s;
    }
    __threadfence();
    __syncthreads();
    const int first_b = block_of_tile(p.lt.tile_off[l], p.lt.tiles_total, nb);
    const int last_b = block_of_tile(p.lt.tile_off[l + 1] - 1, p.lt.tiles_total, nb);
    const int n_contrib = last_b - first_b + 1;
    if (tid == 0) {
      const unsigned int prev = atomicAdd(&p.st[l].ticket, 1u);
      s_flag = (prev == (unsigned int)(n_contrib - 1));
    }
    __syncthreads();
    if (!s_flag) return;
    __threadfence();
    // second level in slot order: PLEN <= 64 outputs, BLOCK / PLEN strided chunks each, then the chunks in order
    double* tot = sm;            // [PLEN]
    double* scratch = sm + PLEN; // [BLOCK]
    const double* base = p.partials + (size_t)(first_b + l) * PLEN;
    constexpr int NCH = BLOCK / PLEN;
    {
      const int ch = tid / PLEN, o = tid % PLEN;
      double s = 0.0;
      if (ch < NCH)
        for (int q = ch; q < n_contrib; q += NCH) s += __ldcg(base + (size_t)q * PLEN + o);
      __syncthreads();
      scratch[tid] = s;
      __syncthreads();
      if (tid < PLEN) {
        double r2 = 0.0;
        for (int c2 = 0; c2 < NCH; ++c2) r2 += scratch[c2 * PLEN + tid];
        tot[tid] = r2;
      }
      __syncthreads();
    }
    if (warp == 0 && p.max_iter < 0) {
      // exact solve instead of the iteration (idkm_set_adjoint_method(ctx, 2))
      LayerState* st = p.st + l;
      const int n = k * D;
      if (lane < n) scratch[lane] = (double)p.gvec[(size_t)l * n + lane];
      __syncwarp();
      const bool ok = warp_solve_adjoint(tot, KD, scratch, n, lane);
      bool finite = true;
      if (lane < n) {
        const double uv = ok ? scratch[lane] : 0.0;
        finite = (uv == uv) && fabs(uv) < 1e300;
        p.u[(size_t)l * n + lane] = (float)uv;
      }
      finite = __all_sync(0xffffffffu, finite);
      if (lane == 0) {
        st->ticket = 0u;
        st->adj_iters = 0;
        st->adj_res = 0.f;
        st->adj_done = 1;
        if (!ok || !finite) st->status = ST_DIVERGED;
      }
    } else if (warp == 0) {
      // The iteration on the small matrix, by one warp: lane q < n owns coordinate q of u and column q of J
      // (J^T u)_q = sum_r J[r][q] u_r; u_r is fetched from lane r by a shuffle.  All lanes see the same residual.
      LayerState* st = p.st + l;
      const int n = k * D;
      const int q = lane;
      double jcol[KD];
#pragma unroll
      for (int r = 0; r < KD; ++r) jcol[r] = (q < n && r < n) ? tot[r * KD + q] : 0.0;
      const double g = (q < n) ? (double)p.gvec[(size_t)l * n + q] : 0.0;
      double u = g;
      const double al = (double)p.alpha;
      int it = 0, up = 0, status = st->status, done = 0;
      float res = 0.f, prev = 3.0e38f;
      double g2 = g * g;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) g2 += __shfl_xor_sync(0xffffffffu, g2, o);
      const double u2_limit = ADJ_GROWTH_LIMIT * ADJ_GROWTH_LIMIT * g2;
      while (it < p.max_iter && !done) {
        double s = 0.0;
#pragma unroll
        for (int r = 0; r < KD; ++r) s = fma(jcol[r], __shfl_sync(0xffffffffu, u, r), s);
        const double un = (q < n) ? al * (s + g) + (1.0 - al) * u : 0.0;
        double num = (un - u) * (un - u), den = un * un;
        double badv = (!(un == un) || fabs(un) > 1e300) ? 1.0 : 0.0;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          num += __shfl_xor_sync(0xffffffffu, num, o);
          den += __shfl_xor_sync(0xffffffffu, den, o);
          badv += __shfl_xor_sync(0xffffffffu, badv, o);
        }
        u = un;
        double dn = sqrt(den);
        if (dn < 1e-300) dn = 1e-300;
        res = (float)(sqrt(num) / dn);
        ++it;
        if (lane == 0 && it <= HIST_CAP) p.hist_adj[(size_t)l * HIST_CAP + it - 1] = res;
        up = (res > prev) ? up + 1 : 0;
        prev = res;
        if (badv > 0.0 || up >= 10 || den > u2_limit) {
          status = ST_DIVERGED;
          done = 1;
        } else if (p.tol > 0.f && res < p.tol) {
          done = 1;
        } else if (p.tol > 0.f && it >= p.max_iter && status == ST_OK) {
          status = ST_MAXITER;
        }
      }
      if (q < n) p.u[(size_t)l * n + q] = (float)u;
      if (lane == 0) {
        st->ticket = 0u;
        st->adj_iters = it;
        st->adj_res = res;
        st->adj_up = up;
        st->adj_prev = prev;
        st->adj_done = 1;
        st->status = status;
      }
    }
    __syncthreads();
  };

  for (int tile = t_lo; tile < t_hi; ++tile) {
    while (p.lt.tile_off[layer + 1] <= tile) ++layer;
    if (layer != cur_layer) {
      if (cur_layer >= 0 && layer_active) finish(cur_layer);
      cur_layer = layer;
      layer_active = (p.st[layer].adj_done == 0);
      since = 0;
      if (layer_active) {
#pragma unroll
        for (int t = 0; t < KPL; ++t) {
          const float s = (t < k) ? p.S[(size_t)layer * k + t] : 0.f;
          ist[t] = (t < k && s >= S_MIN_F) ? p.inv_tau / s : 0.f;
#pragma unroll
          for (int a = 0; a < D; ++a) {
            c[t][a] = (t < k) ? p.C[((size_t)layer * k + t) * D + a] : PAD_COORD;
            fj[t][a] = (t < k) ? p.F[((size_t)layer * k + t) * D + a] : 0.f;
          }
        }
#pragma unroll
        for (int r = 0; r < KD; ++r)
#pragma unroll
          for (int q = 0; q < KD; ++q) {
            jac[r][q] = 0.f;
            jac_hi[r][q] = 0.f;
          }
      }
    }
    if (!layer_active) continue;
    const long long row0 = p.lt.row_off[layer];
    const long long rows = p.lt.row_off[layer + 1] - row0;
    const long long loc0 = (long long)(tile - p.lt.tile_off[layer]) * TILE + (long long)tid * VEC;
    const bool vec_ok = ((row0 * D) % 4 == 0) && (loc0 + VEC <= rows);
    float wv[VEC][D];
    if (vec_ok) {
      const float4 x = __ldg(reinterpret_cast<const float4*>(p.W + (row0 + loc0) * D));
      const float xs[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
      for (int v = 0; v < VEC; ++v)
#pragma unroll
        for (int a = 0; a < D; ++a) wv[v][a] = xs[v * D + a];
    } else {
#pragma unroll
      for (int v = 0; v < VEC; ++v)
#pragma unroll
        for (int a = 0; a < D; ++a) wv[v][a] = (loc0 + v < rows) ? __ldg(p.W + (row0 + loc0 + v) * D + a) : 0.f;
    }
#pragma unroll
    for (int v = 0; v < VEC; ++v) {
      const bool valid = (loc0 + v < rows);
      float dist[KPL], rs[KPL], e[KPL];
      (void)rs;
#pragma unroll
      for (int t = 0; t < KPL; ++t) {
        if constexpr (D == 1) {
          dist[t] = fabsf(wv[v][0] - c[t][0]);
        } else {
          float sq = 1e-30f;
#pragma unroll
          for (int a = 0; a < D; ++a) {
            const float df = wv[v][a] - c[t][a];
            sq = fmaf(df, df, sq);
          }
          rs[t] = rsqrt_approx(sq);
          dist[t] = sq * rs[t];
        }
      }
      const float mref = tree_reduce<KPL, 1>(dist) * p.scale;
#pragma unroll
      for (int t = 0; t < KPL; ++t) e[t] = ex2_approx(fmaf(-p.scale, dist[t], mref));
      const float r = valid ? rcp_approx(tree_reduce<KPL, 0>(e)) : 0.f;
      float P[KD], Y[KD], Q[KD];
#pragma unroll
      for (int t = 0; t < KPL; ++t) {
        const float at = e[t] * r;
#pragma unroll
        for (int a = 0; a < D; ++a) {
          const float df = wv[v][a] - c[t][a];
          float n;
          if constexpr (D == 1) n = (df > 0.f) ? 1.f : ((df < 0.f) ? -1.f : 0.f);
          else n = df * rs[t];
          Q[t * D + a] = n;
          Y[t * D + a] = at * n;
          P[t * D + a] = at * ist[t] * (wv[v][a] - fj[t][a]);
        }
      }
#pragma unroll
      for (int rr = 0; rr < KD; ++rr)
#pragma unroll
        for (int q = 0; q < KD; ++q) {
          jac[rr][q] = fmaf(-P[rr], Y[q], jac[rr][q]);
          if (rr / D == q / D) jac[rr][q] = fmaf(P[rr], Q[q], jac[rr][q]);   // the delta_jl block
        }
    }
    since += VEC;
    if (since >= 64) {
#pragma unroll
      for (int rr = 0; rr < KD; ++rr)
#pragma unroll
        for (int q = 0; q < KD; ++q) {
          jac_hi[rr][q] += jac[rr][q];
          jac[rr][q] = 0.f;
        }
      since = 0;
    }
  }
  grid_release_dependents();
  if (cur_layer >= 0 && layer_active) finish(cur_layer);
}

// host-side dispatch (defined in the per-mode instantiation units)
typedef cudaError_t (*LaunchFn)(const PassParams& p, int grid, cudaStream_t stream);
struct KernelEntry {
  LaunchFn launch;
  const void* func;
  int kpl, lpw, tile, plen;
  int dyn_smem;   // dynamic shared memory the launch asks for (bytes)
};
// dual step kernel (idkm_pass_step_dual.cu): exists where PreciseCfg<D, KPL, 1>::MIN_BLOCKS == 4
typedef cudaError_t (*DualLaunchFn)(const DualParams& dp, int grid, cudaStream_t stream);
struct DualEntry {
  DualLaunchFn launch;
  const void* func;
  int dyn_smem;
};
// Single-launch forward loop for small layers (idkm_small_loop.cu): k <= 2, 4, 8, 16 centroids per thread.
struct SmallLoopParams {
  const float* W;
  int n_layers;
  long long row_off[MAX_LAYERS + 1];   // first row of each layer
  int blk_first[MAX_LAYERS + 1];       // first block of each layer; blk_first[n_layers] = grid size
  float* C;              // [L][k][d]: starting centroids in, returned centroids out
  LayerState* st;        // [L] layer states: `precise` is read at the start, the outcome written at the end
  double* partials;      // [2][grid][k_pad (d+1) + d] fp64 block partials, alternating by iteration
  unsigned int* sync;    // [0] barrier arrivals (only grows), [1] error word; both zero before the launch
  int k;
  float scale;           // log2(e) / tau
  float tol;
  double inv_tau_d;
  int max_iter;
  float* hist;           // [L][HIST_CAP] residual histories
  int chunked;           // 1: some thread has more than 32 rows, fp32 sums are moved out every 32 rows
  int missing_arrivals;  // 0 in production.  Host-side fault injection for the timeout path: the barriers wait for
                         // this many arrivals more than the grid has, so every wait runs out (see idkm.h)
  long long spin_limit;  // clock64() ticks a block waits at a barrier before it gives up
};
typedef cudaError_t (*SmallLaunchFn)(const SmallLoopParams& sp, int grid, cudaStream_t stream);
struct SmallLoopEntry {
  SmallLaunchFn launch;
  const void* func;
  int kpl, plen, dyn_smem;
};
constexpr int N_SMALL_FAMILY = 4;
// family index f: 0..7 -> supports k <= kpl*lpw
constexpr int N_FAMILY = 11;
constexpr int FAM_WIDE = 8;    // the alternative layout for the largest codebooks (see the tables in idkm_inst.cuh)
constexpr int FAM_4x4 = 9;     // 4 centroids per lane on 4 lanes, 8 centroids per lane on 2 lanes: group layouts for
constexpr int FAM_8x2 = 10;    // 16 centroids, picked by rule (pick_family), never by the first-fit search
const KernelEntry* kernel_entry(int mode, int d, int family);
int pick_family(int mode, int d, int k);

}  // namespace idkm
