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
#include <cuda_runtime.h>
#include <stdint.h>

namespace idkm {

constexpr int BLOCK = 256;
constexpr int NWARP = BLOCK / 32;
constexpr int MAX_LAYERS = 64;
constexpr float PAD_COORD = 1e18f;   // coordinate of a padding centroid: exp underflows to exactly 0
constexpr double S_MIN = 1e-20;      // column sums below this mark a dead cluster
constexpr float S_MIN_F = 1e-20f;
constexpr int MAX_BLOCKS_PER_SM = 8;
// When the bounding box of a layer's centroids is smaller than PRECISE_SPAN * tau, all softmax logits of a
// weight differ by less than PRECISE_SPAN and the centroid update is decided by attention differences far below
// fp32 resolution (w - c_j rounds away the differences between the c_j).  Such layers step in fp64.
constexpr double PRECISE_SPAN = 0.0625;

enum Mode { STEP = 0, FINAL = 1, GRAD = 2, ADJ = 3, SCATTER = 4, STEP_PRECISE = 5 };
constexpr int N_MODES = 6;

// status values mirrored from idkm.h (device side needs only these)
constexpr int ST_OK = 0, ST_MAXITER = 1, ST_NONFINITE = -9, ST_DIVERGED = -10;

struct LayerState {   // 64 bytes, one per layer, in the workspace
  int fwd_done, fwd_iters;
  float fwd_res;
  int dead;
  int adj_done, adj_iters;
  float adj_res;
  int status;
  unsigned int ticket;
  int adj_up;        // consecutive adjoint steps whose residual grew
  float adj_prev;
  int precise;       // 1: the layer's centroids lie within PRECISE_SPAN * tau of each other (collapsing); the
                     // forward step then runs in the fp64 kernel
  int pad[4];
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
  float* Wq;          // FINAL (may be null)
  float* A;           // FINAL (may be null)
  float* dW;          // SCATTER
  float* C;           // [L][k][d] centroids, updated in place by STEP
  float* S;           // [L][k]   column sums at the returned centroids (FINAL writes)
  float* F;           // [L][k][d] F(C_T, W) (FINAL writes)
  float* gvec;        // [L][k][d] direct codebook gradient (GRAD writes)
  float* u;           // [L][k][d] adjoint (GRAD initialises, ADJ updates)
  double* partials;   // [(n_blocks + L)][PLEN]
  LayerState* st;
  float inv_tau;      // 1 / tau
  float scale;        // log2(e) / tau
  float tol;          // stop tolerance of the loop this pass belongs to
  float alpha;        // averaging weight of the adjoint iteration
  double inv_tau_d;   // 1 / tau in double (fp64 step)
  int k;
  int max_iter;       // iteration cap of the loop (for the advisory status)
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
  static constexpr int UNROLL = (LPW == 1) ? ((KPL * D >= 32) ? 1 : 2) : 1;
  static constexpr int WPG = (LPW == 1) ? VEC * UNROLL : 16;      // weight-vectors per group per tile
  static constexpr int TILE = GROUPS * WPG;
};

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

template <int LPW>
__device__ __forceinline__ float group_sum(float v) {
#pragma unroll
  for (int o = LPW / 2; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
template <int LPW>
__device__ __forceinline__ float group_min(float v) {
#pragma unroll
  for (int o = LPW / 2; o > 0; o >>= 1) v = fminf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
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

// After a block has written its partial of layer l: take a ticket; the last contributing block adds the
// layer's partials in slot order (fp64) and applies the epilogue of the pass.  Called by all threads of the block.
// smem_raw must hold (PLEN + BLOCK) doubles.
template <int MODE, int D, int PLEN, int NA>
__device__ __forceinline__ void finish_layer(const PassParams& p, int l, int b, unsigned char* smem_raw, int* s_flag) {
  const int tid = threadIdx.x;
  const int k = p.k;
  const int nb = p.lt.n_blocks;
  __threadfence();
  __syncthreads();
  // ticket: the last contributing block of this layer reduces all of the layer's partials
  const int first_b = block_of_tile(p.lt.tile_off[l], p.lt.tiles_total, nb);
  const int last_b = block_of_tile(p.lt.tile_off[l + 1] - 1, p.lt.tiles_total, nb);
  const int n_contrib = last_b - first_b + 1;
  if (tid == 0) {
    const unsigned int prev = atomicAdd(&p.st[l].ticket, 1u);
    *s_flag = (prev == (unsigned int)(n_contrib - 1));
  }
  __syncthreads();
  if (!*s_flag) return;
  __threadfence();
  double* tot = reinterpret_cast<double*>(smem_raw);   // [PLEN]
  double* scratch = tot + PLEN;                          // [BLOCK]
  const double* base = p.partials + (size_t)(first_b + l) * PLEN;
  if constexpr (PLEN >= BLOCK) {
    for (int o = tid; o < PLEN; o += BLOCK) {
      double s = 0.0;
      for (int q = 0; q < n_contrib; ++q) s += __ldcg(base + (size_t)q * PLEN + o);
      tot[o] = s;
    }
    __syncthreads();
  } else {
    constexpr int NCH = BLOCK / PLEN;   // PLEN is a power of two times (d+1); BLOCK % PLEN may be nonzero
    const int ch = tid / PLEN, o = tid % PLEN;
    double s = 0.0;
    if (ch < NCH)
      for (int q = ch; q < n_contrib; q += NCH) s += __ldcg(base + (size_t)q * PLEN + o);
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
    for (int j = tid; j < k; j += BLOCK) {
      const double s = tot[j * NA];
      const bool alive = (s >= S_MIN);
      if (!alive) dead += 1.0;
      if (!(s == s) || s > 1e300) bad += 1.0;
#pragma unroll
      for (int a = 0; a < D; ++a) {
        const double cold = (double)Cl[j * D + a];
        const double cnew = alive ? tot[j * NA + 1 + a] / s : cold;
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
  bad = block_sum_double(bad, scratch);
  if constexpr (MODE == STEP || MODE == ADJ) {
    num = block_sum_double(num, scratch);
    den = block_sum_double(den, scratch);
  }
  double box2 = 0.0;
  if constexpr (MODE == STEP) {
    dead = block_sum_double(dead, scratch);
#pragma unroll
    for (int a = 0; a < D; ++a) {
      const double lo = block_reduce_double<1>(cmin[a], scratch);
      const double hi = block_reduce_double<2>(cmax[a], scratch);
      box2 += (hi - lo) * (hi - lo);
    }
  }
  if (tid == 0) {
    st->ticket = 0u;
    if constexpr (MODE == STEP) {
      st->precise = (sqrt(box2) * p.inv_tau_d <= PRECISE_SPAN) ? 1 : 0;
      double dn = sqrt(den);
      if (dn < 1e-300) dn = 1e-300;
      const float res = (float)(sqrt(num) / dn);
      const int it = st->fwd_iters + 1;
      st->fwd_iters = it;
      st->fwd_res = res;
      st->dead = (int)dead;
      if (bad > 0.0) {
        st->status = ST_NONFINITE;
        st->fwd_done = 1;
      } else if (p.tol > 0.f && res < p.tol) {
        st->fwd_done = 1;
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
      if (bad > 0.0) st->status = ST_NONFINITE;
      else if (st->status == ST_DIVERGED) st->status = ST_OK;
    } else if constexpr (MODE == ADJ) {
      double dn = sqrt(den);
      if (dn < 1e-300) dn = 1e-300;
      const float res = (float)(sqrt(num) / dn);
      const int it = st->adj_iters + 1;
      st->adj_iters = it;
      st->adj_res = res;
      const int up = (res > st->adj_prev) ? st->adj_up + 1 : 0;
      st->adj_up = up;
      st->adj_prev = res;
      if (bad > 0.0 || up >= 10) {
        st->status = ST_DIVERGED;
        st->adj_done = 1;
      } else if (p.tol > 0.f && res < p.tol) {
        st->adj_done = 1;
      } else if (p.tol > 0.f && it >= p.max_iter && st->status == ST_OK) {
        st->status = ST_MAXITER;
      }
    }
  }
  __syncthreads();
}

// ---- the pass ------------------------------------------------------------------------------------
template <int MODE, int D, int KPL, int LPW>
__global__ void __launch_bounds__(BLOCK) idkm_pass(const __grid_constant__ PassParams p) {
  using Cfg = PassCfg<MODE, D, KPL, LPW>;
  constexpr int KP = Cfg::KP;
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

  // shared: cross-warp reduction buffer (floats), reused by the last block as fp64 scratch
  constexpr int RED_BYTES = ACCUM ? NWARP * PLEN * 4 : 16;
  constexpr int LAST_BYTES = ACCUM ? (PLEN + BLOCK) * 8 : 16;
  constexpr int SMEM_BYTES = RED_BYTES > LAST_BYTES ? RED_BYTES : LAST_BYTES;
  __shared__ __align__(16) unsigned char smem_raw[SMEM_BYTES];
  __shared__ int s_flag;

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
  if (t_lo >= t_hi) return;

  float c[KPL][D];                 // owned centroids
  float fj[NEED_U ? KPL : 1][D];   // F(C_T, W)_j
  float us[NEED_U ? KPL : 1][D];   // u_j / S_j (0 for a dead cluster)
  float acc[ACCUM ? KPL : 1][NA];
  (void)fj; (void)us; (void)acc;

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
      for (int a = 0; a < D; ++a) c[t][a] = (j < k) ? Cl[j * D + a] : PAD_COORD;
      if constexpr (NEED_U) {
        const float s = (j < k) ? p.S[(size_t)l * k + j] : 0.f;
        const float inv = (s >= S_MIN_F) ? 1.f / s : 0.f;
#pragma unroll
        for (int a = 0; a < D; ++a) {
          fj[t][a] = (j < k) ? p.F[((size_t)l * k + j) * D + a] : 0.f;
          us[t][a] = (j < k) ? p.u[((size_t)l * k + j) * D + a] * inv : 0.f;
        }
      }
      if constexpr (ACCUM) {
#pragma unroll
        for (int a = 0; a < NA; ++a) acc[t][a] = 0.f;
      }
    }
  };

  // ---- per weight-vector work: returns through the accumulators / writes row outputs ----------
  auto process = [&](const float (&w)[D], const float (&gi)[D], bool valid, long long row, float (&out)[D]) {
    float dist[KPL];
    float rs[(D > 1 && !FWD) ? KPL : 1];
    (void)rs;
    float lmin = 3.0e38f;
#pragma unroll
    for (int t = 0; t < KPL; ++t) {
      if constexpr (D == 1) {
        dist[t] = fabsf(w[0] - c[t][0]);
      } else {
        float sq = 0.f;
#pragma unroll
        for (int a = 0; a < D; ++a) {
          const float df = w[a] - c[t][a];
          sq = fmaf(df, df, sq);
        }
        if constexpr (FWD) {
          dist[t] = sqrt_approx(sq);
        } else {
          rs[t] = rsqrt_approx(fmaxf(sq, 1e-30f));
          dist[t] = sq * rs[t];
        }
      }
      lmin = fminf(lmin, dist[t]);
    }
    const float gmin = group_min<LPW>(lmin);
    const float mref = gmin * p.scale;
    float e[KPL];
    float lsum = 0.f;
#pragma unroll
    for (int t = 0; t < KPL; ++t) {
      e[t] = ex2_approx(fmaf(-p.scale, dist[t], mref));
      lsum += e[t];
    }
    const float gsum = group_sum<LPW>(lsum);
    const float r = valid ? rcp_approx(gsum) : 0.f;

    if constexpr (MODE == STEP || MODE == FINAL) {
      float rw[D];
#pragma unroll
      for (int a = 0; a < D; ++a) rw[a] = r * w[a];
#pragma unroll
      for (int t = 0; t < KPL; ++t) {
        acc[t][0] = fmaf(e[t], r, acc[t][0]);
#pragma unroll
        for (int a = 0; a < D; ++a) acc[t][1 + a] = fmaf(e[t], rw[a], acc[t][1 + a]);
      }
      if constexpr (MODE == FINAL) {
        if (p.Wq != nullptr) {
#pragma unroll
          for (int a = 0; a < D; ++a) {
            float s = 0.f;
#pragma unroll
            for (int t = 0; t < KPL; ++t) s = fmaf(e[t], (gl * KPL + t < k) ? c[t][a] : 0.f, s);
            out[a] = group_sum<LPW>(s) * r;
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
      float lz = 0.f;
#pragma unroll
      for (int t = 0; t < KPL; ++t) {
        float v = 0.f;
        if constexpr (NEED_G) {
#pragma unroll
          for (int a = 0; a < D; ++a) v = fmaf(gi[a], (gl * KPL + t < k) ? c[t][a] : 0.f, v);
        }
        if constexpr (NEED_U) {
#pragma unroll
          for (int a = 0; a < D; ++a) v = fmaf(us[t][a], w[a] - fj[t][a], v);
        }
        z[t] = v;
        lz = fmaf(e[t], v, lz);
      }
      const float zbar = group_sum<LPW>(lz) * r;
      const float rt = r * p.inv_tau;
      float dwl[D];
#pragma unroll
      for (int a = 0; a < D; ++a) dwl[a] = 0.f;
#pragma unroll
      for (int t = 0; t < KPL; ++t) {
        const float at = e[t] * r;                    // A_ij
        const float et = e[t] * rt * (z[t] - zbar);   // e_ij(z) / tau
#pragma unroll
        for (int a = 0; a < D; ++a) {
          const float df = w[a] - c[t][a];
          float n;
          if constexpr (D == 1) n = (df > 0.f) ? 1.f : ((df < 0.f) ? -1.f : 0.f);
          else n = df * rs[t];
          if constexpr (MODE == GRAD) acc[t][a] = fmaf(at, gi[a], fmaf(et, n, acc[t][a]));
          if constexpr (MODE == ADJ) acc[t][a] = fmaf(et, n, acc[t][a]);
          if constexpr (MODE == SCATTER) dwl[a] = fmaf(at, us[t][a], fmaf(-et, n, dwl[a]));
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
      // across the groups of a warp (lanes with equal gl)
#pragma unroll
      for (int t = 0; t < KPL; ++t)
#pragma unroll
        for (int a = 0; a < NA; ++a) {
          float v = acc[t][a];
#pragma unroll
          for (int o = LPW; o < 32; o <<= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
          acc[t][a] = v;
        }
      __syncthreads();
      if (lane < LPW) {
#pragma unroll
        for (int t = 0; t < KPL; ++t)
#pragma unroll
          for (int a = 0; a < NA; ++a) red[warp * PLEN + (gl * KPL + t) * NA + a] = acc[t][a];
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

  // ---- persistent loop over this block's tiles -------------------------------------------------
  for (int tile = t_lo; tile < t_hi; ++tile) {
    while (p.lt.tile_off[layer + 1] <= tile) ++layer;
    if (layer != cur_layer) {
      if (cur_layer >= 0 && layer_active) flush(cur_layer);
      cur_layer = layer;
      if constexpr (MODE == STEP)
        layer_active = (p.st[layer].fwd_done == 0) && (p.st[layer].precise == 0) && (p.st[layer].fwd_iters == p.iter);
      else if constexpr (MODE == ADJ) layer_active = (p.st[layer].adj_done == 0);
      else layer_active = true;
      if (layer_active) load_layer(layer);
    }
    if (!layer_active) continue;
    const long long row0 = p.lt.row_off[layer];
    const long long rows = p.lt.row_off[layer + 1] - row0;
    const long long tbase = (long long)(tile - p.lt.tile_off[layer]) * TILE;   // first row of the tile in the layer

    if constexpr (LPW == 1) {
      const bool vec_ok = ((row0 * D) % 4 == 0);
      constexpr int UN = Cfg::UNROLL;
      float wv[UN][VEC][D];
      float gv[UN][VEC][D];
      (void)gv;
      long long first[UN];
      // issue all loads of the tile first
#pragma unroll
      for (int un = 0; un < UN; ++un) {
        const long long loc = tbase + (long long)(un * BLOCK + tid) * VEC;
        first[un] = loc;
        const long long grow = row0 + loc;
        if (vec_ok && loc + VEC <= rows) {
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
          if constexpr (NEED_G) process(wv[un][v], gv[un][v], loc + v < rows, grow + v, outv[v]);
          else process(wv[un][v], gdummy, loc + v < rows, grow + v, outv[v]);
        }
        if constexpr (MODE == FINAL || MODE == SCATTER) {
          float* dst = (MODE == FINAL) ? p.Wq : p.dW;
          if (dst != nullptr) {
            if (vec_ok && loc + VEC <= rows) {
              float os[4];
#pragma unroll
              for (int v = 0; v < VEC; ++v)
#pragma unroll
                for (int a = 0; a < D; ++a) os[v * D + a] = outv[v][a];
              *reinterpret_cast<float4*>(dst + grow * D) = make_float4(os[0], os[1], os[2], os[3]);
            } else {
#pragma unroll
              for (int v = 0; v < VEC; ++v)
                if (loc + v < rows)
#pragma unroll
                  for (int a = 0; a < D; ++a) dst[(grow + v) * D + a] = outv[v][a];
            }
          }
        }
      }
    } else {
      // group-per-weight: every lane of the group reads the same row (one broadcast request)
      const long long gbase = tbase + (long long)grp * WPG;
#pragma unroll 2
      for (int t = 0; t < WPG; ++t) {
        const long long loc = gbase + t;
        const bool ok = (loc < rows);
        const long long grow = row0 + (ok ? loc : 0);
        float w[D], gi[D], outv[D];
        if constexpr (D == 4) {
          const float4 x = __ldg(reinterpret_cast<const float4*>(p.W + grow * 4));
          w[0] = x.x; w[1] = x.y; w[2] = x.z; w[3] = x.w;
        } else if constexpr (D == 2) {
          const float2 x = __ldg(reinterpret_cast<const float2*>(p.W + grow * 2));
          w[0] = x.x; w[1] = x.y;
        } else {
          w[0] = __ldg(p.W + grow);
        }
#pragma unroll
        for (int a = 0; a < D; ++a) gi[a] = 0.f;
        if constexpr (NEED_G) {
          if constexpr (D == 4) {
            const float4 y = __ldg(reinterpret_cast<const float4*>(p.G + grow * 4));
            gi[0] = y.x; gi[1] = y.y; gi[2] = y.z; gi[3] = y.w;
          } else if constexpr (D == 2) {
            const float2 y = __ldg(reinterpret_cast<const float2*>(p.G + grow * 2));
            gi[0] = y.x; gi[1] = y.y;
          } else {
            gi[0] = __ldg(p.G + grow);
          }
        }
        process(w, gi, ok, grow, outv);
        if constexpr (MODE == FINAL || MODE == SCATTER) {
          float* dst = (MODE == FINAL) ? p.Wq : p.dW;
          if (dst != nullptr && ok && gl == 0) {
            if constexpr (D == 4) *reinterpret_cast<float4*>(dst + grow * 4) = make_float4(outv[0], outv[1], outv[2], outv[3]);
            else if constexpr (D == 2) *reinterpret_cast<float2*>(dst + grow * 2) = make_float2(outv[0], outv[1]);
            else dst[grow] = outv[0];
          }
        }
      }
    }
  }
  if (cur_layer >= 0 && layer_active) flush(cur_layer);
}


// ---- fp64 forward step for collapsing layers ------------------------------------------------------------
// Same sums as the STEP pass, for the layers flagged `precise`.  There every logit difference is below
// PRECISE_SPAN, so exp is a short Taylor series, and everything from w - c to the accumulation is fp64.
template <int D, int KPL, int LPW>
struct PreciseCfg {
  static constexpr int KP = KPL * LPW;
  static constexpr int NA = D + 1;
  static constexpr int PLEN = KP * NA;
  static constexpr int WPG = 16;
  static constexpr int TILE = (BLOCK / LPW) * WPG;
};

__device__ __forceinline__ double exp_small(double y) {   // |y| <= PRECISE_SPAN: truncation error < 1e-16
  double s = 1.0 / 40320.0;
  s = fma(s, y, 1.0 / 5040.0);
  s = fma(s, y, 1.0 / 720.0);
  s = fma(s, y, 1.0 / 120.0);
  s = fma(s, y, 1.0 / 24.0);
  s = fma(s, y, 1.0 / 6.0);
  s = fma(s, y, 0.5);
  s = fma(s, y, 1.0);
  return fma(s, y, 1.0);
}

template <int LPW>
__device__ __forceinline__ double group_sum_d(double v) {
#pragma unroll
  for (int o = LPW / 2; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
template <int LPW>
__device__ __forceinline__ double group_min_d(double v) {
#pragma unroll
  for (int o = LPW / 2; o > 0; o >>= 1) v = fmin(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

template <int D, int KPL, int LPW>
__global__ void __launch_bounds__(BLOCK) idkm_step_precise(const __grid_constant__ PassParams p) {
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
  if (t_lo >= t_hi) return;

  double c[KPL][D];
  double acc[KPL][NA];
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
      layer_active = (p.st[layer].fwd_done == 0) && (p.st[layer].precise != 0) && (p.st[layer].fwd_iters == p.iter);
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
    const long long gbase = (long long)(tile - p.lt.tile_off[layer]) * TILE + (long long)grp * WPG;
#pragma unroll 1
    for (int q = 0; q < WPG; ++q) {
      const long long loc = gbase + q;
      const bool ok = (loc < rows);
      const long long grow = row0 + (ok ? loc : 0);
      double w[D];
#pragma unroll
      for (int a = 0; a < D; ++a) w[a] = (double)__ldg(p.W + grow * D + a);
      double dist[KPL];
      double lmin = 1e300;
#pragma unroll
      for (int t = 0; t < KPL; ++t) {
        double sq = 0.0;
#pragma unroll
        for (int a = 0; a < D; ++a) {
          const double df = w[a] - c[t][a];
          sq = (D == 1) ? fabs(df) : fma(df, df, sq);
        }
        dist[t] = (D == 1) ? sq : sqrt(sq);
        if (gl * KPL + t < k) lmin = fmin(lmin, dist[t]);
      }
      const double gmin = group_min_d<LPW>(lmin);
      double e[KPL];
      double lsum = 0.0;
#pragma unroll
      for (int t = 0; t < KPL; ++t) {
        e[t] = (gl * KPL + t < k) ? exp_small((gmin - dist[t]) * p.inv_tau_d) : 0.0;
        lsum += e[t];
      }
      const double gsum = group_sum_d<LPW>(lsum);
      const double r = ok ? 1.0 / gsum : 0.0;
#pragma unroll
      for (int t = 0; t < KPL; ++t) {
        const double at = e[t] * r;
        acc[t][0] += at;
#pragma unroll
        for (int a = 0; a < D; ++a) acc[t][1 + a] = fma(at, w[a], acc[t][1 + a]);
      }
    }
  }
  if (cur_layer >= 0 && layer_active) flush(cur_layer);
}

// host-side dispatch (defined in the per-mode instantiation units)
typedef cudaError_t (*LaunchFn)(const PassParams& p, int grid, cudaStream_t stream);
struct KernelEntry {
  LaunchFn launch;
  const void* func;
  int kpl, lpw, tile, plen;
};
// family index f: 0..7 -> supports k <= kpl*lpw
constexpr int N_FAMILY = 8;
const KernelEntry* kernel_entry(int mode, int d, int family);
int pick_family(int mode, int d, int k);

}  // namespace idkm
