// Algorithm 1's whole loop in ONE cooperative launch, for a small layer or a batch of layers (k <= 16, a few million
// weights per layer at most).  Every block works for exactly one layer: the layers share the grid in proportion to their
// rows (at least one block each) and the grid-wide barrier; everything else below happens per layer, among its blocks.
//
// There one iteration is a few microseconds of arithmetic, and a launch per iteration -- with its chain of dependent
// trips to L2 (partials, ticket, totals, centroids, state) -- costs more than the arithmetic.  Here all blocks are
// co-resident; per iteration each block adds up its rows, publishes one fp64 partial, waits at a grid-wide barrier
// (one counter that only grows), and then EVERY block adds all partials in the same fixed order and takes the M-step
// itself: centroids, iteration count, residual and stop flag live in registers / shared memory of every block and are
// bit-identical everywhere, so nothing but the partials crosses L2 inside the loop.  W is read through the read-only
// path and stays in L1 from the second iteration on.  Block 0 writes the centroids and the layer state once, at the end.
#include "idkm_kernels.cuh"

namespace idkm {

constexpr int SMALL_CHUNK = 32;   // rows a thread adds into one fp32 accumulator before it moves the sum out

template <int D, int KPL>
struct SmallCfg {
  static constexpr int NA = D + 1;
  static constexpr int PLENK = KPL * NA;           // per-centroid sums
  // ... then, for increment-form iterations, the sum of the weights and (scalar weights) count and sum of the rows
  // above / below all centroids, which need no per-centroid work
  static constexpr int NEXTRA = (D == 1) ? 4 : 0;
  static constexpr int PLEN = PLENK + D + NEXTRA;
  static constexpr int CH = BLOCK / PLEN;          // chunks of partial rows added in parallel in the second level
  static constexpr int KD = KPL * D;
  static constexpr int DYN_SMEM = PLEN * BLOCK * 4;
};

// Grid-wide barrier of a cooperative launch: one arrival counter that only grows (sync[0]) and an error word (sync[1]).
// Bounded wait until the arrival counter has reached `target`.  Returns false if the wait ran out or another block
// raised the error word.
__device__ __forceinline__ bool small_barrier(unsigned int* sync, unsigned int target, long long spin_limit, int* s_ok) {
  __syncthreads();
  if (threadIdx.x == 0) {
    volatile unsigned int* vs = sync;
    int ok = 1;
    __threadfence();
    atomicAdd(&sync[0], 1u);
    const long long t0 = clock64();
    while ((int)(vs[0] - target) < 0) {
      if (vs[1] != 0u || clock64() - t0 > spin_limit) {
        atomicExch(&sync[1], 1u);
        ok = 0;
        break;
      }
    }
    if (vs[1] != 0u) ok = 0;
    __threadfence();
    *s_ok = ok;
  }
  __syncthreads();
  return *s_ok != 0;
}

// CHUNKED: some thread has more than SMALL_CHUNK rows; its fp32 sums are then moved out every SMALL_CHUNK rows.
template <int D, int KPL, bool CHUNKED>
__global__ void __launch_bounds__(BLOCK, 2) idkm_small_loop(const __grid_constant__ SmallLoopParams sp) {
  using Cfg = SmallCfg<D, KPL>;
  constexpr int NA = Cfg::NA, PLEN = Cfg::PLEN, PLENK = Cfg::PLENK, CH = Cfg::CH, KD = Cfg::KD;
  __shared__ float red[NWARP][PLEN];
  __shared__ double chunk[CH][PLEN];
  __shared__ double tot[PLEN];
  __shared__ float c_sm[KD > 0 ? KD : 1];   // the current centroids (every block holds the same values)
  __shared__ double s_res[4];       // residual, dead, bad, collapse flag
  __shared__ int s_ok;
  extern __shared__ __align__(16) float slots[];   // [PLEN][BLOCK] second-level fp32 sums (CHUNKED only)

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = gridDim.x;
  const int k = sp.k;
  // this block's layer, its rank among the layer's blocks (b) and their number (NB)
  int layer = 0;
  while (layer + 1 < sp.n_layers && (int)blockIdx.x >= sp.blk_first[layer + 1]) ++layer;
  const int first_blk = sp.blk_first[layer];
  const int b = (int)blockIdx.x - first_blk, NB = sp.blk_first[layer + 1] - first_blk;
  const long long m = sp.row_off[layer + 1] - sp.row_off[layer];
  const float* Wl = sp.W + sp.row_off[layer] * D;
  float* Cl = sp.C + (size_t)layer * k * D;
  LayerState* st = sp.st + layer;

  // uniform loop state (identical in every thread of every block of the layer)
  int iters = 0, done = 0, status = ST_OK, dead_n = 0;
  int precise = st->precise[0];
  float res_f = 0.f;
  if (tid < k * D) c_sm[tid] = Cl[tid];
  __syncthreads();
  float c[KPL][D];
#pragma unroll
  for (int t = 0; t < KPL; ++t)
#pragma unroll
    for (int a = 0; a < D; ++a) c[t][a] = (t < k) ? c_sm[t * D + a] : PAD_COORD;
  const float inv_tau = (float)sp.inv_tau_d;
  const float inv_k = 1.f / (float)k;
  bool ok = true;
  // a grid of one block (a layer of a few thousand weights) needs neither the partial buffers nor the barrier
  const bool solo = (G == 1) && (sp.missing_arrivals == 0);

  for (int it = 0; it < sp.max_iter; ++it) {
    if (sp.n_layers == 1 && done) break;   // (a batch goes on meeting at the barrier until every layer has ended)
    // ---- this block's rows and its partial (fixed order: lanes by shuffle tree, warps in index order) ----
    double* mine = sp.partials + ((size_t)(it & 1) * G + blockIdx.x) * PLEN;
    auto load_row = [&](long long r, float (&w)[D]) {
      if constexpr (D == 4) {
        const float4 x = __ldg(reinterpret_cast<const float4*>(Wl) + r);
        w[0] = x.x; w[1] = x.y; w[2] = x.z; w[3] = x.w;
      } else if constexpr (D == 2) {
        const float2 x = __ldg(reinterpret_cast<const float2*>(Wl) + r);
        w[0] = x.x; w[1] = x.y;
      } else {
        w[0] = __ldg(Wl + r);
      }
    };
    if (!done) {
    // Sums of this thread: [t * NA + a] per centroid, then D entries for the sum of the weights (increment form only).
    // A long fp32 running sum drops the many terms below half its ulp (one-sided): threads with more than
    // SMALL_CHUNK rows move their sums into a private shared-memory slot every SMALL_CHUNK rows.
    float sum[PLEN];
#pragma unroll
    for (int o = 0; o < PLEN; ++o) {
      sum[o] = 0.f;
      if constexpr (CHUNKED) slots[o * BLOCK + tid] = 0.f;
    }
    int since = 0;
    auto spill = [&]() {
#pragma unroll
      for (int o = 0; o < PLEN; ++o) {
        slots[o * BLOCK + tid] += sum[o];
        sum[o] = 0.f;
      }
    };
    // The rows of this block, grid-strided: 128-bit loads of 4 / D rows each, two in flight beyond the one being
    // processed; what does not fill a 128-bit load (and everything, if W is not 16-byte aligned) by row.
    auto walk = [&](auto&& row) {
      constexpr int VEC = 4 / D;
      const long long stride = (long long)NB * BLOCK;
      long long first_by_row = 0;
      if ((reinterpret_cast<size_t>(Wl) & 15) == 0) {
        const long long nvec = m / VEC;
        const float4* W4 = reinterpret_cast<const float4*>(Wl);
        long long q = (long long)b * BLOCK + tid;
        float4 cur = make_float4(0.f, 0.f, 0.f, 0.f), n1 = cur, n2 = cur;
        if (q < nvec) cur = __ldg(W4 + q);
        if (q + stride < nvec) n1 = __ldg(W4 + q + stride);
        for (; q < nvec; q += stride) {
          if (q + 2 * stride < nvec) n2 = __ldg(W4 + q + 2 * stride);
          if constexpr (CHUNKED) {
            if (since >= SMALL_CHUNK) {
              spill();
              since = 0;
            }
            since += VEC;
          }
          const float xs[4] = {cur.x, cur.y, cur.z, cur.w};
#pragma unroll
          for (int v = 0; v < VEC; ++v) {
            float w[D];
#pragma unroll
            for (int a = 0; a < D; ++a) w[a] = xs[v * D + a];
            row(w);
          }
          cur = n1;
          n1 = n2;
        }
        first_by_row = nvec * VEC;
      }
      for (long long r = first_by_row + (long long)b * BLOCK + tid; r < m; r += stride) {
        float w[D];
        load_row(r, w);
        if constexpr (CHUNKED) {
          if (since >= SMALL_CHUNK) {
            spill();
            since = 0;
          }
          ++since;
        }
        row(w);
      }
    };
    if (!precise) {
      // fp32 rows: the arithmetic of the fused forward step (Algorithm 1, steps 3-5)
      walk([&](const float (&w)[D]) {
        float dist[KPL], e[KPL];
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
            dist[t] = sqrt_approx(sq);
          }
        }
        const float mref = tree_reduce<KPL, 1>(dist) * sp.scale;
#pragma unroll
        for (int t = 0; t < KPL; ++t) e[t] = ex2_approx(fmaf(-sp.scale, dist[t], mref));
        const float rr = rcp_approx(tree_reduce<KPL, 0>(e));
        float rw[D];
#pragma unroll
        for (int a = 0; a < D; ++a) rw[a] = rr * w[a];
#pragma unroll
        for (int t = 0; t < KPL; ++t) {
          sum[t * NA] = fmaf(e[t], rr, sum[t * NA]);
#pragma unroll
          for (int a = 0; a < D; ++a) sum[t * NA + 1 + a] = fmaf(e[t], rw[a], sum[t * NA + 1 + a]);
        }
      });
    } else {
      // A collapsing layer (all centroids within PRECISE_SPAN * tau of each other) steps in the fp32 increment form
      // (see delta_body): with c_0 the reference, delta_j = c_j - c_0 and u_i = w_i - c_0, the logit differences
      // x_ij = -(D_ij - D_i0) / tau and the attention increments A_ij - 1/k = (t_ij - tbar_i) / (k (1 + tbar_i)),
      // t = exp(x) - 1, are formed to fp32 accuracy RELATIVE to delta; summed: dS_j, dN_j = sum (A_ij - 1/k) u_i and
      // sum_i w_i.  The M-step below turns them into C+_j = c_0 + (U / k + dN_j) / (m / k + dS_j) in fp64.
      float c0[D], dl[KPL][D], dl2[KPL];
#pragma unroll
      for (int a = 0; a < D; ++a) c0[a] = c[0][a];
#pragma unroll
      for (int t = 0; t < KPL; ++t) {
        double d2 = 0.0;
#pragma unroll
        for (int a = 0; a < D; ++a) {
          const double dd = (t < k) ? (double)c[t][a] - (double)c0[a] : 0.0;
          dl[t][a] = (float)dd;
          d2 += dd * dd;
        }
        dl2[t] = (float)d2;
      }
      // scalar weights: a row farther than twice the largest |delta_j| from c_0 lies outside all centroids; its
      // attention increments take one of two values per centroid (applied in the M-step), so it is only counted
      float dmax2 = 0.f;
      if constexpr (D == 1) {
#pragma unroll
        for (int t = 0; t < KPL; ++t) dmax2 = fmaxf(dmax2, 2.f * fabsf(dl[t][0]));
      }
      walk([&](const float (&w)[D]) {
        float u[D], x[KPL];
#pragma unroll
        for (int a = 0; a < D; ++a) u[a] = w[a] - c0[a];
        if constexpr (D == 1) {
          if (fabsf(u[0]) > dmax2) {
            const bool pos = (u[0] > 0.f);
            sum[PLENK + 1] += pos ? 1.f : 0.f;
            sum[PLENK + 2] += pos ? w[0] : 0.f;
            sum[PLENK + 3] += pos ? 0.f : 1.f;
            sum[PLENK + 4] += pos ? 0.f : w[0];
            return;
          }
        }
        if constexpr (D == 1) {
          // |u - delta| - |u| without forming u - delta: with s = sign(u), -s delta + 2 max(0, s delta - |u|)
          const float aut = fabsf(u[0]) * inv_tau;
          const float sg = copysignf(inv_tau, u[0]);
#pragma unroll
          for (int t = 0; t < KPL; ++t) {
            const float sd = sg * dl[t][0];
            x[t] = fmaf(-2.f, fmaxf(sd - aut, 0.f), sd);
          }
        } else {
          float d0sq = 0.f, v[D];
#pragma unroll
          for (int a = 0; a < D; ++a) {
            d0sq = fmaf(u[a], u[a], d0sq);
            v[a] = -2.f * u[a];
          }
          const float d0 = sqrt_approx(d0sq);
#pragma unroll
          for (int t = 0; t < KPL; ++t) {
            float q = dl2[t];
#pragma unroll
            for (int a = 0; a < D; ++a) q = fmaf(dl[t][a], v[a], q);          // D_ij^2 - D_i0^2
            const float dij = sqrt_approx(fmaxf(d0sq + q, 0.f));
            x[t] = -q * inv_tau * rcp_approx(fmaxf(dij + d0, 1e-30f));
          }
        }
        float tt[KPL], lsum = 0.f;
#pragma unroll
        for (int t = 0; t < KPL; ++t) {
          tt[t] = (t < k) ? expm1_small(x[t]) : 0.f;
          lsum += tt[t];
        }
        const float tbar = lsum * inv_k;
        const float rr = inv_k * rcp_approx(1.f + tbar);
        const float ntr = -tbar * rr;
#pragma unroll
        for (int t = 0; t < KPL; ++t) {
          const float aij = (t < k) ? fmaf(tt[t], rr, ntr) : 0.f;
          sum[t * NA] += aij;
#pragma unroll
          for (int a = 0; a < D; ++a) sum[t * NA + 1 + a] = fmaf(aij, u[a], sum[t * NA + 1 + a]);
        }
#pragma unroll
        for (int a = 0; a < D; ++a) sum[PLENK + a] += w[a];
      });
    }
#pragma unroll
    for (int o2 = 0; o2 < PLEN; ++o2) {
      float v = sum[o2];
      if constexpr (CHUNKED) v += slots[o2 * BLOCK + tid];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
      if (lane == 0) red[warp][o2] = v;
    }
    __syncthreads();
    if (tid < PLEN) {
      double s = 0.0;
#pragma unroll
      for (int wv = 0; wv < NWARP; ++wv) s += (double)red[wv][tid];
      if (solo) tot[tid] = s;   // a grid of one block: the layer's totals, no trip through global memory
      else __stcg(mine + tid, s);
    }
    }   // !done
    if (solo) {
      __syncthreads();
    } else {
    // ---- everyone has published: grid-wide barrier ----
    ok = small_barrier(sp.sync, (unsigned int)(it + 1) * (unsigned int)(G + sp.missing_arrivals), sp.spin_limit, &s_ok);
    if (!ok) break;
    }
    // A batch ends at the first barrier at which every layer's loop has ended: the first block of a layer publishes
    // fwd_done = (iterations taken) before it arrives at the next barrier, so after barrier `it` every value in
    // (0, it] is final and seen by all blocks alike; a later value cannot be mistaken for one of them.
    if (sp.n_layers > 1 && sp.tol > 0.f) {
      int ended = 1;
      for (int l = tid; l < sp.n_layers; l += BLOCK) {
        const int fd = *reinterpret_cast<const volatile int*>(&sp.st[l].fwd_done);
        if (fd == 0 || fd > it) ended = 0;
      }
      if (__syncthreads_and(ended)) break;
    }
    if (done) continue;
    // ---- every block of the layer adds the layer's partials in the same order ----
    if (!solo) {
      const double* base = sp.partials + ((size_t)(it & 1) * G + first_blk) * PLEN;
      const int ch = tid / PLEN, o = tid % PLEN;
      if (ch < CH) {
        double s = 0.0;
        for (int q = ch; q < NB; q += CH) s += __ldcg(base + (size_t)q * PLEN + o);
        chunk[ch][o] = s;
      }
      __syncthreads();
      if (tid < PLEN) {
        double s = 0.0;
#pragma unroll 1
        for (int q = 0; q < CH; ++q) s += chunk[q][tid];
        tot[tid] = s;
      }
      __syncthreads();
    }
    // ---- M-step by the first warp: lane (j, a) owns coordinate a of centroid j ----
    if (warp == 0) {
      const int j = lane / D, a = lane % D;
      (void)a;
      const bool own = (lane < k * D);
      double num = 0.0, den = 0.0, bad = 0.0, dead = 0.0, cq = 0.0;
      // increment form: centroid 0 as it was when the rows were taken (read by all lanes before any lane writes)
      const double c0a = (double)c_sm[own ? a : 0];
      double tS = own ? tot[j * NA] : 0.0, tN = own ? tot[j * NA + 1 + a] : 0.0, wsum = own ? tot[PLENK + a] : 0.0;
      if constexpr (D == 1) {
        if (precise) {
          // the rows that were only counted: above all centroids their logit differences are +delta_j / tau, below
          // -delta_j / tau, whatever their own value
          const double cp = tot[PLENK + 1], sp_ = tot[PLENK + 2], cm = tot[PLENK + 3], sm = tot[PLENK + 4];
          const double dj = own ? ((double)c_sm[lane] - c0a) * sp.inv_tau_d : 0.0;
          const double tpj = own ? expm1(dj) : 0.0, tmj = own ? expm1(-dj) : 0.0;
          double tbp = tpj, tbm = tmj;
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) {
            tbp += __shfl_xor_sync(0xffffffffu, tbp, o);
            tbm += __shfl_xor_sync(0xffffffffu, tbm, o);
          }
          tbp /= (double)k;
          tbm /= (double)k;
          const double ap = (tpj - tbp) / ((double)k * (1.0 + tbp)), am = (tmj - tbm) / ((double)k * (1.0 + tbm));
          tS += ap * cp + am * cm;
          tN += ap * (sp_ - cp * c0a) + am * (sm - cm * c0a);
          wsum += sp_ + sm;
        }
      }
      __syncwarp();
      if (own) {
        const double mk = (double)m / (double)k;
        const double s = precise ? mk + tS : tS;
        const bool alive = (s >= S_MIN);
        const double cold = (double)c_sm[lane];
        const double ubar = precise ? (wsum - (double)m * c0a) / (double)k : 0.0;
        const double cnew = alive ? (precise ? c0a + (ubar + tN) / s : tN / s) : cold;
        if (!alive && a == 0) dead = 1.0;
        if (!(s == s) || s > 1e300 || !(cnew == cnew) || fabs(cnew) > 1e300) bad = 1.0;
        num = (cnew - cold) * (cnew - cold);
        den = cnew * cnew;
        cq = (double)(float)cnew;
        c_sm[lane] = (float)cnew;
      }
      double lo = own ? cq : 1e300, hi = own ? cq : -1e300;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        num += __shfl_xor_sync(0xffffffffu, num, o);
        den += __shfl_xor_sync(0xffffffffu, den, o);
        bad += __shfl_xor_sync(0xffffffffu, bad, o);
        dead += __shfl_xor_sync(0xffffffffu, dead, o);
      }
      // bounding box per coordinate: lanes with equal a differ by multiples of D
#pragma unroll
      for (int o = 16; o >= D; o >>= 1) {
        lo = fmin(lo, __shfl_xor_sync(0xffffffffu, lo, o));
        hi = fmax(hi, __shfl_xor_sync(0xffffffffu, hi, o));
      }
      double ext = (lane < D) ? (hi - lo) * (hi - lo) : 0.0;
#pragma unroll
      for (int o = D / 2; o > 0; o >>= 1) ext += __shfl_xor_sync(0xffffffffu, ext, o);
      if (lane == 0) {
        // (one fp64 division, the square root in fp32, the collapse test on squares and by this thread alone instead of
        // an fp64 square root in every thread of the block: 0.1 of an iteration's 5 us on the smallest layers)
        s_res[0] = (double)sqrtf((float)(num / fmax(den, 1e-300)));
        s_res[1] = dead;
        s_res[2] = bad;
        s_res[3] = (ext * sp.inv_tau_d * sp.inv_tau_d <= (double)PRECISE_SPAN * (double)PRECISE_SPAN) ? 1.0 : 0.0;
      }
    }
    __syncthreads();
#pragma unroll
    for (int t = 0; t < KPL; ++t)
#pragma unroll
      for (int a = 0; a < D; ++a) c[t][a] = (t < k) ? c_sm[t * D + a] : PAD_COORD;
    iters = it + 1;
    res_f = (float)s_res[0];
    if (b == 0 && tid == 0 && iters <= HIST_CAP) sp.hist[(size_t)layer * HIST_CAP + iters - 1] = res_f;
    dead_n = (int)s_res[1];
    precise = (s_res[3] != 0.0) ? 1 : 0;
    if (s_res[2] > 0.0) {
      status = ST_NONFINITE;
      done = iters;
    } else if (sp.tol > 0.f && res_f < sp.tol) {
      done = iters;
      status = ST_OK;
    } else if (sp.tol > 0.f && iters >= sp.max_iter) {
      status = ST_MAXITER;
    }
    if (done && b == 0 && tid == 0) st->fwd_done = done;   // (seen by the other layers' blocks after the next barrier)
    __syncthreads();
  }

  if (b == 0) {
    if (tid < k * D) Cl[tid] = c_sm[tid];
    if (tid == 0) {
      st->fwd_iters = iters;
      st->fwd_res = res_f;
      st->dead = dead_n;
      st->fwd_done = done;
      st->precise[0] = st->precise[1] = precise;
      st->status = ok ? status : ST_TIMEOUT;
      st->ticket = 0u;
    }
  }
}

template <int D, int KPL>
static cudaError_t launch_small(const SmallLoopParams& sp, int grid, cudaStream_t stream) {
  constexpr int DYN = SmallCfg<D, KPL>::DYN_SMEM;
  static bool configured = false;   // the slots of the widest layouts reach the 48 KB default limit
  if (!configured) {
    const cudaError_t rc = cudaFuncSetAttribute(idkm_small_loop<D, KPL, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, DYN);
    if (rc != cudaSuccess) return rc;
    configured = true;
  }
  void* args[1] = {const_cast<SmallLoopParams*>(&sp)};
  // cooperative launch: refused (instead of hanging at the first barrier) if the grid cannot be co-resident
  if (sp.chunked)
    return cudaLaunchCooperativeKernel((const void*)&idkm_small_loop<D, KPL, true>, dim3((unsigned)grid, 1, 1),
                                       dim3(BLOCK, 1, 1), args, (size_t)DYN, stream);
  return cudaLaunchCooperativeKernel((const void*)&idkm_small_loop<D, KPL, false>, dim3((unsigned)grid, 1, 1),
                                     dim3(BLOCK, 1, 1), args, 0, stream);
}
#define IDKM_SMALL_ENTRY(D, KPL) \
  { &launch_small<D, KPL>, (const void*)&idkm_small_loop<D, KPL, true>, KPL, SmallCfg<D, KPL>::PLEN, SmallCfg<D, KPL>::DYN_SMEM }
#define IDKM_SMALL_NONE { nullptr, nullptr, 0, 0, 0 }
// 16 centroids per thread only for d = 1, 2: with d = 4 the centroids and sums alone exceed the register budget
extern const SmallLoopEntry k_table_small[3][N_SMALL_FAMILY] = {
    {IDKM_SMALL_ENTRY(1, 2), IDKM_SMALL_ENTRY(1, 4), IDKM_SMALL_ENTRY(1, 8), IDKM_SMALL_ENTRY(1, 16)},
    {IDKM_SMALL_ENTRY(2, 2), IDKM_SMALL_ENTRY(2, 4), IDKM_SMALL_ENTRY(2, 8), IDKM_SMALL_ENTRY(2, 16)},
    {IDKM_SMALL_ENTRY(4, 2), IDKM_SMALL_ENTRY(4, 4), IDKM_SMALL_ENTRY(4, 8), IDKM_SMALL_NONE}};

}  // namespace idkm
