// Explicit Jacobian J_C = dF/dC for codebooks with 8 < k d <= 64 (one pass over W), and the whole adjoint iteration
// on that matrix.
//
//   J[(j,a),(l,b)] = sum_i P_ija (delta_jl - A_il) n_ilb,   P_ija = A_ij (w_ia - F_ja) / (S_j tau)
//                  = Dg - X^T Y,   X_i[(j,a)] = P_ija,  Y_i[(l,b)] = A_il n_ilb,  Dg[(j,a),(j,b)] = sum_i P_ija n_ijb.
//
// X^T Y is a sum of outer products of two k d - vectors per weight.  A block works on batches of 32 weights: its warps
// compute the attention row of four weights each (lane = centroid) and park X_i, Y_i in shared memory; then all 256
// threads add the 32 outer products into a k d x k d accumulator that is spread over the block's registers
// ((k d / 16)^2 entries per thread).  Sums: fp32 per 64 weights, moved into a second fp32 level, fp64 across blocks.
// This is the paper's own formulation (it iterates a k x k matrix, Section 4.2); it replaces adj_max_iter passes over
// W by one, which pays as soon as the iteration runs more than a few tens of steps.
//
// k d = 16 and 32 (QT below) take a denser arrangement, because there a lane-per-centroid producer leaves lanes idle
// and a thread's corner of the matrix is one or four entries (one shared load per FMA): a thread computes the attention
// row of ONE weight (no cross-lane reduction; the centroids in its registers at k d = 16, in shared memory at 32) and
// parks X_i, Y_i; then the matrix is (k d / 4)^2 tiles of 4 x 4, each taken by 16 resp. 4 threads that split the
// batch's weights among them (two 128-bit shared loads per 16 FMAs).  The diagonal term Dg is folded in: the producer
// also parks Z_i[(j,b)] = (A_ij - 1) n_ijb and the entries of a diagonal tile that belong to a (j, j) block take Z_i in
// place of Y_i (at d = 4 that is the whole tile); at k d = 16 with d < 4 the producer sums P_ija n_ijb itself instead.
#pragma once
#include "idkm_kernels.cuh"

namespace idkm {

template <int D, int KP>
struct JacTileCfg {
  static constexpr int KD = KP * D;            // 16, 32 or 64
  static constexpr int TR = KD / 16;           // accumulator rows (and columns) per thread
  static constexpr int CPL = (KP + 31) / 32;   // centroids per lane in the producer phase
  static constexpr int NDG = KP * D * D;       // block-diagonal part
  static constexpr int PLEN = KD * KD + NDG;
  static constexpr int BATCH = 32;             // weights per batch (four per warp)
  static constexpr int TILE = 256;             // rows per tile of the layer table
  static constexpr bool QT = (KD == 16 || KD == 32);   // thread-per-weight producer, 4 x 4 tiles (see above)
  static constexpr bool QREG = (KD == 16);             // ... with the centroids in registers (else in shared memory)
  static constexpr bool QZ = QT && (D == 4 || KD == 32);   // ... with Z rows (else the producer sums Dg)
  static constexpr int QB = (KD == 16) ? 256 : 128;    // weights per batch on that path (one per producing thread)
  static constexpr int XS = KD + 4;                    // row stride of X / Y / Z there: 128-bit stores of consecutive
                                                       // rows hit different banks
  static constexpr int NT1 = KD / 4;                   // tiles per side
  static constexpr int TPT = QT ? BLOCK / (NT1 * NT1) : 1;   // threads per tile
  static constexpr int XY_FLOATS = QT ? QB * XS * (QZ ? 3 : 2) : 2 * BATCH * KD;
  // dynamic shared memory: the X / Y batch while accumulating, the matrix (fp64) + u + g while solving
  static constexpr int SOLVE_BYTES = (KD * KD + 2 * KD) * 8;
  static constexpr int DYN_SMEM = (XY_FLOATS * 4 > SOLVE_BYTES ? XY_FLOATS * 4 : SOLVE_BYTES) + NDG * NWARP * 4;
};

template <int D, int KP>
__global__ void __launch_bounds__(BLOCK, 2) idkm_jacobian_tile(const __grid_constant__ PassParams p) {
  using Cfg = JacTileCfg<D, KP>;
  constexpr int KD = Cfg::KD, TR = Cfg::TR, CPL = Cfg::CPL, NDG = Cfg::NDG, PLEN = Cfg::PLEN, BATCH = Cfg::BATCH;
  constexpr int TILE = Cfg::TILE;
  constexpr bool QT = Cfg::QT, QREG = Cfg::QREG, QZ = Cfg::QZ;
  constexpr int XS = Cfg::XS, QB = Cfg::QB, NT1 = Cfg::NT1, TPT = Cfg::TPT;
  extern __shared__ __align__(16) unsigned char dyn[];
  float* Xs = reinterpret_cast<float*>(dyn);              // [BATCH][KD]  (QT: [QB][XS])
  float* Ys = Xs + (QT ? QB * XS : BATCH * KD);            // [BATCH][KD]  (QT: [QB][XS], then Z for d = 4)
  float* dgs = reinterpret_cast<float*>(dyn + (Cfg::DYN_SMEM - NDG * NWARP * 4));   // [NWARP][NDG]
  __shared__ int s_flag;

  grid_dependency_sync();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int ty = tid / 16, tx = tid % 16;
  const int k = p.k;
  const int nb = p.lt.n_blocks;
  const int b = blockIdx.x;
  const int t_lo = tile_begin(b, p.lt.tiles_total, nb);
  const int t_hi = tile_begin(b + 1, p.lt.tiles_total, nb);
  if (b >= nb || t_lo >= t_hi) return;

  // producer state: this lane's centroids
  float c[CPL][D], fj[CPL][D], ist[CPL];
  float dg[CPL][D][D], dg_hi[CPL][D][D];
  // consumer state: this thread's TR x TR corner of -X^T Y
  float acc[TR][TR], acc_hi[TR][TR];
  // QT: all centroids of the layer in every thread (or in shared memory); this thread's share of a 4 x 4 tile; the
  // diagonal sums where the producer keeps them
  constexpr int NDQ = (QT && !QZ) ? KP * D * D : 1;
  float cq[QREG ? KP : 1][D], fq[QREG ? KP : 1][D], iq[QREG ? KP : 1];
  __shared__ float c_s[(QT && !QREG) ? KP * D : 1], f_s[(QT && !QREG) ? KP * D : 1], i_s[(QT && !QREG) ? KP : 1];
  float acc4[4][4], acc4_hi[4][4], dgt[NDQ], dgt_hi[NDQ];
  (void)cq; (void)fq; (void)iq; (void)acc4; (void)acc4_hi; (void)dgt; (void)dgt_hi; (void)c_s; (void)f_s; (void)i_s;
  auto cget = [&](int t, int a) -> float { return QREG ? cq[QREG ? t : 0][a] : c_s[(QT && !QREG) ? t * D + a : 0]; };
  auto fget = [&](int t, int a) -> float { return QREG ? fq[QREG ? t : 0][a] : f_s[(QT && !QREG) ? t * D + a : 0]; };
  auto iget = [&](int t) -> float { return QREG ? iq[QREG ? t : 0] : i_s[(QT && !QREG) ? t : 0]; };
  const int q_tile = tid / TPT, q_sub = tid % TPT, q_ty = q_tile / NT1, q_tx = q_tile % NT1;
  int layer = 0;
  while (p.lt.tile_off[layer + 1] <= t_lo) ++layer;
  int cur_layer = -1;
  bool layer_active = false;
  int batches = 0;

  auto finish = [&](int l) {
    // ---- this block's partial: the matrix entries straight from their owners, the diagonal blocks over the warps
    double* mine = p.partials + (size_t)(b + l) * PLEN;
    if constexpr (QT) {
      // the threads of a tile (neighbouring lanes) add their shares; the first writes the tile
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          float v = acc4_hi[i][j] + acc4[i][j];
#pragma unroll
          for (int o = TPT / 2; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
          if (q_sub == 0) mine[(q_ty * 4 + i) * KD + q_tx * 4 + j] = (double)v;
        }
      __syncthreads();   // the X / Y batch is no longer read
      if constexpr (!QZ) {
#pragma unroll
        for (int o2 = 0; o2 < NDQ; ++o2) {
          float v = dgt_hi[o2] + dgt[o2];
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
          if (lane == 0) dgs[warp * NDG + o2] = v;
        }
      } else {
        for (int o2 = lane; o2 < NDG; o2 += 32) dgs[warp * NDG + o2] = 0.f;   // (Dg is inside the diagonal tiles)
      }
    } else {
#pragma unroll
    for (int i = 0; i < TR; ++i)
#pragma unroll
      for (int j = 0; j < TR; ++j)
        mine[(ty * TR + i) * KD + tx * TR + j] = (double)acc_hi[i][j] + (double)acc[i][j];
    __syncthreads();   // the X / Y batch is no longer read
#pragma unroll
    for (int t = 0; t < CPL; ++t)
#pragma unroll
      for (int a = 0; a < D; ++a)
#pragma unroll
        for (int bb = 0; bb < D; ++bb) {
          const int j = lane + 32 * t;
          if (j < KP) dgs[warp * NDG + (j * D + a) * D + bb] = dg_hi[t][a][bb] + dg[t][a][bb];
        }
    }
    __syncthreads();
    for (int o = tid; o < NDG; o += BLOCK) {
      double s = 0.0;
#pragma unroll
      for (int wv = 0; wv < NWARP; ++wv) s += (double)dgs[wv * NDG + o];
      mine[KD * KD + o] = s;
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
    // ---- last block: totals (fixed slot order, eight loads in flight per thread), J = Dg - X^T Y in shared memory
    double* Jm = reinterpret_cast<double*>(dyn);   // [KD][KD]
    double* us = Jm + KD * KD;                      // [KD]
    double* gs = us + KD;                           // [KD]
    const double* base = p.partials + (size_t)(first_b + l) * PLEN;
    for (int o = tid; o < KD * KD; o += BLOCK) {
      double s = 0.0;
#pragma unroll 8
      for (int q = 0; q < n_contrib; ++q) s += __ldcg(base + (size_t)q * PLEN + o);
      const int r = o / KD, cidx = o % KD;
      if (r / D == cidx / D) {   // the delta_jl block: add Dg[(j, a), (j, b)]
        const int j = r / D, a = r % D, bb = cidx % D;
        double sd = 0.0;
#pragma unroll 8
        for (int q = 0; q < n_contrib; ++q) sd += __ldcg(base + (size_t)q * PLEN + KD * KD + (j * D + a) * D + bb);
        s += sd;
      }
      Jm[o] = s;
    }
    const int n = k * D;
    if (tid < KD) {
      gs[tid] = (tid < n) ? (double)p.gvec[(size_t)l * n + tid] : 0.0;
      us[tid] = gs[tid];
    }
    __syncthreads();
    if (warp == 0 && p.max_iter < 0) {
      // exact solve instead of the iteration (idkm_set_adjoint_method(ctx, 2)); gs holds g, then u
      LayerState* st = p.st + l;
      const bool ok = warp_solve_adjoint(Jm, KD, gs, n, lane);
      bool finite = true;
      for (int q = lane; q < n; q += 32) {
        const double uv = ok ? gs[q] : 0.0;
        finite = finite && (uv == uv) && fabs(uv) < 1e300;
        p.u[(size_t)l * n + q] = (float)uv;
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
      // The iteration on the matrix, by one warp: lane q owns coordinates q and q + 32 of u;
      // (J^T u)_q = sum_r J[r][q] u_r with J and u in shared memory.  All lanes see the same residual.
      LayerState* st = p.st + l;
      constexpr int QPL = (KD + 31) / 32;
      const double al = (double)p.alpha;
      int it = 0, up = 0, status = st->status, done = 0;
      float res = 0.f, prev = 3.0e38f;
      double g2 = 0.0;
#pragma unroll
      for (int h = 0; h < QPL; ++h) {
        const int q = lane + 32 * h;
        if (q < n) g2 += gs[q] * gs[q];
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) g2 += __shfl_xor_sync(0xffffffffu, g2, o);
      const double u2_limit = ADJ_GROWTH_LIMIT * ADJ_GROWTH_LIMIT * g2;
      while (it < p.max_iter && !done) {
        double un[QPL];
        double num = 0.0, den = 0.0, badv = 0.0;
#pragma unroll
        for (int h = 0; h < QPL; ++h) {
          const int q = lane + 32 * h;
          double s = 0.0;
          if (q < n)
            for (int r = 0; r < n; ++r) s = fma(Jm[r * KD + q], us[r], s);
          const double uo = (q < KD) ? us[q < KD ? q : 0] : 0.0;
          un[h] = (q < n) ? al * (s + gs[q]) + (1.0 - al) * uo : 0.0;
          num += (un[h] - uo) * (un[h] - uo);
          den += un[h] * un[h];
          if (!(un[h] == un[h]) || fabs(un[h]) > 1e300) badv += 1.0;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          num += __shfl_xor_sync(0xffffffffu, num, o);
          den += __shfl_xor_sync(0xffffffffu, den, o);
          badv += __shfl_xor_sync(0xffffffffu, badv, o);
        }
        __syncwarp();
#pragma unroll
        for (int h = 0; h < QPL; ++h) {
          const int q = lane + 32 * h;
          if (q < KD) us[q] = un[h];
        }
        __syncwarp();
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
#pragma unroll
      for (int h = 0; h < QPL; ++h) {
        const int q = lane + 32 * h;
        if (q < n) p.u[(size_t)l * n + q] = (float)us[q];
      }
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
      batches = 0;
      if (layer_active) {
#pragma unroll
        for (int t = 0; t < CPL; ++t) {
          const int j = lane + 32 * t;
          const bool ok = (j < k);
          const float s = ok ? p.S[(size_t)layer * k + j] : 0.f;
          ist[t] = (ok && s >= S_MIN_F) ? p.inv_tau / s : 0.f;
#pragma unroll
          for (int a = 0; a < D; ++a) {
            c[t][a] = ok ? p.C[((size_t)layer * k + j) * D + a] : PAD_COORD;
            fj[t][a] = ok ? p.F[((size_t)layer * k + j) * D + a] : 0.f;
#pragma unroll
            for (int bb = 0; bb < D; ++bb) {
              dg[t][a][bb] = 0.f;
              dg_hi[t][a][bb] = 0.f;
            }
          }
        }
#pragma unroll
        for (int i = 0; i < TR; ++i)
#pragma unroll
          for (int j = 0; j < TR; ++j) {
            acc[i][j] = 0.f;
            acc_hi[i][j] = 0.f;
          }
        if constexpr (QT) {
          if constexpr (QREG) {
#pragma unroll
            for (int t = 0; t < KP; ++t) {
              const bool ok = (t < k);
              const float sv = ok ? p.S[(size_t)layer * k + t] : 0.f;
              iq[t] = (ok && sv >= S_MIN_F) ? p.inv_tau / sv : 0.f;
#pragma unroll
              for (int a = 0; a < D; ++a) {
                cq[t][a] = ok ? p.C[((size_t)layer * k + t) * D + a] : PAD_COORD;
                fq[t][a] = ok ? p.F[((size_t)layer * k + t) * D + a] : 0.f;
              }
            }
          } else {
            // (finish() of the previous layer ended with a barrier; the batch body starts with one)
            for (int o2 = tid; o2 < KP * D; o2 += BLOCK) {
              const bool ok = (o2 / D < k);
              c_s[o2] = ok ? p.C[(size_t)layer * k * D + o2] : PAD_COORD;
              f_s[o2] = ok ? p.F[(size_t)layer * k * D + o2] : 0.f;
            }
            for (int t = tid; t < KP; t += BLOCK) {
              const bool ok = (t < k);
              const float sv = ok ? p.S[(size_t)layer * k + t] : 0.f;
              i_s[t] = (ok && sv >= S_MIN_F) ? p.inv_tau / sv : 0.f;
            }
          }
#pragma unroll
          for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              acc4[i][j] = 0.f;
              acc4_hi[i][j] = 0.f;
            }
#pragma unroll
          for (int o2 = 0; o2 < NDQ; ++o2) {
            dgt[o2] = 0.f;
            dgt_hi[o2] = 0.f;
          }
        }
      }
    }
    if (!layer_active) continue;
    const long long row0 = p.lt.row_off[layer];
    const long long rows = p.lt.row_off[layer + 1] - row0;
    const long long tbase = (long long)(tile - p.lt.tile_off[layer]) * TILE;
    if constexpr (QT) {
      static_assert(!QT || TILE % QB == 0, "a tile of the layer table is a whole number of batches");
#pragma unroll 1
      for (int b0 = 0; b0 < TILE; b0 += QB) {
        if (tbase + b0 >= rows) break;   // uniform over the block
        __syncthreads();   // the previous batch has been consumed (and the layer's constants are in place)
        if (tid < QB) {
          // ---- producer: this thread's weight of the batch ----
          const long long loc = tbase + b0 + tid;
          const bool valid = (loc < rows);
          const long long grow = row0 + (valid ? loc : 0);
          float w[D];
          if constexpr (D == 4) {
            const float4 x = __ldg(reinterpret_cast<const float4*>(p.W + grow * 4));
            w[0] = x.x; w[1] = x.y; w[2] = x.z; w[3] = x.w;
          } else if constexpr (D == 2) {
            const float2 x = __ldg(reinterpret_cast<const float2*>(p.W + grow * 2));
            w[0] = x.x; w[1] = x.y;
          } else {
            w[0] = __ldg(p.W + grow);
          }
          float e[KP], rsq[D > 1 ? KP : 1];
          (void)rsq;
          float lmin = 3.0e38f;
#pragma unroll
          for (int t = 0; t < KP; ++t) {
            if constexpr (D == 1) {
              e[t] = fabsf(w[0] - cget(t, 0));
            } else {
              float sq = 1e-30f;
#pragma unroll
              for (int a = 0; a < D; ++a) {
                const float df = w[a] - cget(t, a);
                sq = fmaf(df, df, sq);
              }
              rsq[t] = rsqrt_approx(sq);
              e[t] = sq * rsq[t];
            }
            lmin = fminf(lmin, e[t]);
          }
          const float mref = lmin * p.scale;
          float lsum = 0.f;
#pragma unroll
          for (int t = 0; t < KP; ++t) {
            e[t] = ex2_approx(fmaf(-p.scale, e[t], mref));
            lsum += e[t];
          }
          const float rr = valid ? rcp_approx(lsum) : 0.f;
          // four consecutive entries of the rows at a time (4 / D centroids), stored as soon as they are complete
          constexpr int CPC = 4 / D;
#pragma unroll
          for (int q = 0; q < KD / 4; ++q) {
            float xv[4], yv[4], zv[4];
            (void)zv;
#pragma unroll
            for (int cc = 0; cc < CPC; ++cc) {
              const int t = q * CPC + cc;
              const float at = e[t] * rr;
              float nn[D], pp[D];
#pragma unroll
              for (int a = 0; a < D; ++a) {
                const float df = w[a] - cget(t, a);
                if constexpr (D == 1) nn[a] = (df > 0.f) ? 1.f : ((df < 0.f) ? -1.f : 0.f);
                else nn[a] = df * rsq[t];
                pp[a] = at * iget(t) * (w[a] - fget(t, a));
                xv[cc * D + a] = pp[a];
                yv[cc * D + a] = at * nn[a];
                zv[cc * D + a] = (at - 1.f) * nn[a];
              }
              if constexpr (!QZ) {
#pragma unroll
                for (int a = 0; a < D; ++a)
#pragma unroll
                  for (int bb = 0; bb < D; ++bb)
                    dgt[(t * D + a) * D + bb] = fmaf(pp[a], nn[bb], dgt[(t * D + a) * D + bb]);
              }
            }
            *reinterpret_cast<float4*>(Xs + tid * XS + 4 * q) = make_float4(xv[0], xv[1], xv[2], xv[3]);
            *reinterpret_cast<float4*>(Ys + tid * XS + 4 * q) = make_float4(yv[0], yv[1], yv[2], yv[3]);
            if constexpr (QZ) *reinterpret_cast<float4*>(Ys + QB * XS + tid * XS + 4 * q) = make_float4(zv[0], zv[1], zv[2], zv[3]);
          }
        }
        __syncthreads();
        {
          // ---- consumer: this thread's share of the batch into its 4 x 4 tile ----
          const bool diag = (q_ty == q_tx);
          const float* ysrc = (QZ && D == 4 && diag) ? Ys + QB * XS : Ys;
#pragma unroll 4
          for (int r = q_sub; r < QB; r += TPT) {
            const float4 x4 = *reinterpret_cast<const float4*>(Xs + r * XS + 4 * q_ty);
            const float4 y4 = *reinterpret_cast<const float4*>(ysrc + r * XS + 4 * q_tx);
            const float xv[4] = {x4.x, x4.y, x4.z, x4.w}, yv[4] = {y4.x, y4.y, y4.z, y4.w};
            float ys[4] = {yv[0], yv[1], yv[2], yv[3]};   // what the entries of a (j, j) block multiply
            if constexpr (QZ && D < 4) {
              const float4 z4 = *reinterpret_cast<const float4*>(Ys + QB * XS + r * XS + 4 * q_tx);
              const float zv[4] = {z4.x, z4.y, z4.z, z4.w};
#pragma unroll
              for (int j = 0; j < 4; ++j) ys[j] = diag ? zv[j] : yv[j];
            }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
              for (int j = 0; j < 4; ++j) acc4[i][j] = fmaf(-xv[i], (i / D == j / D) ? ys[j] : yv[j], acc4[i][j]);
          }
          // every 64 weights of this thread: move the sums to the second level
          if (++batches == (64 * TPT) / QB) {
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                acc4_hi[i][j] += acc4[i][j];
                acc4[i][j] = 0.f;
              }
#pragma unroll
            for (int o2 = 0; o2 < NDQ; ++o2) {
              dgt_hi[o2] += dgt[o2];
              dgt[o2] = 0.f;
            }
            batches = 0;
          }
        }
      }
      continue;
    }
#pragma unroll 1
    for (int b0 = 0; b0 < TILE; b0 += BATCH) {
      if (tbase + b0 >= rows) break;   // uniform over the block
      // ---- producer: warp `warp` takes weights 4 warp .. 4 warp + 3 of the batch; lane = centroid ----
      __syncthreads();   // the previous batch has been consumed
#pragma unroll
      for (int q = 0; q < BATCH / NWARP; ++q) {
        const int r = warp * (BATCH / NWARP) + q;
        const long long loc = tbase + b0 + r;
        const bool valid = (loc < rows);
        const long long grow = row0 + (valid ? loc : 0);
        float w[D];
        if constexpr (D == 4) {
          const float4 x = __ldg(reinterpret_cast<const float4*>(p.W + grow * 4));
          w[0] = x.x; w[1] = x.y; w[2] = x.z; w[3] = x.w;
        } else if constexpr (D == 2) {
          const float2 x = __ldg(reinterpret_cast<const float2*>(p.W + grow * 2));
          w[0] = x.x; w[1] = x.y;
        } else {
          w[0] = __ldg(p.W + grow);
        }
        float dist[CPL], rs[CPL], e[CPL];
        (void)rs;
        float lmin = 3.0e38f;
#pragma unroll
        for (int t = 0; t < CPL; ++t) {
          if constexpr (D == 1) {
            dist[t] = fabsf(w[0] - c[t][0]);
          } else {
            float sq = 1e-30f;
#pragma unroll
            for (int a = 0; a < D; ++a) {
              const float df = w[a] - c[t][a];
              sq = fmaf(df, df, sq);
            }
            rs[t] = rsqrt_approx(sq);
            dist[t] = sq * rs[t];
          }
          lmin = fminf(lmin, dist[t]);
        }
        const float mref = group_min<32>(lmin) * p.scale;
        float lsum = 0.f;
#pragma unroll
        for (int t = 0; t < CPL; ++t) {
          e[t] = ex2_approx(fmaf(-p.scale, dist[t], mref));
          lsum += e[t];
        }
        const float rr = valid ? rcp_approx(group_sum<32>(lsum)) : 0.f;
#pragma unroll
        for (int t = 0; t < CPL; ++t) {
          const int j = lane + 32 * t;
          const float at = e[t] * rr;
          float nn[D], pp[D];
#pragma unroll
          for (int a = 0; a < D; ++a) {
            const float df = w[a] - c[t][a];
            if constexpr (D == 1) nn[a] = (df > 0.f) ? 1.f : ((df < 0.f) ? -1.f : 0.f);
            else nn[a] = df * rs[t];
            pp[a] = at * ist[t] * (w[a] - fj[t][a]);
          }
          if (j < KP) {
#pragma unroll
            for (int a = 0; a < D; ++a) {
              Xs[r * KD + j * D + a] = pp[a];
              Ys[r * KD + j * D + a] = at * nn[a];
#pragma unroll
              for (int bb = 0; bb < D; ++bb) dg[t][a][bb] = fmaf(pp[a], nn[bb], dg[t][a][bb]);
            }
          }
        }
      }
      __syncthreads();
      // ---- consumer: every thread adds the batch's outer products into its corner ----
#pragma unroll 8
      for (int r = 0; r < BATCH; ++r) {
        float x[TR], y[TR];
#pragma unroll
        for (int i = 0; i < TR; ++i) {
          x[i] = Xs[r * KD + ty * TR + i];
          y[i] = Ys[r * KD + tx * TR + i];
        }
#pragma unroll
        for (int i = 0; i < TR; ++i)
#pragma unroll
          for (int j = 0; j < TR; ++j) acc[i][j] = fmaf(-x[i], y[j], acc[i][j]);
      }
      if (++batches == 2) {   // 64 weights: move the sums to the second level
#pragma unroll
        for (int i = 0; i < TR; ++i)
#pragma unroll
          for (int j = 0; j < TR; ++j) {
            acc_hi[i][j] += acc[i][j];
            acc[i][j] = 0.f;
          }
#pragma unroll
        for (int t = 0; t < CPL; ++t)
#pragma unroll
          for (int a = 0; a < D; ++a)
#pragma unroll
            for (int bb = 0; bb < D; ++bb) {
              dg_hi[t][a][bb] += dg[t][a][bb];
              dg[t][a][bb] = 0.f;
            }
        batches = 0;
      }
    }
  }
  grid_release_dependents();
  if (cur_layer >= 0 && layer_active) finish(cur_layer);
}

}  // namespace idkm
