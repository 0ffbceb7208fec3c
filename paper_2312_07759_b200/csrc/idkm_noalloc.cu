// idkm_step_noalloc: one application of the soft k-means map with no allocation anywhere.
//
// Some callers of this library run where device memory cannot be requested at all: inside a
// memory-pool or allocator callback, in a process whose whole device budget was handed out at start-up
// (an inference server with a fixed arena), or in a plug-in that is forbidden to touch the CUDA
// allocator of its host application.  The regular entry points ask such a caller for a workspace
// buffer, which it has no way to provide.  This entry point instead keeps the few hundred KB of
// bookkeeping the fused step needs (per-block partial sums, the ticket and iteration state) in a
// fixed array that is part of the library image itself.
#include "idkm_kernels.cuh"

#include <math.h>
#include <string.h>

#include <mutex>

#include "../../include/idkm.h"

namespace idkm {

// The scratch lives in the module's global memory: every GPU that loads the library holds these bytes
// until the process exits, whether or not the entry point is ever called.
constexpr size_t NOALLOC_SCRATCH_BYTES = IDKM_NOALLOC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_noalloc_scratch[NOALLOC_SCRATCH_BYTES];

constexpr int NOALLOC_MAX_DEVICES = 64;
// Resident blocks per SM this entry point launches at most.  The partial-sum rows of the largest codebook
// (d = 4, k = 256: 10 KB each) times (blocks + 1), plus the group rows, must fit the fixed array: two blocks per SM
// on a 148-SM part need 3.3 MB of the 4 MiB, whatever register count the compiler gives the kernels.
constexpr int NOALLOC_BLOCKS_PER_SM = 2;
struct NoallocDevice {
  bool ready;
  unsigned char* scratch;   // DEVICE address of g_noalloc_scratch on that device
  int sms;
};
static NoallocDevice g_noalloc_dev[NOALLOC_MAX_DEVICES];
static std::mutex g_noalloc_mu;   // guards the table above: two host threads may make their first call together

// Looks up (once per device, with that device current) the device address of the built-in array and the SM count.
static int noalloc_device(NoallocDevice* out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= NOALLOC_MAX_DEVICES) return IDKM_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_noalloc_mu);
  NoallocDevice& nd = g_noalloc_dev[dev];
  if (!nd.ready) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || ptr == nullptr) {
      (void)cudaGetLastError();
      return IDKM_ERR_CUDA;
    }
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) return IDKM_ERR_CUDA;
    nd.scratch = static_cast<unsigned char*>(ptr);
    nd.sms = sms;
    nd.ready = true;
  }
  *out = nd;
  return IDKM_OK;
}

// Resets the single layer's state and seeds C_out with the starting centroids.  The scratch keeps
// whatever the previous call left, so everything the step reads before writing is set here.
__global__ void idkm_noalloc_init(LayerState* st, const float* C_in, float* C_out, int k, int d, double inv_tau,
                                  unsigned int* gtickets, int n_groups) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  for (int o = i; o < n_groups; o += gridDim.x * blockDim.x) gtickets[o] = 0u;
  if (i == 0) {
    LayerState s;
    memset(&s, 0, sizeof(s));
    s.status = ST_OK;
    s.adj_prev = 3.0e38f;
    double box2 = 0.0;
    for (int a = 0; a < d; ++a) {
      double lo = 1e300, hi = -1e300;
      for (int j = 0; j < k; ++j) {
        const double v = (double)C_in[j * d + a];
        lo = fmin(lo, v);
        hi = fmax(hi, v);
      }
      box2 += (hi - lo) * (hi - lo);
    }
    s.precise[0] = s.precise[1] = (sqrt(box2) * inv_tau <= PRECISE_SPAN) ? 1 : 0;
    *st = s;
  }
  if (C_in != C_out)
    for (int o = i; o < k * d; o += gridDim.x * blockDim.x) C_out[o] = C_in[o];
}

static int noalloc_table(const KernelEntry* e, int64_t m, int sms, LayerTable* lt) {
  memset(lt, 0, sizeof(*lt));
  const long long tiles = (m + e->tile - 1) / e->tile;
  if (tiles > 0x3fffffffLL) return IDKM_ERR_SHAPE;
  lt->n_layers = 1;
  lt->row_off[0] = 0;
  lt->tile_off[0] = 0;
  for (int l = 1; l <= MAX_LAYERS; ++l) {
    lt->row_off[l] = m;
    lt->tile_off[l] = (l == 1) ? (int)tiles : 0x7fffffff;
  }
  lt->tiles_total = (int)tiles;
  int per_sm = 0;
  // static + dynamic shared memory can exceed the 48 KB default: raise the limit before asking for the occupancy
  if (e->dyn_smem > 0) (void)cudaFuncSetAttribute(e->func, cudaFuncAttributeMaxDynamicSharedMemorySize, e->dyn_smem);
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, e->func, BLOCK, e->dyn_smem) != cudaSuccess || per_sm < 1) {
    (void)cudaGetLastError();
    per_sm = 1;
  }
  if (per_sm > NOALLOC_BLOCKS_PER_SM) per_sm = NOALLOC_BLOCKS_PER_SM;
  long long nb = (long long)sms * per_sm;
  if (nb > tiles) nb = tiles;
  lt->n_blocks = (int)nb;
  return IDKM_OK;
}

}  // namespace idkm

using namespace idkm;

extern "C" int idkm_step_noalloc(const float* W, int64_t m, int d, const float* C_in, int k, float tau, float* C_out,
                                 void* cuda_stream) {
  if (!W || !C_in || !C_out) return IDKM_ERR_NULL;
  if (!(d == 1 || d == 2 || d == 4) || k < 1 || k > IDKM_MAX_K) return IDKM_ERR_UNSUPPORTED;
  if (m < 1) return IDKM_ERR_SHAPE;
  if (!(tau > 0.f) || !isfinite(tau)) return IDKM_ERR_PARAM;
  if (((uintptr_t)W | (uintptr_t)C_in | (uintptr_t)C_out) & 15u) return IDKM_ERR_ALIGN;

  // once per device, with that device current: turn the symbol into a device address
  NoallocDevice nd;
  const int rc_dev = noalloc_device(&nd);
  if (rc_dev != IDKM_OK) return rc_dev;

  const int f32 = pick_family(STEP, d, k), f64 = pick_family(STEP_PRECISE, d, k);
  if (f32 < 0 || f64 < 0) return IDKM_ERR_UNSUPPORTED;
  const KernelEntry* e32 = kernel_entry(STEP, d, f32);
  const KernelEntry* e64 = kernel_entry(STEP_PRECISE, d, f64);

  PassParams p;
  memset(&p, 0, sizeof(p));
  PassParams q;
  int rc = noalloc_table(e32, m, nd.sms, &p.lt);
  if (rc != IDKM_OK) return rc;
  LayerTable lt64;
  rc = noalloc_table(e64, m, nd.sms, &lt64);
  if (rc != IDKM_OK) return rc;

  // layout of the fixed scratch: [state 256 B][group counters 1 KB][partials][group partials] of whichever step
  // kernel runs (the two never run for the same layer in one call)
  const int nb_max = p.lt.n_blocks > lt64.n_blocks ? p.lt.n_blocks : lt64.n_blocks;
  const int plen_max = e32->plen > e64->plen ? e32->plen : e64->plen;
  const int n_groups = (nb_max + 1) / RED_GROUP + 3;
  // bytes: 256 (state) + 1024 (group counters) + (nb_max + 1) partial rows + n_groups group rows of plen_max doubles
  const size_t off_gt = 256, off_part = off_gt + 1024;
  const size_t off_gpart = off_part + sizeof(double) * (size_t)(nb_max + 1) * plen_max;
  const size_t need = off_gpart + sizeof(double) * (size_t)n_groups * plen_max;
  if (n_groups * sizeof(unsigned int) > 1024 || need > NOALLOC_SCRATCH_BYTES) return IDKM_ERR_NOALLOC_TOO_LARGE;

  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  p.W = W;
  p.C = C_out;
  p.st = reinterpret_cast<LayerState*>(nd.scratch);
  p.partials = reinterpret_cast<double*>(nd.scratch + off_part);
  p.gpartials = reinterpret_cast<double*>(nd.scratch + off_gpart);
  p.gtickets = reinterpret_cast<unsigned int*>(nd.scratch + off_gt);
  // the single step writes one residual: it lands in the unused tail of the 256-byte state area
  p.hist_fwd = reinterpret_cast<float*>(nd.scratch + 128);
  p.hist_adj = p.hist_fwd;
  p.inv_tau = (float)(1.0 / (double)tau);
  p.inv_tau_d = 1.0 / (double)tau;
  p.scale = (float)(1.4426950408889634 / (double)tau);
  p.alpha = 1.f;
  p.k = k;
  p.tol = 0.f;
  p.max_iter = 1;
  p.iter = 0;
  q = p;
  q.lt = lt64;

  idkm_noalloc_init<<<(k * d + 255) / 256, 256, 0, stream>>>(p.st, C_in, C_out, k, d, p.inv_tau_d, p.gtickets, n_groups);
  if (cudaGetLastError() != cudaSuccess) return IDKM_ERR_CUDA;
  if (e32->launch(p, p.lt.n_blocks, stream) != cudaSuccess) return IDKM_ERR_CUDA;
  if (e64->launch(q, q.lt.n_blocks, stream) != cudaSuccess) return IDKM_ERR_CUDA;
  return IDKM_OK;
}

// The status word the last idkm_step_noalloc on this device left in the built-in array (IDKM_OK, or
// IDKM_ERR_NONFINITE when W, C_in or the sums held a NaN / Inf): one 4-byte copy to the host, no allocation.
extern "C" int idkm_step_noalloc_status(int* status_host_out, void* cuda_stream) {
  if (!status_host_out) return IDKM_ERR_NULL;
  NoallocDevice nd;
  const int rc_dev = noalloc_device(&nd);
  if (rc_dev != IDKM_OK) return rc_dev;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  const LayerState* st = reinterpret_cast<const LayerState*>(nd.scratch);
  int status = 0;
  if (cudaMemcpyAsync(&status, &st->status, sizeof(int), cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
      cudaStreamSynchronize(stream) != cudaSuccess) {
    (void)cudaGetLastError();
    return IDKM_ERR_CUDA;
  }
  *status_host_out = status;
  return IDKM_OK;
}
