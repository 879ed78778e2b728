// dk_decode_verify_static: decode + integrity check without any allocation.
//
// Some callers of this library are not allowed to allocate device memory at
// the point where they need the check: code that runs inside a memory pool
// with a fixed budget, inside a real-time or fault-handling section where
// cudaMalloc's implicit device synchronisation is not acceptable, or in a
// process that must not create a dk_ctx (dk_create allocates).  For them the
// scratch memory that the check needs (coefficient tables, per-group
// statistics, the counter and the candidate list) lives in one file-scope
// device array of fixed size that is part of the loaded library image.
#include <math.h>
#include <string.h>

#include "dk_internal.h"

namespace {

using dk::Candidate;

constexpr size_t kCoefFloats = 16384;                 // 64 KiB of coefficient tables
constexpr size_t kStatFloats = 16384;                 // 64 KiB: G*(K+3) statistics
constexpr size_t kCountFloats = 64;                   // the candidate counter (padded)
constexpr size_t kCandBytes = (size_t)dk::kCandCap * sizeof(Candidate);   // 1 MiB
constexpr size_t kScratchBytes = (kCoefFloats + kStatFloats + kCountFloats) * sizeof(float) + kCandBytes;

// In host code this name is only a handle for cudaGetSymbolAddress; it is not
// a device address and must never be handed to a kernel as it stands.
static __device__ __align__(256) unsigned char g_static_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
unsigned char* g_scratch_addr[kMaxDevices] = {nullptr};
int g_sm_count[kMaxDevices] = {0};

// Once per device, with that device current: resolve the array's device address.
dk_status setup_device(int device) {
  if (g_scratch_addr[device]) return DK_OK;
  void* p = nullptr;
  if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) return DK_ERR_CUDA;
  int sms = 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess)
    return DK_ERR_CUDA;
  g_sm_count[device] = sms;
  g_scratch_addr[device] = static_cast<unsigned char*>(p);
  return DK_OK;
}

// fp64 Gauss-Jordan with partial pivoting on an n x n block (n <= DK_MAX_K+1).
bool invert_block(const double* M, int n, double* inv) {
  double a[(DK_MAX_K + 1) * (DK_MAX_K + 1)];
  double big = 0.0;
  for (int i = 0; i < n * n; ++i) { a[i] = M[i]; big = fmax(big, fabs(M[i])); }
  if (!(big > 0.0) || !isfinite(big)) return false;
  for (int i = 0; i < n * n; ++i) inv[i] = (i / n == i % n) ? 1.0 : 0.0;
  for (int c = 0; c < n; ++c) {
    int piv = c;
    for (int r = c + 1; r < n; ++r)
      if (fabs(a[r * n + c]) > fabs(a[piv * n + c])) piv = r;
    if (!(fabs(a[piv * n + c]) > 1e-10 * big)) return false;
    for (int j = 0; j < n && piv != c; ++j) {
      double t = a[c * n + j]; a[c * n + j] = a[piv * n + j]; a[piv * n + j] = t;
      t = inv[c * n + j]; inv[c * n + j] = inv[piv * n + j]; inv[piv * n + j] = t;
    }
    const double ip = 1.0 / a[c * n + c];
    for (int j = 0; j < n; ++j) { a[c * n + j] *= ip; inv[c * n + j] *= ip; }
    for (int r = 0; r < n; ++r) {
      const double f = a[r * n + c];
      if (r == c || f == 0.0) continue;
      for (int j = 0; j < n; ++j) { a[r * n + j] -= f * a[c * n + j]; inv[r * n + j] -= f * inv[c * n + j]; }
    }
  }
  return true;
}

}  // namespace

extern "C" dk_status dk_decode_verify_static(int device, const dk_problem* p, const float* ybar,
                                             const float* C_host, const float* bias, float* y,
                                             dk_verdict* verdict, void* stream) {
  if (!p || !ybar || !C_host || !y || !verdict) return DK_ERR_INVALID_ARG;
  if (device < 0 || device >= kMaxDevices) return DK_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(ybar) | reinterpret_cast<uintptr_t>(y) |
       reinterpret_cast<uintptr_t>(verdict)) & 15)
    return DK_ERR_INVALID_ARG;
  dk::Geom g;
  dk_status s = dk::make_geom(p, &g);
  if (s != DK_OK) return s;
  const int K = g.K, K1 = K + 1, E = K + 2, G = g.G;
  const size_t n_dec = (size_t)G * K * K1, n_nul = (size_t)G * E;
  // limits of the fixed array: refuse clearly instead of overrunning it
  if (2 * n_dec + n_nul > kCoefFloats) return DK_ERR_WORKSPACE;
  if ((size_t)G * (E + 1) > kStatFloats) return DK_ERR_WORKSPACE;

  int prev = -1;
  if (cudaGetDevice(&prev) != cudaSuccess) return DK_ERR_CUDA;
  if (prev != device && cudaSetDevice(device) != cudaSuccess) return DK_ERR_CUDA;
  s = setup_device(device);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // The coefficient tables below are copied from this call's stack frame; a
  // copy recorded by a stream capture would read the frame after it is gone.
  if (s == DK_OK) {
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &cap) != cudaSuccess) s = DK_ERR_CUDA;
    else if (cap != cudaStreamCaptureStatusNone) s = DK_ERR_UNSUPPORTED;
  }
  if (s == DK_OK) {
    // decode rows (two-float split of the fp64 inverse) and null vector, on the stack
    float tab[kCoefFloats];
    float* h_dec = tab;
    float* h_decl = tab + n_dec;
    float* h_nul = tab + 2 * n_dec;
    double sq[(DK_MAX_K + 1) * (DK_MAX_K + 1)], inv[(DK_MAX_K + 1) * (DK_MAX_K + 1)];
    for (int gi = 0; gi < G && s == DK_OK; ++gi) {
      const float* Cg = C_host + (size_t)gi * E * K1;
      for (int i = 0; i < K1 * K1; ++i) sq[i] = (double)Cg[i];
      if (!invert_block(sq, K1, inv)) { s = DK_ERR_SINGULAR; break; }
      for (int k = 0; k < K; ++k)
        for (int i = 0; i < K1; ++i) {
          const double v = inv[k * K1 + i];
          const float hi = (float)v;
          h_dec[((size_t)gi * K + k) * K1 + i] = hi;
          h_decl[((size_t)gi * K + k) * K1 + i] = (float)(v - (double)hi);
        }
      for (int i = 0; i < K1; ++i) {
        double acc = 0.0;
        for (int k = 0; k < K1; ++k) acc += (double)Cg[(size_t)K1 * K1 + k] * inv[k * K1 + i];
        h_nul[(size_t)gi * E + i] = (float)(-acc);
      }
      h_nul[(size_t)gi * E + K1] = 1.f;
    }
    if (s == DK_OK) {
      unsigned char* base = g_scratch_addr[device];
      float* d_tab = reinterpret_cast<float*>(base);
      float* d_stat = d_tab + kCoefFloats;
      // the host table is pageable: the copy has been staged when this returns
      if (cudaMemcpyAsync(d_tab, tab, (2 * n_dec + n_nul) * sizeof(float), cudaMemcpyHostToDevice,
                          st) != cudaSuccess)
        s = DK_ERR_CUDA;
      dk::CoefView cv;
      cv.enc = nullptr;
      cv.dec = d_tab;
      cv.decl = d_tab + n_dec;
      cv.nul = d_tab + 2 * n_dec;
      cv.dmix = nullptr;
      cv.chunk_cap = 8;
      cv.chunk_tab = nullptr;
      dk::VerifyScratch vs;
      vs.sumsq = d_stat;
      vs.maxrho = reinterpret_cast<int*>(d_stat + (size_t)G * E);
      vs.count = reinterpret_cast<unsigned int*>(d_stat + kStatFloats);
      vs.cand = reinterpret_cast<Candidate*>(base + (kCoefFloats + kStatFloats + kCountFloats) * sizeof(float));
      // the array keeps the previous call's statistics, counter and candidates:
      // verify_begin clears what must start at zero
      if (s == DK_OK) s = dk::launch_verify_begin(g, vs, st);
      if (s == DK_OK) s = dk::launch_decode_verify(g, ybar, cv, bias, y, vs, g_sm_count[device], st);
      if (s == DK_OK) s = dk::launch_verify_finalize(g, cv.nul, vs, verdict, st);
    }
  }
  if (prev != device) cudaSetDevice(prev);
  return s;
}
