// asd_denoise_static: the network drift for a handful of rows, with the activation scratch of the
// GEMM chain (input rows, two ping-pong hidden buffers, a row counter) taken from a fixed array that
// lives in the library image instead of from cudaMalloc'd workspaces.  See include/asd.h.
#include <string.h>

#include "asd_internal.h"

using namespace asd;

struct asd_ctx {
  Ctx c;
};

namespace {

constexpr size_t kStaticBytes = 8u << 20;  // ASD_STATIC_SCRATCH_BYTES
constexpr size_t kHeaderBytes = 256;       // row counter lives here
constexpr int kMaxDevices = 64;

// The scratch itself.  In host code this name is only a handle for the runtime (not a device
// address), so the host never passes it to a kernel: it asks the runtime for the device address.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

// Device address of g_static_scratch per device ordinal, resolved on first use on that device.
unsigned char* g_scratch_addr[kMaxDevices] = {};

asd_status fail(Ctx* c, asd_status st, const char* msg) {
  c->err = msg;
  return st;
}

size_t round256(size_t x) { return (x + 255) / 256 * 256; }

}  // namespace

extern "C" asd_status asd_denoise_static_max_rows(const asd_ctx* ctx, int32_t* max_rows_out) {
  if (!ctx || !max_rows_out) return ASD_ERR_INVALID_ARG;
  const Ctx* c = &ctx->c;
  *max_rows_out = 0;
  if (c->kind != ASD_DEN_RESMLP_BF16) return ASD_ERR_UNSUPPORTED;
  const size_t per_row = ((size_t)c->mlp.in_pad + 2 * (size_t)c->mlp.width) * sizeof(__nv_bfloat16);
  // three sub-buffers, each rounded up to 256 bytes
  const size_t usable = kStaticBytes - kHeaderBytes - 3 * 256;
  *max_rows_out = (int32_t)(usable / per_row);
  return ASD_OK;
}

extern "C" asd_status asd_denoise_static(asd_ctx* ctx, int32_t n_rows, const int32_t* step_dev, const float* y_dev,
                                         const int32_t* slot_dev, float* out_dev) {
  if (!ctx) return ASD_ERR_INVALID_ARG;
  Ctx* c = &ctx->c;
  if (c->kind != ASD_DEN_RESMLP_BF16)
    return fail(c, ASD_ERR_UNSUPPORTED, "asd_denoise_static: only the network drift uses scratch; call asd_denoise");
  int32_t max_rows = 0;
  asd_denoise_static_max_rows(ctx, &max_rows);
  if (n_rows < 0 || n_rows > max_rows)
    return fail(c, ASD_ERR_INVALID_ARG, "asd_denoise_static: n_rows exceeds what the fixed scratch array holds "
                                        "(see asd_denoise_static_max_rows)");
  if (n_rows == 0) return ASD_OK;
  if (!step_dev || !y_dev || !out_dev) return fail(c, ASD_ERR_INVALID_ARG, "step_dev, y_dev, out_dev required");
  if (c->mlp.d_cond > 0 && !slot_dev) return fail(c, ASD_ERR_INVALID_ARG, "slot_dev required (d_cond > 0)");
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev != c->device)
    return fail(c, ASD_ERR_STATE, "asd_denoise_static: the context's device must be current");
  if (dev < 0 || dev >= kMaxDevices) return fail(c, ASD_ERR_UNSUPPORTED, "device ordinal too large");

  // One-time set-up per device: resolve the device address of the scratch array.
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    const cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess || !p) return fail(c, ASD_ERR_CUDA, "cudaGetSymbolAddress(static scratch) failed");
    g_scratch_addr[dev] = static_cast<unsigned char*>(p);
  }
  unsigned char* base = g_scratch_addr[dev];

  // Carve the array for the largest supported row count, so the layout (and with it the cached TMA
  // descriptors) is the same for every call: [row counter | X | H0 | H1]
  const size_t x_bytes = round256((size_t)max_rows * c->mlp.in_pad * sizeof(__nv_bfloat16));
  const size_t h_bytes = round256((size_t)max_rows * c->mlp.width * sizeof(__nv_bfloat16));
  int* n_dev = reinterpret_cast<int*>(base);
  __nv_bfloat16* X = reinterpret_cast<__nv_bfloat16*>(base + kHeaderBytes);
  __nv_bfloat16* H0 = reinterpret_cast<__nv_bfloat16*>(base + kHeaderBytes + x_bytes);
  __nv_bfloat16* H1 = reinterpret_cast<__nv_bfloat16*>(base + kHeaderBytes + x_bytes + h_bytes);
  if (kHeaderBytes + x_bytes + 2 * h_bytes > kStaticBytes) return fail(c, ASD_ERR_INVALID_ARG, "scratch overflow");

  // The array keeps whatever the previous call left.  The row counter is rewritten here; X, H0 and H1
  // are fully overwritten for rows < n_rows before they are read (pack kernel, then each layer's
  // epilogue), and rows >= n_rows are never stored from, so nothing else has to start at zero.
  if (cudaMemcpyAsync(n_dev, &n_rows, sizeof(int), cudaMemcpyHostToDevice, c->stream) != cudaSuccess)
    return fail(c, ASD_ERR_CUDA, "asd_denoise_static: copying the row count failed");

  // Point the GEMM chain at the static buffers for the duration of this call.
  const MlpParams saved = c->mlp;
  c->mlp.X = X;
  c->mlp.H[0] = H0;
  c->mlp.H[1] = H1;
  c->mlp.row_cap = max_rows;
  RowSet rs{n_dev, n_rows, y_dev, nullptr, step_dev, slot_dev};
  launch_pack(c, rs);
  const asd_status st = mlp_forward(c, rs, out_dev, 2);
  c->mlp = saved;
  if (st != ASD_OK) return st;
  if (cudaGetLastError() != cudaSuccess) return fail(c, ASD_ERR_CUDA, "asd_denoise_static: launch failed");
  // wait for the result and read the device error word (bounded waits in the GEMM kernels)
  if (cudaMemcpyAsync(c->counters_host, c->counters, sizeof(RoundCounters), cudaMemcpyDeviceToHost, c->stream) !=
          cudaSuccess ||
      cudaStreamSynchronize(c->stream) != cudaSuccess)
    return fail(c, ASD_ERR_CUDA, "asd_denoise_static: sync failed");
  if (c->counters_host->err != 0) {
    cudaMemsetAsync(&c->counters->err, 0, sizeof(int), c->stream);
    return fail(c, ASD_ERR_TIMEOUT, "a bounded device-side wait ran out (kernel returned early)");
  }
  return ASD_OK;
}
