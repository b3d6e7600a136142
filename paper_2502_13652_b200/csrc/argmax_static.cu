// c2t_row_argmax_static: the arg-max pass with its scratch memory in a fixed device array of
// this library, for callers that cannot allocate device memory.  See include/c2t.h.
#include <mutex>

#include "c2t_internal.h"

namespace c2t {
namespace {

constexpr int kStaticMaxRows = C2T_STATIC_MAX_ROWS;
constexpr int kStaticMaxVocab = C2T_STATIC_MAX_VOCAB;
// slots per row the arg-max pass can need at the largest vocabulary (fp32: 4 elements per vector)
constexpr int kStaticMaxSplits = (kStaticMaxVocab / 4 + kMinSpanVectors - 1) / kMinSpanVectors + 1;
constexpr int kMaxDevices = 64;
// the arg-max kernel keeps one row offset per "sequence" in shared memory, sized by the batch limit
static_assert(C2T_STATIC_MAX_ROWS <= C2T_MAX_BATCH, "the static entry point passes its rows as the batch of the pass");

struct StaticScratch {
  PassInfo info;                                              // what the pass derived from the row counts
  int32_t counts[kStaticMaxRows];                             // one active row per "sequence"
  unsigned long long best[(size_t)kStaticMaxRows * kStaticMaxSplits];   // best key per (row, split)
};

// The scratch itself.  Every GPU that loads the library holds these ~2.1 MB until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[sizeof(StaticScratch)];

// Host side: the array's name is only a handle here; the device address comes from
// cudaGetSymbolAddress, once per device, with that device current.
struct PerDevice {
  StaticScratch *scratch = nullptr;
  int grid = 0;
};
PerDevice g_dev[kMaxDevices];
std::mutex g_dev_mutex;

__global__ void static_prepare_kernel(StaticScratch *s, int rows, int max_splits) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < rows) s->counts[i] = 1;
  // stale keys of an earlier call must never be taken for this call's
  for (size_t k = i; k < (size_t)rows * max_splits; k += (size_t)gridDim.x * blockDim.x) s->best[k] = 0ull;
}

__global__ void static_finish_kernel(const StaticScratch *s, int rows, int max_splits, int32_t *out) {
  const int a = blockIdx.x * blockDim.x + threadIdx.x;
  if (a >= rows) return;
  const PassInfo info = s->info;
  const long long first_vec = (long long)a * info.vec_per_row;
  const int c_first = (int)(first_vec / info.span);
  const int c_last = (int)((first_vec + info.vec_per_row - 1) / info.span);
  int n_splits = c_last - c_first + 1;
  if (n_splits > max_splits) n_splits = max_splits;
  unsigned long long best = 0ull;
  for (int k = 0; k < n_splits; ++k) {
    const unsigned long long key = s->best[(size_t)a * max_splits + k];
    best = key > best ? key : best;
  }
  out[a] = best ? key_token(best) : -1;
}

}  // namespace
}  // namespace c2t

using namespace c2t;

extern "C" int c2t_row_argmax_static(const void *logits_dev, int32_t rows, int32_t vocab, int32_t dtype,
                                     int64_t row_stride, int32_t *argmax_dev, void *stream) {
  if (!logits_dev || !argmax_dev || rows < 1 || vocab < 1) return C2T_EINVAL;
  if (dtype != C2T_F32 && dtype != C2T_BF16) return C2T_EINVAL;
  if (rows > kStaticMaxRows || vocab > kStaticMaxVocab) return C2T_ERANGE;   // beyond the fixed scratch
  if (row_stride < vocab) return C2T_EINVAL;
  const int eb = dtype == C2T_BF16 ? 2 : 4;
  if ((reinterpret_cast<uintptr_t>(logits_dev) & 15) || (row_stride * eb) % 16) return C2T_EALIGN;

  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { cudaGetLastError(); return C2T_ECUDA; }
  PerDevice pd;
  {
    std::lock_guard<std::mutex> lock(g_dev_mutex);
    if (!g_dev[dev].scratch) {   // first call on this device: look the array's device address up
      void *ptr = nullptr;
      int sms = 0;
      if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr ||
          cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) {
        cudaGetLastError();
        return C2T_ECUDA;
      }
      g_dev[dev].scratch = static_cast<StaticScratch *>(ptr);
      g_dev[dev].grid = sms * kPassCtasPerSm;
    }
    pd = g_dev[dev];
  }

  cudaStream_t s = (cudaStream_t)stream;
  const int max_splits = max_splits_for(vocab, eb, pd.grid, 0);   // <= kStaticMaxSplits by the limits above
  static_prepare_kernel<<<(rows + 255) / 256, 256, 0, s>>>(pd.scratch, rows, max_splits);
  if (cudaGetLastError() != cudaSuccess) return C2T_ECUDA;

  PassParams p;
  memset(&p, 0, sizeof p);
  p.logits = logits_dev;
  p.seq_stride = row_stride;      // every row is a "sequence" with one active row
  p.row_stride = row_stride;
  p.V = vocab; p.K = 1; p.B = rows; p.rows_per_seq_max = 1;
  p.counts = pd.scratch->counts;  // address arithmetic on a device pointer, never dereferenced here
  p.max_splits = max_splits;
  p.n_slots = (int64_t)rows * max_splits;
  p.info = &pd.scratch->info;
  p.part_best = pd.scratch->best;
  if (launch_argmax_pass(p, dtype, pd.grid, s) != cudaSuccess) return C2T_ECUDA;

  static_finish_kernel<<<(rows + 255) / 256, 256, 0, s>>>(pd.scratch, rows, max_splits, argmax_dev);
  if (cudaGetLastError() != cudaSuccess) return C2T_ECUDA;
  return C2T_OK;
}
