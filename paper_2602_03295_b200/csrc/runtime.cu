// Host-side runtime pieces shared by all kernels: the device status word, the launch counter and
// tensor-map encoding through the driver entry point.
#include "common.cuh"

#include <cstdlib>

#include <atomic>
#include <mutex>
#include <vector>

namespace pop {

static __device__ int g_status_word = 0;

int* status_word() {
  // one address per device; the library is used with one device per process
  static int* ptr = nullptr;
  static int ptr_dev = -1;
  int dev = 0;
  cudaGetDevice(&dev);
  if (ptr == nullptr || dev != ptr_dev) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_status_word) != cudaSuccess) return nullptr;
    ptr = static_cast<int*>(p);
    ptr_dev = dev;
  }
  return ptr;
}

int read_and_clear_status(cudaStream_t s) {
  if (cudaStreamSynchronize(s) != cudaSuccess) return POP_E_CUDA;
  int v = 0;
  if (cudaMemcpyFromSymbol(&v, g_status_word, sizeof(int)) != cudaSuccess) return POP_E_CUDA;
  if (v != 0) {
    int zero = 0;
    if (cudaMemcpyToSymbol(g_status_word, &zero, sizeof(int)) != cudaSuccess) return POP_E_CUDA;
  }
  if (cudaGetLastError() != cudaSuccess) return POP_E_CUDA;
  return v;
}

static std::atomic<int64_t> g_launches{0};
void count_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }
int64_t launch_count() { return g_launches.load(std::memory_order_relaxed); }
void reset_launch_count() { g_launches.store(0, std::memory_order_relaxed); }

struct ProfRecord { cudaEvent_t e0, e1; double work; };
static std::atomic<bool> g_prof_on{false};
static std::mutex g_prof_mu;
static std::vector<ProfRecord> g_prof[PROF_KINDS];

void prof_enable(bool on) { g_prof_on.store(on); }
bool prof_enabled() { return g_prof_on.load(std::memory_order_relaxed); }

bool chained_launch_enabled() {
  static const bool on = [] {
    const char* e = std::getenv("POP_CHAINED_LAUNCH");
    return !(e && e[0] == '0');
  }();
  return on;
}

ProfScope::ProfScope(int kind_, double work_, cudaStream_t s)
    : kind(kind_), work(work_), stream(s), e0(nullptr), e1(nullptr), active(false) {
  if (!prof_enabled()) return;
  if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) return;
  active = true;
  cudaEventRecord(e0, stream);
}
ProfScope::~ProfScope() {
  if (!active) return;
  cudaEventRecord(e1, stream);
  std::lock_guard<std::mutex> lk(g_prof_mu);
  g_prof[kind].push_back({e0, e1, work});
}

int prof_summary(int kind, double* total_ms, double* total_work, int64_t* launches) {
  if (kind < 0 || kind >= PROF_KINDS) return POP_E_INVALID;
  std::lock_guard<std::mutex> lk(g_prof_mu);
  double ms = 0, work = 0;
  for (auto& r : g_prof[kind]) {
    float t = 0;
    if (cudaEventSynchronize(r.e1) != cudaSuccess || cudaEventElapsedTime(&t, r.e0, r.e1) != cudaSuccess)
      return POP_E_CUDA;
    ms += t;
    work += r.work;
    cudaEventDestroy(r.e0);
    cudaEventDestroy(r.e1);
  }
  if (total_ms) *total_ms = ms;
  if (total_work) *total_work = work;
  if (launches) *launches = (int64_t)g_prof[kind].size();
  g_prof[kind].clear();
  return POP_OK;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  });
  return fn;
}

int make_tmap_bf16_3d(CUtensorMap* out, const void* base, uint64_t dim0, uint64_t dim1, uint64_t dim2,
                      uint64_t stride1_elems, uint64_t stride2_elems, uint32_t box0, uint32_t box1) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return POP_E_CUDA;
  cuuint64_t dims[3] = {dim0, dim1, dim2};
  cuuint64_t strides[2] = {stride1_elems * 2, stride2_elems * 2};
  cuuint32_t box[3] = {box0, box1, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? POP_OK : POP_E_CUDA;
}

int make_tmap_u8_3d(CUtensorMap* out, const void* base, uint64_t dim0, uint64_t dim1, uint64_t dim2,
                    uint64_t stride1_bytes, uint64_t stride2_bytes, uint32_t box1) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return POP_E_CUDA;
  cuuint64_t dims[3] = {dim0, dim1, dim2};
  cuuint64_t strides[2] = {stride1_bytes, stride2_bytes};
  cuuint32_t box[3] = {128, box1, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? POP_OK : POP_E_CUDA;
}

int make_tmap_f32_3d(CUtensorMap* out, const void* base, uint64_t dim0, uint64_t dim1, uint64_t dim2,
                     uint64_t stride1_elems, uint64_t stride2_elems, uint32_t box1) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return POP_E_CUDA;
  cuuint64_t dims[3] = {dim0, dim1, dim2};
  cuuint64_t strides[2] = {stride1_elems * 4, stride2_elems * 4};
  cuuint32_t box[3] = {32, box1, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? POP_OK : POP_E_CUDA;
}

int make_tmap_bf16_nd(CUtensorMap* out, const void* base, int rank, const uint64_t dims[5],
                      const uint64_t strides_elems[4], const uint32_t box[5]) {
  EncodeTiledFn fn = encode_fn();
  if (!fn || rank < 3 || rank > 5) return POP_E_CUDA;
  cuuint64_t d[5], st[4];
  cuuint32_t b[5], estr[5] = {1, 1, 1, 1, 1};
  for (int i = 0; i < 5; ++i) {
    d[i] = dims[i];
    b[i] = box[i];
  }
  for (int i = 0; i < 4; ++i) st[i] = strides_elems[i] * 2;
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), d, st, b, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? POP_OK : POP_E_CUDA;
}

}  // namespace pop
