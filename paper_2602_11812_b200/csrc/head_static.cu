// egtp_head_forward_static: the prediction head for callers that must not allocate.
//
// Some users of this library run inside a component that owns all device memory itself and
// forbids any other allocation while it serves requests: an inference engine whose memory pool was
// sized up front, a plugin called from inside someone else's runtime, or a process whose memory
// budget is fixed at start-up.  For them cudaMalloc (and therefore egtp_create, which sizes its
// workspace with cudaMalloc) is not an option.  The head's first layer needs scratch for its
// split-K partial sums; here that scratch is a fixed array that is part of the loaded library
// image, so the call itself allocates nothing.  See include/egtp.h for the contract.
#include "../../include/egtp.h"
#include "kernels.h"

#include <cuda_runtime.h>

#include <mutex>

using namespace egtp;

namespace {

constexpr int64_t kStaticPartialFloats = 1ll << 20;   // 4 MiB of split-K partial sums
constexpr int kStatusFloats = 64;                     // first 256 bytes: the device status word
constexpr int kMaxDevices = 64;

// Lives in every GPU's memory for as long as the library is loaded there.
static __device__ __align__(256) float g_head_scratch[kStatusFloats + kStaticPartialFloats];

struct DeviceSetup {
  bool ready = false;
  float* scratch = nullptr;   // device address of g_head_scratch on that device
  int num_sms = 0;
};
DeviceSetup g_setup[kMaxDevices];
std::mutex g_setup_mutex;

// Once per device, with that device current: resolve the array's device address.  In host code
// `g_head_scratch` itself is only a handle for the runtime, never something a kernel may be given.
int setup_current_device(int device, DeviceSetup* out) {
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  DeviceSetup& s = g_setup[device];
  if (!s.ready) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_head_scratch) != cudaSuccess || ptr == nullptr) {
      cudaGetLastError();
      return EGTP_ERR_CUDA;
    }
    int sms = 0, major = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess ||
        cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device) != cudaSuccess) {
      cudaGetLastError();
      return EGTP_ERR_CUDA;
    }
    if (major != 10) return EGTP_ERR_UNSUPPORTED;
    s.scratch = static_cast<float*>(ptr);
    s.num_sms = sms;
    s.ready = true;
  }
  *out = s;
  return EGTP_OK;
}

}  // namespace

extern "C" int egtp_head_forward_static(const egtp_head* head, const float* z, int64_t ldz, int32_t rows,
                                        float* y_out, float* phat_out, void* stream_v) {
  if (!head || !z || !y_out || rows < 0) return EGTP_ERR_INVALID_ARG;
  if (rows == 0) return EGTP_OK;
  if (!head->W1 || !head->b1 || !head->W2 || !head->b2) return EGTP_ERR_INVALID_ARG;
  if (head->d <= 0 || head->m_h <= 0 || head->d_out <= 0 || ldz < head->d) return EGTP_ERR_INVALID_ARG;
  if (head->wdtype != EGTP_F32 && head->wdtype != EGTP_BF16) return EGTP_ERR_UNSUPPORTED;
  if (head->mode == EGTP_HEAD_SCALAR) {
    if (head->d_out != 1) return EGTP_ERR_INVALID_ARG;
  } else if (head->mode == EGTP_HEAD_BINS) {
    if (!head->centres) return EGTP_ERR_INVALID_ARG;
  } else {
    return EGTP_ERR_INVALID_ARG;
  }
  if (head->m_h > 8192 || head->d_out > 256 || head->d % 16 != 0 || ldz % 4 != 0) return EGTP_ERR_UNSUPPORTED;
  if (reinterpret_cast<uintptr_t>(z) % 16 != 0 || reinterpret_cast<uintptr_t>(head->W1) % 16 != 0)
    return EGTP_ERR_UNSUPPORTED;
  // the scratch must hold at least one full set of layer-1 sums: rows * m_h floats
  if (static_cast<int64_t>(rows) * head->m_h > kStaticPartialFloats) return EGTP_ERR_CAPACITY;

  int device = 0;
  if (cudaGetDevice(&device) != cudaSuccess) return EGTP_ERR_CUDA;
  if (device < 0 || device >= kMaxDevices) return EGTP_ERR_UNSUPPORTED;
  DeviceSetup s;
  int rc = setup_current_device(device, &s);
  if (rc != EGTP_OK) return rc;

  HeadArgs ha{};
  ha.W1 = head->W1; ha.b1 = head->b1; ha.W2 = head->W2; ha.b2 = head->b2; ha.centres = head->centres;
  ha.d = head->d; ha.m_h = head->m_h; ha.d_out = head->d_out;
  ha.bf16 = head->wdtype == EGTP_BF16; ha.mode = head->mode;
  const int splits = head_pick_splits(rows, ha.d, ha.m_h, s.num_sms, kStaticPartialFloats);
  if (splits <= 0) return EGTP_ERR_CAPACITY;

  cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
  int32_t* status = reinterpret_cast<int32_t*>(s.scratch);
  float* partial = s.scratch + kStatusFloats;
  // The array keeps whatever the previous call left.  Only the status word the kernels consult has
  // to start at zero; every partial sum that layer 2 reads is written by layer 1 of this call first.
  if (cudaMemsetAsync(status, 0, sizeof(int32_t), stream) != cudaSuccess) return EGTP_ERR_CUDA;
  if (launch_head_hidden(ha, z, ldz, rows, splits, partial, status, stream) != cudaSuccess) return EGTP_ERR_CUDA;
  if (launch_head_out(ha, partial, rows, splits, y_out, phat_out, status, stream) != cudaSuccess) return EGTP_ERR_CUDA;
  return EGTP_OK;
}
