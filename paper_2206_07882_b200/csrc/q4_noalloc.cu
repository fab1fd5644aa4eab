// qjoint_logprobs_static: the joint network with its scratch held inside the library.
//
// Some callers cannot hand the library a workspace because they cannot allocate device memory
// at the point of the call: a real-time decoding thread that must never block on the
// allocator's device-wide synchronisation, a host application that gives a plug-in a fixed
// memory budget at start-up and forbids later cudaMalloc calls, or code that runs while another
// thread of the process is capturing a stream (an allocation would invalidate that capture).
// For them the scratch of the joint network lives in a fixed-size array in device memory that
// is part of the library image.
#include <mutex>

#include "q4_internal.h"

using namespace q4;

// Largest problem the built-in scratch serves: N * D <= Q4_JOINT_STATIC_MAX_ND elements.
#define Q4_JOINT_STATIC_MAX_ND 65536
#define Q4_JOINT_STATIC_BYTES (Q4_JOINT_STATIC_MAX_ND * 5 + 512)

// Every GPU that loads the library holds this array until the process exits.
static __device__ __align__(256) unsigned char g_joint_scratch[Q4_JOINT_STATIC_BYTES];

namespace {
constexpr int kMaxDevices = 64;
void* g_scratch_ptr[kMaxDevices];   // device address of g_joint_scratch, per device
std::once_flag g_scratch_once[kMaxDevices];

// The array's name is only a host-side handle; the device address has to be asked for, once
// per device, with that device current.  Host threads that make their first call at the same
// time are serialised by the once-flag, and a thread that finds the flag set also sees the
// stored address.  The address stays valid until the device is reset (cudaDeviceReset): after
// a reset the library must be reloaded before this entry point is used again.
int scratch_for_current_device(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return Q4_ERR_CUDA;
  std::call_once(g_scratch_once[dev], [dev]() {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_joint_scratch) == cudaSuccess) g_scratch_ptr[dev] = p;
  });
  if (g_scratch_ptr[dev] == nullptr) return Q4_ERR_CUDA;
  *out = g_scratch_ptr[dev];
  return Q4_OK;
}
}  // namespace

extern "C" int qjoint_logprobs_static(const float* e, const int32_t* frame_idx, const void* pq,
                                      const q4_act* p_act, int32_t N, const q4_mat* w_pred,
                                      const float* b_pred, const q4_act* z_act, const q4_mat* w_out,
                                      const float* b_out, float* logp, q4_stream stream) {
  if (!w_pred || N < 0) return w_pred ? Q4_ERR_DIM : Q4_ERR_NULL;
  const long long nd = (long long)N * w_pred->rows;
  if (w_pred->rows <= 0 || nd > Q4_JOINT_STATIC_MAX_ND) return Q4_ERR_WORKSPACE;
  void* scratch = nullptr;
  const int r = scratch_for_current_device(&scratch);
  if (r != Q4_OK) return r;
  // Same kernels as qjoint_logprobs; every scratch element that is read is written first by
  // the call itself, so nothing has to be cleared between calls.
  return qjoint_logprobs(e, frame_idx, pq, p_act, N, w_pred, b_pred, z_act, w_out, b_out, logp, nullptr, nullptr,
                         scratch, Q4_JOINT_STATIC_BYTES, stream);
}
