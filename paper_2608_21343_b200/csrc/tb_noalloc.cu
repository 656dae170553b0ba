// tb_greedy_decode_noalloc: unboosted greedy decoding for callers that must not allocate device
// memory.  The general decode kernel needs a little device memory of its own besides the caller's
// inputs and outputs -- a status word and one slot record per stream saying "no graph bound".  The
// normal entry points keep these in a tb_batch, which tb_batch_create allocates; this file keeps
// them in a fixed array that is part of the library image instead.
#include <cstring>
#include <mutex>

#include "tb_launch.h"

namespace {

constexpr int kMaxStreams = TB_NOALLOC_MAX_STREAMS;
constexpr size_t kStatusBytes = 256;  // the status word sits alone in the first 256 bytes
constexpr size_t kScratchBytes = kStatusBytes + sizeof(TbSlotRec) * kMaxStreams;

// Scratch of the no-allocation entry point: [status word | kMaxStreams slot records].  Every GPU
// that loads the library holds these 33 KB until the process exits.  In host code this name is
// only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
unsigned char* g_scratch_ptr[kMaxDevices] = {};  // device address of g_noalloc_scratch, per device

// Device address of the scratch array on `device` (which must be current).  Looked up once per device.
int scratch_for_device(int device, unsigned char** out) {
  if (device < 0 || device >= kMaxDevices) return TB_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(g_mutex);
  if (!g_scratch_ptr[device]) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || !ptr) {
      cudaGetLastError();
      return TB_ERR_CUDA;
    }
    g_scratch_ptr[device] = static_cast<unsigned char*>(ptr);
  }
  *out = g_scratch_ptr[device];
  return TB_OK;
}

}  // namespace

extern "C" int tb_greedy_decode_noalloc(int device, const void* logits, int dtype, int32_t B, int32_t T, int32_t S,
                                        int32_t vocab, const int64_t* strides, const int32_t* lengths,
                                        int32_t* out_tokens, int32_t* out_frames, int32_t* out_counts,
                                        float* out_scores, int32_t* out_states, int32_t* out_status, void* stream_) {
  if (!logits || !strides || !out_tokens || !out_frames || !out_counts || !out_scores || !out_states) return TB_ERR_INVALID_ARG;
  if (dtype != TB_BF16 && dtype != TB_F32) return TB_ERR_INVALID_ARG;
  if (B < 1 || B > kMaxStreams || T < 1 || S < 1 || vocab < 1 || vocab > TB_MAX_VOCAB) return TB_ERR_INVALID_ARG;
  if (static_cast<int64_t>(T) * S > INT32_MAX) return TB_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  int prev = -1;
  if (cudaGetDevice(&prev) != cudaSuccess) { cudaGetLastError(); return TB_ERR_CUDA; }
  if (prev != device && cudaSetDevice(device) != cudaSuccess) { cudaGetLastError(); return TB_ERR_CUDA; }
  unsigned char* scratch = nullptr;
  int rc = scratch_for_device(device, &scratch);
  if (rc == TB_OK) {
    // The array keeps whatever the previous call left: the status word must start at zero, and the
    // slot records must read "unbound" (all zero), so both are cleared in stream order.
    if (cudaMemsetAsync(scratch, 0, kStatusBytes + sizeof(TbSlotRec) * static_cast<size_t>(B), stream) != cudaSuccess) {
      cudaGetLastError();
      rc = TB_ERR_CUDA;
    }
  }
  if (rc == TB_OK) {
    TbDecodeParams p;
    std::memset(&p, 0, sizeof p);
    p.logits = logits; p.dtype = dtype; p.n_streams = B; p.frames = T; p.S = S; p.V = vocab; p.n_dur = 0;
    p.C = 1;  // no class is ever looked up: every stream is unbound
    p.sb = strides[0]; p.st = strides[1]; p.ss = strides[2]; p.sv = strides[3];
    p.lengths = lengths; p.persistent = 0;
    p.out_tokens = out_tokens; p.out_frames = out_frames; p.out_counts = out_counts;
    p.out_scores = out_scores; p.out_states = out_states; p.out_cap = T * S;
    p.slots = reinterpret_cast<const TbSlotRec*>(scratch + kStatusBytes);
    p.sstate = nullptr; p.arena = nullptr; p.cls = nullptr;
    p.status = reinterpret_cast<int32_t*>(scratch);
    rc = tb_launch_decode_general(p, stream);
  }
  if (rc == TB_OK && out_status &&
      cudaMemcpyAsync(out_status, scratch, sizeof(int32_t), cudaMemcpyDeviceToDevice, stream) != cudaSuccess) {
    cudaGetLastError();
    rc = TB_ERR_CUDA;
  }
  if (prev != device) cudaSetDevice(prev);
  return rc;
}
