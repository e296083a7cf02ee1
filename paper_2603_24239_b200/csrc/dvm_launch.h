// Launch-side declarations shared by the CUDA translation units of libdvm (not part of the ABI).
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

// Device status word values (read back by dvm_last_device_status).
namespace dvm {
enum { ST_OK = 0, ST_BAD_CODE = 1, ST_TIMEOUT = 2 };
}

// Records a failed CUDA runtime call (dvm_last_cuda_error) and returns DVM_ERR_CUDA from the caller.
#define DVM_CUDA(call)                \
  do {                                \
    cudaError_t e_ = (call);          \
    if (e_ != cudaSuccess) {          \
      dvm_note_cuda_error((int)e_);   \
      return DVM_ERR_CUDA;            \
    }                                 \
  } while (0)

struct DvmDeviceInfo {
  unsigned int* scratch;  // library-owned device words: [0] status, then work-queue counter pairs
  int sm_count;
  unsigned queue_slot;    // work-queue slot reserved for this launch
};

// Per-device lazy set-up (scratch allocation, occupancy) for the current device.
int dvm_device_state(DvmDeviceInfo* info);
void dvm_note_cuda_error(int e);
void dvm_count_launch();

int dvm_launch_matmul(const uint32_t* code, size_t n_words, void* const* tensors, int n_tensors,
                      cudaStream_t stream);
