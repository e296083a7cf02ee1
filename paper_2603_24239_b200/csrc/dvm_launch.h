// Launch-side declarations shared by the CUDA translation units of libdvm (not part of the ABI).
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

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
