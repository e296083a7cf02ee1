// Matmul meta-kernel (placeholder until the tcgen05 path lands): reports "unsupported".
#include "../../include/dvm.h"
#include "dvm_format.h"
#include "dvm_internal.h"
#include "dvm_launch.h"

int dvm_encode_matmul(const dvm_program*, const dvm_shape*, int, const float*, int, void*, size_t, size_t*,
                      dvm_shape*, int) {
  return DVM_ERR_UNSUPPORTED;
}
int dvm_verify_matmul(const uint32_t*, size_t) { return DVM_ERR_BAD_CODE; }
int dvm_disassemble_matmul(const uint32_t*, size_t, char*, size_t) { return DVM_ERR_BAD_CODE; }
int dvm_launch_matmul(const uint32_t*, size_t, void* const*, int, cudaStream_t) { return DVM_ERR_UNSUPPORTED; }
