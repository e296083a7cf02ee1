// Declarations shared by the translation units of libdvm (not part of the ABI).
#pragma once
#include <stddef.h>
#include <stdint.h>

#include "../../include/dvm.h"

int dvm_encode_matmul(const dvm_program* p, const dvm_shape* in_shapes, int n_in, const float* scalars,
                      int n_scalars, void* code, size_t code_capacity, size_t* code_size,
                      dvm_shape* out_shapes, int n_out);
int dvm_verify_matmul(const uint32_t* w, size_t n_words);
int dvm_disassemble_matmul(const uint32_t* w, size_t n_words, char* buf, size_t cap);
