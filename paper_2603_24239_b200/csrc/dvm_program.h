// The operator program as the library holds it (private to libdvm; the ABI sees an opaque handle).
#pragma once
#include <stdint.h>

#include "../../include/dvm.h"
#include "dvm_format.h"

enum NodeKind : uint8_t { NK_INPUT, NK_UNARY, NK_BINARY, NK_SCALAR, NK_CAST, NK_REDUCE, NK_MATMUL, NK_COMPARE, NK_SELECT };

struct Node {
  uint8_t kind;
  uint8_t op;
  uint8_t dtype;
  int8_t rank;
  int16_t x, y;
  int16_t param;  // NK_SCALAR: >= 0: the scalar comes from the runtime argument list; NK_SELECT: the third operand
  float imm;
};

struct OutputRef {
  int16_t value;
  uint8_t dtype;
};

struct dvm_program {
  Node nodes[DVM_MAX_NODES];
  int n_nodes;
  int16_t inputs[DVM_MAX_TENSORS];
  int n_inputs;
  OutputRef outputs[DVM_MAX_TENSORS];
  int n_outputs;
  int n_params;
  int n_matmul;
  bool finalized;
};
