// The interpreter kernel exists in many template variants (elements per thread, parameter-block size, one
// program or a stacked launch, extension level, level waits).  They are compiled in separate translation units
// (dvm_vm_inst.cu, once per group) so that the library builds in parallel; the launch code reaches them through
// this table of plain functions.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>

constexpr int DVM_PW_SMALL = 496;    // words of code in a 2 KB parameter block
constexpr int DVM_PW_LARGE = 8000;   // ... in a 32 KB parameter block (the limit is 32764 bytes)

struct DvmVmVariant {
  int V;        // elements of a tile register per thread: 16, 24 or 32
  int large;    // 1: the 32 KB parameter block
  int single;   // 1: one program per launch (dvm_launch)
  int ext;      // 0 basic, 1 + Cmp / Select / Pow / IsFinite, 2 + views
  int levels;   // 1: stacked launch with waits between dependent levels
  int lean;     // 1: the lean kernel for the basic instruction set (no level waits, no wrap-around rows); 2: its variant
                // for phased programs (rows longer than a tile, DVM_OP_PHASE; one program per launch); 3: the
                // one-program lean kernel for launches with two tile slots (the one-slot path compiled out); 4: that
                // for programs whose loads are all one thread's (no row-by-row copies, per-row scalar inputs, outer dims);
                // 5: that for programs all of whose operands are aligned like the tile's chunks (no realignment of reads);
                // 6: two slots and aligned operands, row-by-row copies allowed; 7: as 5 for programs whose rows fill the
                // tile's slots exactly (no slot masks); 8: as 6 for such programs; 9: aligned programs with one tile slot (three CTAs)
  int heavy;    // unary functions log / erf / tanh / sqrt / floor / round on tiles: 1 present, 0 absent (lean only)
  int ctas;     // resident CTAs per SM the kernel is compiled for: 2, or 3 (variants for one-slot launches)
  // launches the kernel; `params` points at a dvm::VMParams<PW> of the variant's block size
  cudaError_t (*launch)(const void* params, int grid, size_t smem, cudaStream_t stream);
  // lifts the dynamic shared memory limit of the kernel and asks how many CTAs of it an SM holds
  cudaError_t (*occupancy)(size_t smem, size_t max_smem, int* ctas_per_sm);
};

// NULL when the library has no such variant.
const DvmVmVariant* dvm_vm_find_variant(int V, bool large, bool single, int ext, bool levels, int lean, bool heavy, int ctas = 2);
