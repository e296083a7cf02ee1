// Instantiations of the interpreter kernel, one group per compilation of this file (-DDVM_INST_GROUP=g):
// group g < 12: V = 16 (g < 6) or 32, parameter block small (g % 6 < 3) or large, extension level g % 3,
// each with the one-program, the stacked and the level-wait variant; group 12: the 24-element one-program
// basic variants; groups 13..16: the lean kernel for V = 16 (13, 14) or 32, parameter block small (13, 15) or
// large, each one-program / stacked, with and without the heavy unary functions; group 17: the lean kernel with
// 24 elements per thread (one program); group 18: the lean kernel for phased programs; groups 19..30: the level-wait
// variant of groups 0..11 compiled for three resident CTAs per SM; group 31: the one-program lean kernel, 16 elements
// per thread, compiled for three; groups 32..34: the one-program lean kernel with 16 / 32 / 24 elements per thread
// for launches with two tile slots (its one-slot path compiled out); groups 35..37: the same for programs whose
// loads are all one thread's; groups 38..40: ... and whose operands are all aligned like the tile's chunks; groups 41..43: two slots, aligned rows,
// row-by-row copies allowed; groups 44..46: groups 38..40 for programs whose rows fill the tile's slots exactly; groups 47..49: groups
// 41..43 for such programs; group 50: group 31's kernel for aligned programs.
#include "dvm_vm.cuh"
#include "dvm_vm_lean.cuh"
#include "dvm_vm_variants.h"

#ifndef DVM_INST_GROUP
#error "compile with -DDVM_INST_GROUP=<0..50>"
#endif

namespace {

template <int V, int PW, bool SINGLE, int EXT, bool LEVELS, int CTAS = DVM_VM_MIN_CTAS>
struct Ops {
  static cudaError_t launch(const void* params, int grid, size_t smem, cudaStream_t stream) {
    dvm::dvm_vm_kernel<V, PW, SINGLE, EXT, LEVELS, CTAS>
        <<<grid, dvm::THREADS, smem, stream>>>(*static_cast<const dvm::VMParams<PW>*>(params));
    return cudaGetLastError();
  }
  static cudaError_t occupancy(size_t smem, size_t max_smem, int* n) {
    cudaError_t e = cudaFuncSetAttribute(dvm::dvm_vm_kernel<V, PW, SINGLE, EXT, LEVELS, CTAS>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)max_smem);
    if (e != cudaSuccess) return e;
    return cudaOccupancyMaxActiveBlocksPerMultiprocessor(n, dvm::dvm_vm_kernel<V, PW, SINGLE, EXT, LEVELS, CTAS>,
                                                         dvm::THREADS, smem);
  }
};

template <int V, int PW, bool SINGLE, bool HEAVY, bool PHASED = false, int CTAS = DVM_LEAN_MIN_CTAS, bool TWO = false, bool DENSE = false,
          bool AL = false, bool FULL = false>
struct LeanOps {
  static cudaError_t launch(const void* params, int grid, size_t smem, cudaStream_t stream) {
    dvm::dvm_vm_lean_kernel<V, PW, SINGLE, HEAVY, PHASED, CTAS, TWO, DENSE, AL, FULL>
        <<<grid, dvm::THREADS, smem, stream>>>(*static_cast<const dvm::VMParams<PW>*>(params));
    return cudaGetLastError();
  }
  static cudaError_t occupancy(size_t smem, size_t max_smem, int* n) {
    cudaError_t e = cudaFuncSetAttribute(dvm::dvm_vm_lean_kernel<V, PW, SINGLE, HEAVY, PHASED, CTAS, TWO, DENSE, AL, FULL>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)max_smem);
    if (e != cudaSuccess) return e;
    return cudaOccupancyMaxActiveBlocksPerMultiprocessor(n, dvm::dvm_vm_lean_kernel<V, PW, SINGLE, HEAVY, PHASED, CTAS, TWO, DENSE, AL, FULL>,
                                                         dvm::THREADS, smem);
  }
};

#define DVM_LEAN_PHASED(V, LARGE, HEAVY)                                                  \
  {V, LARGE, 1, 0, 0, 2, HEAVY, 2,                                                        \
   &LeanOps<V, (LARGE) ? DVM_PW_LARGE : DVM_PW_SMALL, true, (HEAVY) != 0, true>::launch,  \
   &LeanOps<V, (LARGE) ? DVM_PW_LARGE : DVM_PW_SMALL, true, (HEAVY) != 0, true>::occupancy}

// the one-program lean kernel for launches with two tile slots (lean = 3: its one-slot path compiled out)
#define DVM_LEAN_TWO(V, LARGE, HEAVY)                                                               \
  {V, LARGE, 1, 0, 0, 3, HEAVY, 2,                                                                  \
   &LeanOps<V, (LARGE) ? DVM_PW_LARGE : DVM_PW_SMALL, true, (HEAVY) != 0, false, 2, true>::launch,  \
   &LeanOps<V, (LARGE) ? DVM_PW_LARGE : DVM_PW_SMALL, true, (HEAVY) != 0, false, 2, true>::occupancy}

// ... and for programs whose loads are all one thread's (lean = 4: also without row-by-row copies, per-row scalar inputs, outer dims)
#define DVM_LEAN_TWO_DENSE(V, LARGE, HEAVY)                                                               \
  {V, LARGE, 1, 0, 0, 4, HEAVY, 2,                                                                        \
   &LeanOps<V, (LARGE) ? DVM_PW_LARGE : DVM_PW_SMALL, true, (HEAVY) != 0, false, 2, true, true>::launch,  \
   &LeanOps<V, (LARGE) ? DVM_PW_LARGE : DVM_PW_SMALL, true, (HEAVY) != 0, false, 2, true, true>::occupancy}

// ... all of whose operands are aligned like the tile's chunks (lean = 5: also without the realignment of reads)
#define DVM_LEAN_TWO_DENSE_AL(V, LARGE, HEAVY)                                                                  \
  {V, LARGE, 1, 0, 0, 5, HEAVY, 2,                                                                              \
   &LeanOps<V, (LARGE) ? DVM_PW_LARGE : DVM_PW_SMALL, true, (HEAVY) != 0, false, 2, true, true, true>::launch,  \
   &LeanOps<V, (LARGE) ? DVM_PW_LARGE : DVM_PW_SMALL, true, (HEAVY) != 0, false, 2, true, true, true>::occupancy}

// ... for programs with row-by-row copies whose rows are all aligned like the tile's chunks (lean = 6)
#define DVM_LEAN_TWO_AL(V, LARGE, HEAVY)                                                                         \
  {V, LARGE, 1, 0, 0, 6, HEAVY, 2,                                                                               \
   &LeanOps<V, (LARGE) ? DVM_PW_LARGE : DVM_PW_SMALL, true, (HEAVY) != 0, false, 2, true, false, true>::launch,  \
   &LeanOps<V, (LARGE) ? DVM_PW_LARGE : DVM_PW_SMALL, true, (HEAVY) != 0, false, 2, true, false, true>::occupancy}

// ... dense, aligned programs whose rows fill the tile's slots exactly (lean = 7: also without the slot masks)
#define DVM_LEAN_TWO_DENSE_AL_FULL(V, LARGE, HEAVY)                                                                   \
  {V, LARGE, 1, 0, 0, 7, HEAVY, 2,                                                                                    \
   &LeanOps<V, (LARGE) ? DVM_PW_LARGE : DVM_PW_SMALL, true, (HEAVY) != 0, false, 2, true, true, true, true>::launch,  \
   &LeanOps<V, (LARGE) ? DVM_PW_LARGE : DVM_PW_SMALL, true, (HEAVY) != 0, false, 2, true, true, true, true>::occupancy}

// ... aligned programs with row-by-row copies whose rows fill the tile's slots exactly (lean = 8)
#define DVM_LEAN_TWO_AL_FULL(V, LARGE, HEAVY)                                                                          \
  {V, LARGE, 1, 0, 0, 8, HEAVY, 2,                                                                                     \
   &LeanOps<V, (LARGE) ? DVM_PW_LARGE : DVM_PW_SMALL, true, (HEAVY) != 0, false, 2, true, false, true, true>::launch,  \
   &LeanOps<V, (LARGE) ? DVM_PW_LARGE : DVM_PW_SMALL, true, (HEAVY) != 0, false, 2, true, false, true, true>::occupancy}

// the one-program lean kernel compiled for three resident CTAs (one-slot programs) for aligned programs (lean = 9)
#define DVM_LEAN3_AL(V, LARGE, HEAVY)                                                                       \
  {V, LARGE, 1, 0, 0, 9, HEAVY, 3,                                                                                \
   &LeanOps<V, (LARGE) ? DVM_PW_LARGE : DVM_PW_SMALL, true, (HEAVY) != 0, false, 3, false, false, true>::launch,   \
   &LeanOps<V, (LARGE) ? DVM_PW_LARGE : DVM_PW_SMALL, true, (HEAVY) != 0, false, 3, false, false, true>::occupancy}

#define DVM_LEAN(V, LARGE, SINGLE, HEAVY)                                                   \
  {V, LARGE, SINGLE, 0, 0, 1, HEAVY, 2,                                                     \
   &LeanOps<V, (LARGE) ? DVM_PW_LARGE : DVM_PW_SMALL, (SINGLE) != 0, (HEAVY) != 0>::launch, \
   &LeanOps<V, (LARGE) ? DVM_PW_LARGE : DVM_PW_SMALL, (SINGLE) != 0, (HEAVY) != 0>::occupancy}

#define DVM_ENTRY(V, LARGE, SINGLE, EXT, LEVELS)                                       \
  {V, LARGE, SINGLE, EXT, LEVELS, 0, 1, 2,                                            \
   &Ops<V, (LARGE) ? DVM_PW_LARGE : DVM_PW_SMALL, (SINGLE) != 0, EXT, (LEVELS) != 0>::launch, \
   &Ops<V, (LARGE) ? DVM_PW_LARGE : DVM_PW_SMALL, (SINGLE) != 0, EXT, (LEVELS) != 0>::occupancy}

// the level-wait variant compiled for three resident CTAs (one-slot launches)
#define DVM_ENTRY3(V, LARGE, EXT)                                                      \
  {V, LARGE, 0, EXT, 1, 0, 1, 3,                                                      \
   &Ops<V, (LARGE) ? DVM_PW_LARGE : DVM_PW_SMALL, false, EXT, true, 3>::launch,       \
   &Ops<V, (LARGE) ? DVM_PW_LARGE : DVM_PW_SMALL, false, EXT, true, 3>::occupancy}
// the one-program lean kernel compiled for three resident CTAs (one-slot programs)
#define DVM_LEAN3(V, LARGE, HEAVY)                                                          \
  {V, LARGE, 1, 0, 0, 1, HEAVY, 3,                                                          \
   &LeanOps<V, (LARGE) ? DVM_PW_LARGE : DVM_PW_SMALL, true, (HEAVY) != 0, false, 3>::launch, \
   &LeanOps<V, (LARGE) ? DVM_PW_LARGE : DVM_PW_SMALL, true, (HEAVY) != 0, false, 3>::occupancy}

#if DVM_INST_GROUP < 12
constexpr int GV = DVM_INST_GROUP < 6 ? 16 : 32;
constexpr int GL = (DVM_INST_GROUP % 6) < 3 ? 0 : 1;
constexpr int GE = DVM_INST_GROUP % 3;
const DvmVmVariant kGroup[] = {DVM_ENTRY(GV, GL, 1, GE, 0), DVM_ENTRY(GV, GL, 0, GE, 0), DVM_ENTRY(GV, GL, 0, GE, 1)};
#elif DVM_INST_GROUP >= 19 && DVM_INST_GROUP < 31
constexpr int G3 = DVM_INST_GROUP - 19;
constexpr int GV = G3 < 6 ? 16 : 32;
constexpr int GL = (G3 % 6) < 3 ? 0 : 1;
constexpr int GE = G3 % 3;
const DvmVmVariant kGroup[] = {DVM_ENTRY3(GV, GL, GE)};
#elif DVM_INST_GROUP == 31
const DvmVmVariant kGroup[] = {DVM_LEAN3(16, 0, 0), DVM_LEAN3(16, 0, 1), DVM_LEAN3(16, 1, 0), DVM_LEAN3(16, 1, 1)};
#elif DVM_INST_GROUP == 50
const DvmVmVariant kGroup[] = {DVM_LEAN3_AL(16, 0, 0), DVM_LEAN3_AL(16, 0, 1), DVM_LEAN3_AL(16, 1, 0), DVM_LEAN3_AL(16, 1, 1)};
#elif DVM_INST_GROUP >= 47
constexpr int GV = DVM_INST_GROUP == 47 ? 16 : (DVM_INST_GROUP == 48 ? 32 : 24);
const DvmVmVariant kGroup[] = {DVM_LEAN_TWO_AL_FULL(GV, 0, 0), DVM_LEAN_TWO_AL_FULL(GV, 0, 1), DVM_LEAN_TWO_AL_FULL(GV, 1, 0), DVM_LEAN_TWO_AL_FULL(GV, 1, 1)};
#elif DVM_INST_GROUP >= 44
constexpr int GV = DVM_INST_GROUP == 44 ? 16 : (DVM_INST_GROUP == 45 ? 32 : 24);
const DvmVmVariant kGroup[] = {DVM_LEAN_TWO_DENSE_AL_FULL(GV, 0, 0), DVM_LEAN_TWO_DENSE_AL_FULL(GV, 0, 1), DVM_LEAN_TWO_DENSE_AL_FULL(GV, 1, 0),
                               DVM_LEAN_TWO_DENSE_AL_FULL(GV, 1, 1)};
#elif DVM_INST_GROUP >= 41
constexpr int GV = DVM_INST_GROUP == 41 ? 16 : (DVM_INST_GROUP == 42 ? 32 : 24);
const DvmVmVariant kGroup[] = {DVM_LEAN_TWO_AL(GV, 0, 0), DVM_LEAN_TWO_AL(GV, 0, 1), DVM_LEAN_TWO_AL(GV, 1, 0), DVM_LEAN_TWO_AL(GV, 1, 1)};
#elif DVM_INST_GROUP >= 38
constexpr int GV = DVM_INST_GROUP == 38 ? 16 : (DVM_INST_GROUP == 39 ? 32 : 24);
const DvmVmVariant kGroup[] = {DVM_LEAN_TWO_DENSE_AL(GV, 0, 0), DVM_LEAN_TWO_DENSE_AL(GV, 0, 1), DVM_LEAN_TWO_DENSE_AL(GV, 1, 0), DVM_LEAN_TWO_DENSE_AL(GV, 1, 1)};
#elif DVM_INST_GROUP >= 35
constexpr int GV = DVM_INST_GROUP == 35 ? 16 : (DVM_INST_GROUP == 36 ? 32 : 24);
const DvmVmVariant kGroup[] = {DVM_LEAN_TWO_DENSE(GV, 0, 0), DVM_LEAN_TWO_DENSE(GV, 0, 1), DVM_LEAN_TWO_DENSE(GV, 1, 0), DVM_LEAN_TWO_DENSE(GV, 1, 1)};
#elif DVM_INST_GROUP >= 32
constexpr int GV = DVM_INST_GROUP == 32 ? 16 : (DVM_INST_GROUP == 33 ? 32 : 24);
const DvmVmVariant kGroup[] = {DVM_LEAN_TWO(GV, 0, 0), DVM_LEAN_TWO(GV, 0, 1), DVM_LEAN_TWO(GV, 1, 0), DVM_LEAN_TWO(GV, 1, 1)};
#elif DVM_INST_GROUP == 12
const DvmVmVariant kGroup[] = {DVM_ENTRY(24, 0, 1, 0, 0), DVM_ENTRY(24, 1, 1, 0, 0)};
#elif DVM_INST_GROUP < 17
constexpr int GV = DVM_INST_GROUP < 15 ? 16 : 32;
constexpr int GL = (DVM_INST_GROUP - 13) % 2;
const DvmVmVariant kGroup[] = {DVM_LEAN(GV, GL, 1, 0), DVM_LEAN(GV, GL, 1, 1), DVM_LEAN(GV, GL, 0, 0), DVM_LEAN(GV, GL, 0, 1)};
#elif DVM_INST_GROUP == 17
const DvmVmVariant kGroup[] = {DVM_LEAN(24, 0, 1, 0), DVM_LEAN(24, 0, 1, 1), DVM_LEAN(24, 1, 1, 0), DVM_LEAN(24, 1, 1, 1)};
#else
// phased programs (rows longer than a tile) are encoded with 32 elements per thread
const DvmVmVariant kGroup[] = {DVM_LEAN_PHASED(32, 0, 0), DVM_LEAN_PHASED(32, 0, 1), DVM_LEAN_PHASED(32, 1, 0), DVM_LEAN_PHASED(32, 1, 1)};
#endif

}  // namespace

#define DVM_CAT_(a, b) a##b
#define DVM_CAT(a, b) DVM_CAT_(a, b)
// each group exports its table under a name of its own: dvm_vm_group_<g>(&count)
const DvmVmVariant* DVM_CAT(dvm_vm_group_, DVM_INST_GROUP)(int* count) {
  *count = (int)(sizeof(kGroup) / sizeof(kGroup[0]));
  return kGroup;
}
